// Tensor-core (tcgen05) kernel for the logit tails when several hidden rows share one pass over the
// LM head: single-sequence verification (SL+1 rows), batched verification, batched draft steps.
//
//   D[r, v] = sum_k H[r, k] * W[v, k]      r on the 128 TMEM lanes, v on the TMEM columns
//
//   * warp 0   producer: one TMA box of H (A operand, up to 128 rows x 64 k) and one of W (B operand, up
//              to 256 vocabulary rows x 64 k) per stage, 128-byte swizzle, through a ring of
//              shared-memory stages;
//   * warp 1   issues tcgen05.mma (M = 128, N = rows of the vocabulary tile, K = 16 per instruction),
//              accumulating in one of two 256-column TMEM buffers; tcgen05.commit frees the stage;
//   * warps 2+ epilogue: tcgen05.ld 32 columns at a time; every thread owns one hidden row and walks
//              over the vocabulary columns, so the running arg-max (verification) or the running
//              soft-max statistics and top-10 values (draft step) live in its registers: no shuffles,
//              and the logits never leave the chip.  Two warps share each TMEM lane quadrant and
//              split the columns.
//
// A CTA keeps one tile of hidden rows (m_tile) and walks over a contiguous range of vocabulary
// tiles; CTAs that share a vocabulary tile run side by side, so the LM head crosses HBM once and is
// shared through L2.  Results leave the CTA as one atomicMax per row (verification) or one partial
// per row (draft step); small separate kernels finish the job.
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "stream_tail.cuh"  // verify_one_sequence, warp_halt_classifier
#include "group_merge.cuh"

namespace disco {

constexpr int kUmmaMaxStages = 16;
constexpr int kUmmaBK = 64;               // k elements per stage (one 128-byte swizzle span)
constexpr int kUmmaRingBytes = 192 * 1024;  // shared memory for the operand stages
constexpr int kUmmaEpiWarps = 8;
constexpr int kUmmaThreads = (2 + kUmmaEpiWarps) * 32;
constexpr int kUmmaXchBytes = 14 * 1024;  // 64-byte records handed between the warps that share a hidden row
// Draft step: the last bytes of the ring are left to the epilogue warps' candidate queues (16 entries per lane)
constexpr int kUmmaQueueEntries = 16;
constexpr int kUmmaQueueBytes = kUmmaEpiWarps * kUmmaQueueEntries * 32 * 4;
constexpr int kUmmaSmemBytes =
    kUmmaRingBytes + 1024 /*align*/ + 512 /*barriers*/ + kUmmaXchBytes;
// the draft step adds the classifier parameters behind the exchange area
inline int umma_clf_bytes(int clf_H) { return (clf_H * (kNFeat + 2) + 4) * 4; }

struct UmmaParams {
    int V, d, R;
    int MT;      // tiles of 128 hidden rows
    int CN;      // CTAs per m_tile (grid = MT * CN)
    int TPC;     // vocabulary tiles per CTA
    int TR;      // vocabulary rows per tile; the MMA and the TMA box use TRN = TR rounded up to 16
    int TRN;
    int a_rows;  // rows of the H box (multiple of 8, <= 128)
    // Draft step with at most 64 hidden rows: the H box is loaded `rep` times per stage, rows_pad rows
    // apart, so every TMEM lane quadrant holds a copy of each row and all epilogue warps share the columns.
    int rep;       // 1, 2 or 4
    int rows_pad;  // 128 / rep
    int stages;  // ring depth (<= kUmmaMaxStages); stage s holds an A tile of a_bytes and a B tile of b_bytes
    int a_bytes, b_bytes;  // multiples of 1024
    int* status;
    // verification
    unsigned long long* keys;  // [R]
    // draft step
    float4* part_rec;   // [R][CN] stamped records of 80 bytes
    float* probs;       // optional [R][V]: raw logits are written here
    // verification finished inside this kernel by the last CTA (few sequences only)
    int fuse_final;
    unsigned int* ticket;
    const int32_t* draft_ids;
    const int32_t* row_off;
    int B, SL;
    int32_t* n_accept;
    int32_t* bonus;
    int32_t* target_ids;
    VerifyPadded padded;   // sl != null: fixed-shape rows, per-sequence look-ahead read from the device
    // Verification whose row count is device memory (rows packed by the kernel before this one): R, MT, CN, TPC, TR
    // above are then upper bounds / unused, the kernel derives the tiling from *dev_R; TRN stays the box height of
    // the LM-head tensor map (256) and the MMAs take the tile height rounded up to 16.
    const int32_t* dev_R;
};

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_load_2d(void* dst_smem, const CUtensorMap* tmap, int c0, int c1, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
            smem_addr(dst_smem)),
        "l"(tmap), "r"(c0), "r"(c1), "r"(smem_addr(bar))
        : "memory");
}
// Bring one box of a tensor map into L2 (no shared-memory destination, nothing to wait for).
__device__ __forceinline__ void tma_prefetch_l2_2d(const CUtensorMap* tmap, int c0, int c1) {
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(tmap), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* tmap) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(tmap) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(dst_smem)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_addr(bar))
                 : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 32 lanes x 32 consecutive fp32 columns -> 32 registers per thread
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor: K-major tile, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_smem_desc(const void* tile) {
    uint64_t desc = 0;
    desc |= static_cast<uint64_t>((smem_addr(tile) & 0x3ffffu) >> 4);  // start address
    desc |= static_cast<uint64_t>(1) << 16;                            // leading byte offset (unused with swizzle)
    desc |= static_cast<uint64_t>(1024 >> 4) << 32;                    // stride byte offset
    desc |= static_cast<uint64_t>(1) << 46;                            // descriptor version
    desc |= static_cast<uint64_t>(2) << 61;                            // 128-byte swizzle
    return desc;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t umma_idesc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) | ((128u >> 4) << 24);
}

// Draft step, second phase: one warp per sequence merges the per-CTA partial records, forms the
// features of Eq. 2 and runs the halt classifier and the stopping rule.
struct DraftFinalParams {
    int B;
    const int32_t* pos;
    const int32_t* n_drafted;
    const uint8_t* active;
    const float* clf_W1;
    const float* clf_b1;
    const float* clf_w2;
    const float* clf_b2;
    int clf_H;
    float tau;
    int sl_max;
    int32_t* token;
    float* conf;
    uint8_t* halt;
    float* feats;
    float* final_stats;
    float* nll_sum;
    int stats_only;
    unsigned int* epoch;  // [0] launches completed so far (stamp of this launch = that + 1), [1] finishing warps done
    ChainLink chain;      // alive != null: this launch is one step of a draft phase chained on the device
    unsigned int test_stamp_skew;   // 0.  Tests: the finishing warps expect a stamp that no CTA writes, so their wait runs out
    // words that the kernel after this one counts in (the tickets of a verification with sampling): cleared here
    unsigned int* clear_words;
    int clear_n;
};

// One warp finishes sequence b from its NP partial records.  clf_s: classifier parameters in shared
// memory (W1, b1, w2, b2 in this order); fpos and n_drafted were fetched by the caller.
__device__ __forceinline__ void umma_finish_sequence(const DraftFinalParams& p, const float4* part_rec, int NP, int b,
                                                     bool active, float fpos, int n_drafted, float* feat16,
                                                     const float* clf_s, uint32_t stamp, int* status, int lane) {
    const MergedPartials mp =
        warp_merge_partials(part_rec + (size_t)b * NP * kStampedPieces, NP, feat16 + 16, lane, stamp, status,
                            p.stats_only != 1);
    if (!active) return;
    const int Hc = p.clf_H;
    const DraftOutputs o{p.token, p.conf, p.halt, p.feats, p.final_stats, p.nll_sum, p.stats_only, p.chain};
    warp_draft_epilogue(mp.st, mp.key, mp.sel, fpos, n_drafted, p.tau, p.sl_max, feat16, clf_s, clf_s + Hc * kNFeat,
                        clf_s + Hc * (kNFeat + 1), clf_s + Hc * (kNFeat + 2), Hc, b, o, lane);
}

// Vocabulary tile t covers rows [t * TR, min(V, (t + 1) * TR)).  The TMA box and the MMA take TRN >= TR
// rows; the extra rows (the next tile's first rows, or zero fill past V) land in columns the epilogue skips.
// ---------------------------------------------------------------------------------------------
// main kernel
// ---------------------------------------------------------------------------------------------
// DRAFT: soft-max statistics, top-10 and arg-max per row (draft step) instead of the arg-max alone
// (verification).  STATS (with DRAFT): no top-10 -- the target rows of a verification with sampling, whose
// second phase wants the statistics and the arg-max only.
template <bool DRAFT, bool STATS = false>
__global__ void __launch_bounds__(kUmmaThreads, 1)
umma_tail_kernel(const __grid_constant__ CUtensorMap tmap_W, const __grid_constant__ CUtensorMap tmap_H,
                 const UmmaParams p, const DraftFinalParams f) {
    extern __shared__ uint8_t smem_dyn[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
    uint8_t* a_tiles = smem;
    uint8_t* b_tiles = smem + p.stages * p.a_bytes;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + kUmmaRingBytes);
    uint64_t* empty = full + kUmmaMaxStages;
    uint64_t* tmem_full = empty + kUmmaMaxStages;
    uint64_t* tmem_empty = tmem_full + 2;
    uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(tmem_empty + 2);
    float4* xch = reinterpret_cast<float4*>(reinterpret_cast<uint8_t*>(full) + 512);
    float* clf_s = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(xch) + kUmmaXchBytes);  // draft step only

    // the next kernel of the stream may begin its prologue; this one touches what its predecessor may
    // have written (hidden states, scratch) only after griddepcontrol.wait
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int KB = (p.d + kUmmaBK - 1) / kUmmaBK;
    // tiling: from the host, or (row count in device memory) derived here by the same rule
    int gR = p.R, gMT = p.MT, gCN = p.CN, gTPC = p.TPC, gTR = p.TR, gTRN = p.TRN;
    bool idle = false;
    if (!DRAFT && p.dev_R) {
        asm volatile("griddepcontrol.wait;" ::: "memory");   // the count is the predecessor's output
        gR = min(max(__ldcg(p.dev_R), 1), p.R);
        gMT = (gR + 127) / 128;
        gCN = (int)gridDim.x / gMT;
        gTPC = max(1, (p.V + 256 * gCN - 1) / (256 * gCN));
        gTR = (p.V + gCN * gTPC - 1) / (gCN * gTPC);
        gTRN = max(16, (gTR + 15) / 16 * 16);
        idle = (int)blockIdx.x >= gMT * gCN;
    }
    const int m_tile = blockIdx.x % gMT;
    const int nslot = blockIdx.x / gMT;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&tmem_full[b], 1);
            mbar_init(&tmem_empty[b], kUmmaEpiWarps);
        }
        fence_mbar_init();
        prefetch_tensormap(&tmap_W);
        prefetch_tensormap(&tmap_H);
    }
    if (warp == 1) {
        tmem_alloc(tmem_base_s, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_base_s;

    // A chained draft step in which no sequence drafts any more has nothing to do.  Every warp finds that out
    // by itself, after the dependency wait (the flags are the predecessor's output), and goes to the exit.
    bool live = !idle;   // (a CTA beyond the tiling derived from the device-side row count has nothing to do either)
    if (DRAFT && f.chain.alive != nullptr && f.chain.step > 1) {
        asm volatile("griddepcontrol.wait;" ::: "memory");
        live = chain_any_live(f.chain, f.B, lane);
    }

    if (warp == 0) {
        // ------------------------------ producer ------------------------------
        if (lane == 0 && live) {
            int stage = 0, phase = 0;
            const uint32_t bytes = (uint32_t)(p.rep * p.a_rows + p.TRN) * 128u;   // the boxes of the two tensor maps
            // The LM head is never written by this library: its first tiles are requested before the
            // dependency wait, the hidden-state tiles of the same stages right after it.
            int pre = 0;
            {
                const int v0 = nslot * gTPC * gTR;
                if (v0 < p.V) {
                    pre = min(p.stages, KB);
                    for (int kb = 0; kb < pre; ++kb) {
                        mbar_arrive_expect_tx(&full[kb], bytes);
                        tma_load_2d(b_tiles + kb * p.b_bytes, &tmap_W, kb * kUmmaBK, v0, &full[kb]);
                    }
                }
            }
            asm volatile("griddepcontrol.wait;" ::: "memory");
            int n = 0;
            for (int i = 0; i < gTPC; ++i) {
                const int v0 = (nslot * gTPC + i) * gTR;
                if (v0 >= p.V) break;
                for (int kb = 0; kb < KB; ++kb, ++n) {
                    if (n >= pre) {
                        mbar_wait(&empty[stage], phase ^ 1, p.status);
                        mbar_arrive_expect_tx(&full[stage], bytes);
                        tma_load_2d(b_tiles + stage * p.b_bytes, &tmap_W, kb * kUmmaBK, v0, &full[stage]);
                    }
                    for (int c = 0; c < p.rep; ++c)
                        tma_load_2d(a_tiles + stage * p.a_bytes + c * p.rows_pad * 128, &tmap_H, kb * kUmmaBK,
                                    m_tile * 128, &full[stage]);
                    if (++stage == p.stages) {
                        stage = 0;
                        phase ^= 1;
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0 && live) {
            int stage = 0, phase = 0, it = 0;
            const uint32_t idesc = umma_idesc(gTRN);
            for (int i = 0; i < gTPC; ++i) {
                if ((nslot * gTPC + i) * gTR >= p.V) break;
                const int buf = it & 1;
                mbar_wait(&tmem_empty[buf], ((it >> 1) & 1) ^ 1, p.status);
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * 256;
                for (int kb = 0; kb < KB; ++kb) {
                    mbar_wait(&full[stage], phase, p.status);
                    tc_fence_after();
                    const uint64_t a_desc = umma_smem_desc(a_tiles + stage * p.a_bytes);
                    const uint64_t b_desc = umma_smem_desc(b_tiles + stage * p.b_bytes);
#pragma unroll
                    for (int k = 0; k < kUmmaBK / 16; ++k)  // 16 k-elements = 32 bytes = 2 descriptor units
                        tc_mma_bf16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0);
                    tc_commit(&empty[stage]);
                    if (++stage == p.stages) {
                        stage = 0;
                        phase ^= 1;
                    }
                }
                tc_commit(&tmem_full[buf]);
                ++it;
            }
        }
    } else if (live) {
        // ------------------------------ epilogue ------------------------------
        asm volatile("griddepcontrol.wait;" ::: "memory");  // scratch and outputs belong to the predecessor until now
        const int ew = warp - 2;            // 0 .. kUmmaEpiWarps-1
        if (DRAFT && blockIdx.x == 0)
            for (int i = ew * 32 + lane; i < f.clear_n; i += kUmmaEpiWarps * 32) f.clear_words[i] = 0u;
        const int quad = warp & 3;          // TMEM lane quadrant this warp may read
        // The warps that hold the same hidden rows (two per quadrant, times the copies of the rows in
        // other quadrants) split the columns of a tile into `nshare` shares.
        const int tile_row = (quad * 32) % p.rows_pad + lane;     // row within this tile of hidden rows
        const int share = (ew >> 2) * p.rep + (quad * 32) / p.rows_pad;
        const int nshare = 2 * p.rep;
        const int row = m_tile * 128 + tile_row;
        const bool warp_has_rows = (m_tile * 128 + (quad * 32) % p.rows_pad) < gR;
        const bool valid = row < gR;
        // the optional probs output receives the raw logits of this row, unless the sequence is masked
        const bool keep_logits = DRAFT && p.probs && valid && (!f.active || f.active[row]);
        // stamp of this launch (the word is advanced by the last warp of the second phase)
        uint32_t stamp = 0u;
        if (DRAFT) stamp = *reinterpret_cast<volatile unsigned int*>(f.epoch) + 1u;
        if (DRAFT && (int)blockIdx.x < f.B && f.clf_H > 0) {
            // this CTA will finish at least one sequence: stage the classifier while the first tile loads
            const int Hc = f.clf_H, t = ew * 32 + lane, nt = kUmmaEpiWarps * 32;
            for (int i = t; i < Hc * kNFeat; i += nt) clf_s[i] = f.clf_W1[i];
            for (int i = t; i < Hc; i += nt) {
                clf_s[Hc * kNFeat + i] = f.clf_b1[i];
                clf_s[Hc * (kNFeat + 1) + i] = f.clf_w2[i];
            }
            if (t == 0) clf_s[Hc * (kNFeat + 2)] = f.clf_b2[0];
        }

        float best_v = DISCO_NEG_INF;
        int best_i = kNoIndex;
        SoftmaxState st;
        st.init();
        RegTop10 top;
        top.init();
        // this lane's candidate queue (draft step): entry i at queue[32 i]
        float* queue = reinterpret_cast<float*>(smem + kUmmaRingBytes - kUmmaQueueBytes) + ew * (kUmmaQueueEntries * 32) + lane;

        int it = 0;
        for (int i = 0; i < gTPC; ++i) {
            const int v0 = (nslot * gTPC + i) * gTR;
            if (v0 >= p.V) break;
            const int buf = it & 1;
            mbar_wait(&tmem_full[buf], (it >> 1) & 1, p.status);
            tc_fence_after();
            const int ncols = min(gTR, p.V - v0);  // further columns belong to the next tile or lie past V
            if (warp_has_rows) {
                const int nchunks = (ncols + 31) >> 5;
                const int c_lo = (nchunks * share + nshare - 1) / nshare;
                const int c_hi = (nchunks * (share + 1) + nshare - 1) / nshare;
                for (int c = c_lo; c < c_hi; ++c) {
                    float z[32];
                    tmem_ld32(tmem_base + buf * 256 + c * 32 + (static_cast<uint32_t>(quad * 32) << 16), z);
                    const int cbase = c * 32;
                    if (DRAFT) {
                        const bool whole = cbase + 32 <= ncols;   // (warp-uniform) no column of the chunk is masked
                        float cmax = DISCO_NEG_INF;
                        if (whole) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                z[j] = __fadd_rn(z[j], 0.f);
                                cmax = fmaxf(cmax, z[j]);
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                z[j] = (cbase + j < ncols) ? __fadd_rn(z[j], 0.f) : DISCO_NEG_INF;
                                cmax = fmaxf(cmax, z[j]);
                            }
                        }
                        if (cmax > st.m) {  // move the reference maximum first, then add the chunk
                            if (st.Z > 0.f) {
                                const float dm = st.m - cmax;
                                const float e = __expf(dm);
                                st.S = e * (st.S + dm * st.Z);
                                st.Z *= e;
                            }
                            st.m = cmax;
                        }
                        if (whole) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                const float t = z[j] - st.m;
                                const float e = __expf(t);
                                st.Z += e;
                                st.S = fmaf(e, t, st.S);
                                if (z[j] > best_v) {
                                    best_v = z[j];
                                    best_i = v0 + cbase + j;
                                }
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                const float t = z[j] - st.m;       // -inf for masked columns: e = 0
                                const float e = __expf(t);
                                st.Z += e;
                                st.S = (cbase + j < ncols) ? fmaf(e, t, st.S) : st.S;
                                if (z[j] > best_v) {
                                    best_v = z[j];
                                    best_i = v0 + cbase + j;
                                }
                            }
                        }
                        if (!STATS) {
                            // The ten largest per row.  A logit enters a row's list with probability about
                            // 10 / (columns seen so far), but in a warp of 32 rows some lane nearly always needs the
                            // insertion network, so running it per logit costs 32 rows' worth for one row's need.
                            // Instead each lane queues the logits above its row's 10th largest (its own slots of
                            // shared memory, 16 logits at a time), and the network then runs as often as the
                            // longest queue of the warp is deep: two or three times per 16 logits, not eight.
#pragma unroll
                            for (int h = 0; h < 32; h += kUmmaQueueEntries) {
                                const float thr = top.t[kTopK - 1];
                                float* qp = queue;
#pragma unroll
                                for (int j = 0; j < kUmmaQueueEntries; ++j) {
                                    if (z[h + j] > thr) {
                                        *qp = z[h + j];
                                        qp += 32;
                                    }
                                }
                                const int cnt = static_cast<int>(qp - queue) >> 5;
                                const int deepest = __reduce_max_sync(kFullMask, cnt);
                                for (int i = 0; i < deepest; i += 2) {
                                    const float a = i < cnt ? queue[i * 32] : DISCO_NEG_INF;
                                    const float b = i + 1 < cnt ? queue[(i + 1) * 32] : DISCO_NEG_INF;
                                    top.push2(a, b);
                                }
                            }
                        }
                        if (keep_logits) {
                            float* dst = p.probs + (size_t)row * p.V + v0 + cbase;
                            if ((((uintptr_t)p.probs & 15) | ((p.V | (v0 + cbase)) & 3)) == 0 && cbase + 32 <= ncols) {  // 16-byte stores
#pragma unroll
                                for (int j = 0; j < 32; j += 4)
                                    *reinterpret_cast<float4*>(dst + j) = make_float4(z[j], z[j + 1], z[j + 2], z[j + 3]);
                            } else {
#pragma unroll
                                for (int j = 0; j < 32; ++j)
                                    if (cbase + j < ncols) dst[j] = z[j];
                            }
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const float zz = __fadd_rn(z[j], 0.f);
                            if (cbase + j < ncols && zz > best_v) {
                                best_v = zz;
                                best_i = v0 + cbase + j;
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tmem_empty[buf]);
            ++it;
        }

        // one result per hidden row and CTA
        if (DRAFT) {
            // the warps that hold the same rows hand their state to the one with share 0
            unsigned long long key = best_i != kNoIndex ? argmax_key(best_v, best_i) : 0ull;
            if (share != 0) {
                float4* mine = xch + ((share - 1) * p.rows_pad + tile_row) * 4;
                mine[0] = make_float4(st.m, st.Z, st.S, 0.f);
                mine[1] = make_float4(top.t[0], top.t[1], top.t[2], top.t[3]);
                mine[2] = make_float4(top.t[4], top.t[5], top.t[6], top.t[7]);
                mine[3] = make_float4(top.t[8], top.t[9], __uint_as_float((uint32_t)(key & 0xffffffffull)),
                                      __uint_as_float((uint32_t)(key >> 32)));
            }
            named_barrier_sync(2, kUmmaEpiWarps * 32);
            if (share == 0 && valid) {
                for (int o = 0; o < nshare - 1; ++o) {
                    const float4* theirs = xch + (o * p.rows_pad + tile_row) * 4;
                    const float4 q = theirs[0], a = theirs[1], bq = theirs[2], cq = theirs[3];
                    st.merge(q.x, q.y, q.z);   // a share without columns has Z = 0 and changes nothing
                    const unsigned long long k2 =
                        (static_cast<unsigned long long>(__float_as_uint(cq.w)) << 32) | __float_as_uint(cq.z);
                    key = k2 > key ? k2 : key;
                    const float lv[kTopK] = {a.x, a.y, a.z, a.w, bq.x, bq.y, bq.z, bq.w, cq.x, cq.y};
                    top.merge(lv);
                }
                store_stamped_record(p.part_rec + ((size_t)row * p.CN + nslot) * kStampedPieces, st.m, st.Z, st.S, top.t,
                                     key, stamp);
            }
            // Second phase inside the same (cooperative) launch: a CTA reads the records of its sequences
            // as the other CTAs publish them (stamped records, bounded waits).  Up to two sequences per CTA
            // are finished by groups of warps (all eight for one sequence, four each for two); beyond that,
            // and for statistics-only rows, the sequences are shared out one warp each.
            named_barrier_sync(2, kUmmaEpiWarps * 32);  // the exchange area is free from here on
            const int grid = (int)gridDim.x;
            if (!STATS && f.B <= 2 * grid) {
                const bool two = f.B > grid;
                const int g = two ? ew >> 2 : 0;
                const int gt = two ? (ew & 3) * 32 + lane : ew * 32 + lane;
                const int b = (int)blockIdx.x + g * grid;
                if (b < f.B) {
                    float* group_s = reinterpret_cast<float*>(xch) + g * kGroupScratchWords;
                    const float4* recs = p.part_rec + (size_t)b * p.CN * kStampedPieces;
                    const uint32_t want = stamp + f.test_stamp_skew;
                    // a masked sequence still waits for its records: the stamp may only advance once every
                    // CTA has taken part in this launch
                    const MergedPartials mp = two ? group_merge_partials<4>(recs, p.CN, want, p.status, group_s, 3 + g, gt)
                                                  : group_merge_partials<8>(recs, p.CN, want, p.status, group_s, 3, gt);
                    if (gt < 32) {
                        const bool chain = f.chain.alive != nullptr;
                        if (chain_seq_live(f.chain, f.active, b)) {
                            const float fpos = chain ? static_cast<float>(f.chain.pos0[b] + f.chain.step)
                                                     : (f.pos ? static_cast<float>(f.pos[b]) : 0.f);
                            const int nd = chain ? f.chain.step : (f.n_drafted ? f.n_drafted[b] : 0);
                            const int Hc = f.clf_H;
                            const DraftOutputs o{f.token, f.conf, f.halt, f.feats, f.final_stats, f.nll_sum,
                                                 f.stats_only, f.chain};
                            warp_draft_epilogue(mp.st, mp.key, mp.sel, fpos, nd, f.tau, f.sl_max, group_s, clf_s,
                                                clf_s + Hc * kNFeat, clf_s + Hc * (kNFeat + 1), clf_s + Hc * (kNFeat + 2),
                                                Hc, b, o, lane);
                        }
                        // the last finished sequence of the grid advances the stamp for the next launch: by
                        // then every record of this launch has been read
                        __syncwarp();
                        if (lane == 0 && atomicAdd(f.epoch + 1, 1u) == (unsigned int)f.B - 1u) {
                            f.epoch[1] = 0u;
                            f.epoch[0] = stamp == 0xffffffffu ? 0u : stamp;   // the stamp is never zero
                        }
                    }
                }
            } else {
                const int first = ew * (int)gridDim.x + (int)blockIdx.x;
                if (first < f.B) {
                    int b = first;
                    const bool chain = f.chain.alive != nullptr;
                    bool act = chain_seq_live(f.chain, f.active, b);
                    float fpos = chain ? static_cast<float>(f.chain.pos0[b] + f.chain.step)
                                       : (f.pos ? static_cast<float>(f.pos[b]) : 0.f);
                    int nd = chain ? f.chain.step : (f.n_drafted ? f.n_drafted[b] : 0);
                    float* feat16 = reinterpret_cast<float*>(xch) + ew * kWarpScratchWords;  // the exchange area is free again
                    for (;;) {
                        // a masked sequence still waits for its records: the stamp may only advance once
                        // every CTA has taken part in this launch
                        umma_finish_sequence(f, p.part_rec, p.CN, b, act, fpos, nd, feat16, clf_s, stamp + f.test_stamp_skew,
                                             p.status, lane);
                        b += kUmmaEpiWarps * (int)gridDim.x;
                        if (b >= f.B) break;
                        act = chain_seq_live(f.chain, f.active, b);
                        fpos = chain ? static_cast<float>(f.chain.pos0[b] + f.chain.step)
                                     : (f.pos ? static_cast<float>(f.pos[b]) : 0.f);
                        nd = chain ? f.chain.step : (f.n_drafted ? f.n_drafted[b] : 0);
                    }
                    // the last finishing warp of the grid advances the stamp for the next launch: by then every
                    // record of this launch has been read
                    const unsigned int nwarps = (unsigned int)min(f.B, kUmmaEpiWarps * (int)gridDim.x);
                    __syncwarp();
                    if (lane == 0 && atomicAdd(f.epoch + 1, 1u) == nwarps - 1) {
                        f.epoch[1] = 0u;
                        f.epoch[0] = stamp == 0xffffffffu ? 0u : stamp;   // the stamp is never zero
                    }
                }
            }
        } else {
            if (valid && best_i != kNoIndex) atomicMax(p.keys + row, argmax_key(best_v, best_i));
            if (p.fuse_final) {
                // ticket: the last CTA to get here matches the prefixes and clears the keys
                __shared__ int s_last;
                __threadfence();
                named_barrier_sync(2, kUmmaEpiWarps * 32);
                if (ew == 0 && lane == 0) s_last = atomicAdd(p.ticket, 1u) == (unsigned)(gMT * gCN) - 1u;   // idle CTAs take none
                named_barrier_sync(2, kUmmaEpiWarps * 32);
                if (s_last) {
                    __threadfence();
                    for (int b = ew; b < p.B; b += kUmmaEpiWarps)
                        verify_one_sequence(p.keys, p.draft_ids, p.row_off, p.B, p.SL, gR, b, p.n_accept, p.bonus,
                                            p.target_ids, p.status, lane, p.padded);
                    if (ew == 0) warp_write_row_offsets(p.padded, p.B, p.SL, lane);
                    named_barrier_sync(2, kUmmaEpiWarps * 32);
                    for (int r = ew * 32 + lane; r < p.R; r += kUmmaEpiWarps * 32) p.keys[r] = 0ull;
                    if (ew == 0 && lane == 0) *p.ticket = 0u;
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ---------------------------------------------------------------------------------------------
// finishing kernels
// ---------------------------------------------------------------------------------------------

// Verification: one warp per sequence decodes the arg-max keys, matches the prefix and picks the
// bonus token.  The last CTA to finish clears the keys for the next call.
struct VerifyFinalParams {
    unsigned long long* keys;
    const int32_t* draft_ids;
    const int32_t* row_off;
    int B, SL, R;
    int32_t* n_accept;
    int32_t* bonus;
    int32_t* target_ids;
    int* status;
    unsigned int* ticket;
    VerifyPadded padded;
    const int32_t* dev_R;   // non-null: the row count is device memory (R is then the upper bound)
};

__global__ void __launch_bounds__(128) verify_finalize_kernel(const VerifyFinalParams p) {
    __shared__ int s_last;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.x * (blockDim.x >> 5) + warp;
    const int R = p.dev_R ? min(max(__ldcg(p.dev_R), 1), p.R) : p.R;
    if (b < p.B)
        verify_one_sequence(p.keys, p.draft_ids, p.row_off, p.B, p.SL, R, b, p.n_accept, p.bonus, p.target_ids,
                            p.status, lane, p.padded);
    if (blockIdx.x == gridDim.x - 1 && warp == (blockDim.x >> 5) - 1) warp_write_row_offsets(p.padded, p.B, p.SL, lane);
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        s_last = atomicAdd(p.ticket, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    for (int r = threadIdx.x; r < p.R; r += blockDim.x) p.keys[r] = 0ull;  // every reader is done
    if (threadIdx.x == 0) *p.ticket = 0u;
}

}  // namespace disco
