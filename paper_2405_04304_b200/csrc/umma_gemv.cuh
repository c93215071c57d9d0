// Tensor-core draft step for a handful of sequences (1..16 hidden rows): the GEMV-shaped case.
//
// Here the LM head is the 128-row operand of tcgen05.mma and the hidden rows are the narrow one:
//
//   D[v, r] = sum_k W[v, k] * H[r, k]       v (128 vocabulary rows of a tile) on the TMEM lanes,
//                                           r (hidden rows, padded to N = 16) on the TMEM columns
//
// so after tcgen05.ld every lane of an epilogue warp holds the logit of "its" vocabulary row: one
// logit per lane, exactly the block that warp_fold_block folds into soft-max statistics, top-10 and
// arg-max in parallel.  The dot products cost the SM a few hundred instructions instead of the
// ~14 k of the CUDA-core kernel, so what is left is HBM streaming plus the fixed reduction tail.
//
//   * one CTA per SM and slab of ceil(V / #SM) vocabulary rows, cut into tiles of 128 rows (the last
//     one shorter: its own TMA box, so nothing beyond the slab is fetched);
//   * warp 0 producer (TMA, 128-byte swizzle, ring of 16 KB stages for the LM head; the hidden rows are
//     loaded once, after the dependency wait, and stay), warp 1 MMA issuer (M = 128, N = 16, K = 16, two
//     16-column TMEM buffers), warps 2-5 epilogue (one TMEM lane quadrant each);
//   * the ring is as deep as shared memory allows (12 stages = one whole tile of the 768-wide heads) and
//     is filled before the dependency wait, so that after the wait the first tile needs nothing but the
//     hidden rows;
//   * MMAs into one accumulator form a dependent chain (about 130 cycles each, measured), and a tile of a
//     768-wide head would be 48 of them: the four K = 16 steps of a k-block go to four accumulators
//     instead (16 TMEM columns each), which the epilogue adds up;
//   * per-CTA records, ticket, last-CTA reduction and classifier exactly as in the streaming kernel.
#pragma once

#include "umma_tail.cuh"

namespace disco {

constexpr int kGemvEpiWarps = 4;
constexpr int kGemvThreads = (2 + kGemvEpiWarps) * 32;
constexpr int kGemvMaxRows = 16;
constexpr int kGemvATile = 128 * 128;   // 128 vocabulary rows x 128 B
constexpr int kGemvMaxStages = 16;
constexpr int kGemvAcc = kUmmaBK / 16;          // independent accumulators per TMEM buffer (4)
constexpr int kGemvBufCols = kGemvAcc * 16;     // TMEM columns per buffer

struct GemvParams {
    TailParams t;     // V, d, R and everything the fused epilogue needs (scratch, classifier, outputs)
    int TR;           // vocabulary rows per CTA
    int tiles;        // ceil(TR / 128)
    int tail_rows;    // rows of the last tile's TMA box (multiple of 8)
    int h_rows;       // rows of the hidden-state box (8 or 16)
    int stages;       // ring depth (2 .. kGemvMaxStages)
};

// Shared memory besides the ring: the resident hidden rows (one k-block of h_rows x 128 B per 64 hidden
// units; the MMA reads 16 rows from each, the surplus lands in columns nobody reads), barriers, records,
// second-phase scratch, classifier.
inline size_t gemv_fixed_smem_bytes(int RK, int clf_H, int d, int h_rows) {
    size_t b = 1024;                                             // alignment
    b += (size_t)((d + kUmmaBK - 1) / kUmmaBK) * h_rows * 128 + 1024;  // hidden rows (+ the 16-row overhang)
    b += 512;                                                    // barriers, TMEM address
    b += (size_t)(kGemvEpiWarps * RK + 1) * kRecordWords * 4;    // warp records / finalize staging
    b += kGemvEpiWarps * kWarpScratchWords * 4;                  // second-phase scratch per warp
    b += ((size_t)clf_H * (kNFeat + 2) + 4) * 4;                 // classifier parameters
    return b + 128;
}
inline size_t gemv_smem_bytes(int RK, int clf_H, int d, int h_rows, int stages) {
    return gemv_fixed_smem_bytes(RK, clf_H, d, h_rows) + (size_t)stages * kGemvATile;
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// RK: compile-time bound on the hidden rows (1, 2, 4, 8 or 16)
template <int RK>
__global__ void __launch_bounds__(kGemvThreads, 1)
umma_gemv_draft_kernel(const __grid_constant__ CUtensorMap tmap_W, const __grid_constant__ CUtensorMap tmap_Wtail,
                       const __grid_constant__ CUtensorMap tmap_H, const GemvParams g) {
    extern __shared__ uint8_t smem_dyn[];
    const TailParams& p = g.t;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
    const int KBs = (p.d + kUmmaBK - 1) / kUmmaBK;
    const int b_stride = g.h_rows * 128;   // bytes between the k-blocks of the resident hidden rows
    uint8_t* a_tiles = smem;
    uint8_t* b_tiles = smem + g.stages * kGemvATile;
    uint8_t* after_b = b_tiles + KBs * b_stride + 1024;
    uint64_t* full = reinterpret_cast<uint64_t*>(after_b);
    uint64_t* empty = full + kGemvMaxStages;
    uint64_t* tmem_full = empty + kGemvMaxStages;
    uint64_t* tmem_empty = tmem_full + 2;
    uint64_t* h_full = tmem_empty + 2;
    uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(h_full + 1);
    float* wstate = reinterpret_cast<float*>(after_b + 512);
    float* feat_s = wstate + (kGemvEpiWarps * RK + 1) * kRecordWords;
    float* clf_s = feat_s + kGemvEpiWarps * kWarpScratchWords;
    __shared__ int s_is_last;

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int grid = gridDim.x;
    const int KB = (p.d + kUmmaBK - 1) / kUmmaBK;
    const int v_begin = blockIdx.x * g.TR;
    const int v_end = min(p.V, v_begin + g.TR);
    const int tiles = v_begin < p.V ? g.tiles : 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < g.stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        mbar_init(h_full, 1);
        for (int b = 0; b < 2; ++b) {
            mbar_init(&tmem_full[b], 1);
            mbar_init(&tmem_empty[b], kGemvEpiWarps);
        }
        fence_mbar_init();
        prefetch_tensormap(&tmap_W);
        prefetch_tensormap(&tmap_Wtail);
        prefetch_tensormap(&tmap_H);
    }
    if (warp == 1) {
        tmem_alloc(tmem_base_s, 2 * kGemvBufCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_base_s;

    if (warp == 0) {
        // ------------------------------ producer ------------------------------
        if (lane == 0) {
            const int total = tiles * KB;
            // the LM head does not depend on the preceding kernel: the whole ring is requested at once
            const int pre = min(g.stages, total);
            for (int n = 0; n < pre; ++n) {
                const int tile = n / KB, kb = n - tile * KB;
                const bool last = tile == g.tiles - 1;
                mbar_arrive_expect_tx(&full[n], (uint32_t)(last ? g.tail_rows : 128) * 128u);
                tma_load_2d(a_tiles + n * kGemvATile, last ? &tmap_Wtail : &tmap_W, kb * kUmmaBK, v_begin + tile * 128,
                            &full[n]);
            }
            asm volatile("griddepcontrol.wait;" ::: "memory");
            // the hidden rows, all k-blocks on one barrier; they stay for the whole kernel
            if (total > 0) {
                mbar_arrive_expect_tx(h_full, (uint32_t)(KB * b_stride));
                for (int kb = 0; kb < KB; ++kb) tma_load_2d(b_tiles + kb * b_stride, &tmap_H, kb * kUmmaBK, 0, h_full);
            }
            int stage = pre == g.stages ? 0 : pre, phase = pre == g.stages ? 1 : 0;
            for (int n = pre; n < total; ++n) {
                const int tile = n / KB, kb = n - tile * KB;
                const bool last = tile == g.tiles - 1;
                mbar_wait(&empty[stage], phase ^ 1, p.status);
                mbar_arrive_expect_tx(&full[stage], (uint32_t)(last ? g.tail_rows : 128) * 128u);
                tma_load_2d(a_tiles + stage * kGemvATile, last ? &tmap_Wtail : &tmap_W, kb * kUmmaBK,
                            v_begin + tile * 128, &full[stage]);
                if (++stage == g.stages) {
                    stage = 0;
                    phase ^= 1;
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            int stage = 0, phase = 0;
            const uint32_t idesc = umma_idesc(16);
            if (tiles > 0) {
                mbar_wait(h_full, 0, p.status);
                tc_fence_after();
            }
            for (int tile = 0; tile < tiles; ++tile) {
                const int buf = tile & 1;
                mbar_wait(&tmem_empty[buf], ((tile >> 1) & 1) ^ 1, p.status);
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * kGemvBufCols;
                for (int kb = 0; kb < KB; ++kb) {
                    mbar_wait(&full[stage], phase, p.status);
                    tc_fence_after();
                    const uint64_t a_desc = umma_smem_desc(a_tiles + stage * kGemvATile);
                    const uint64_t b_desc = umma_smem_desc(b_tiles + kb * b_stride);
#pragma unroll
                    for (int k = 0; k < kGemvAcc; ++k)  // step k of every k-block accumulates into accumulator k
                        tc_mma_bf16(d_tmem + k * 16, a_desc + 2 * k, b_desc + 2 * k, idesc, kb != 0);
                    tc_commit(&empty[stage]);
                    if (++stage == g.stages) {
                        stage = 0;
                        phase ^= 1;
                    }
                }
                tc_commit(&tmem_full[buf]);
            }
        }
    } else {
        // ------------------------------ epilogue ------------------------------
        constexpr int BAR_THREADS = kGemvEpiWarps * 32;
        const int ew = warp - 2;    // 0..3: role in the reductions
        const int quad = warp & 3;  // TMEM lane quadrant this warp may read
        const int tid = ew * 32 + lane;
        if (p.clf_H > 0) {  // classifier parameters -> shared, asynchronously; only the last CTA reads them
            const int Hc = p.clf_H;
            const int n1 = Hc * kNFeat;
            for (int i = tid; i < n1 + 2 * Hc + 1; i += BAR_THREADS) {
                const float* src = i < n1 ? p.clf_W1 + i
                                          : (i < n1 + Hc ? p.clf_b1 + (i - n1)
                                                         : (i < n1 + 2 * Hc ? p.clf_w2 + (i - n1 - Hc) : p.clf_b2));
                cp_async4(clf_s + i, src);
            }
            cp_async_commit();
        }
        asm volatile("griddepcontrol.wait;" ::: "memory");  // scratch and outputs belong to the predecessor until now

        SoftmaxState st[RK];
        float top_v[RK], best_v[RK];
        int best_i[RK];
#pragma unroll
        for (int r = 0; r < RK; ++r) {
            st[r].init();
            top_v[r] = DISCO_NEG_INF;
            best_v[r] = DISCO_NEG_INF;
            best_i[r] = kNoIndex;
        }
        float* fold_scratch = wstate + (ew * RK) * kRecordWords + 4;

        for (int tile = 0; tile < tiles; ++tile) {
            const int buf = tile & 1;
            mbar_wait(&tmem_full[buf], (tile >> 1) & 1, p.status);
            tc_fence_after();
            const int v_lane0 = v_begin + tile * 128 + quad * 32;  // vocabulary row of lane 0 of this warp
            const int n = max(0, min(32, v_end - v_lane0));        // rows of the slab in this warp's quadrant
            float z[16];
            tmem_ld16(tmem_base + buf * kGemvBufCols + (static_cast<uint32_t>(quad * 32) << 16), z);
#pragma unroll
            for (int a = 1; a < kGemvAcc; ++a) {
                float za[16];
                tmem_ld16(tmem_base + buf * kGemvBufCols + a * 16 + (static_cast<uint32_t>(quad * 32) << 16), za);
#pragma unroll
                for (int r = 0; r < 16; ++r) z[r] += za[r];
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tmem_empty[buf]);  // the values are in registers: the buffer is free
            if (n > 0) {
                const int idx = v_lane0 + lane;
#pragma unroll
                for (int r = 0; r < RK; ++r) {
                    if (r < p.R) {
                        const float val = lane < n ? __fadd_rn(z[r], 0.f) : DISCO_NEG_INF;
                        if (p.probs && lane < n) p.probs[(size_t)r * p.V + idx] = val;
                        warp_fold_block(val, idx, n, lane, st[r], best_v[r], best_i[r], top_v[r],
                                        fold_scratch + r * kRecordWords);
                    }
                }
            }
        }

        // ---- merge the four warps of this CTA, publish the CTA's record for each hidden row ----
#pragma unroll
        for (int r = 0; r < RK; ++r) {
            const unsigned long long key = best_i[r] != kNoIndex ? argmax_key(best_v[r], best_i[r]) : 0ull;
            warp_store_record(wstate + (ew * RK + r) * kRecordWords, st[r], key, top_v[r], lane);
        }
        named_barrier_sync(1, BAR_THREADS);
        for (int r = ew; r < p.R; r += kGemvEpiWarps) {
            LaneRecord rec;
            rec.clear();
            if (lane < kGemvEpiWarps) {
                const float4* sr = reinterpret_cast<const float4*>(wstate + (lane * RK + r) * kRecordWords);
                rec.set(sr[0], sr[1], sr[2], sr[3]);
            }
            warp_reduce_records(rec, 2);
            warp_store_record(reinterpret_cast<float*>(p.part_rec + ((size_t)r * grid + blockIdx.x) * 4), rec, lane);
        }

        // ---- ticket: the last CTA reduces the records of all CTAs and runs the fused epilogue ----
        __threadfence();
        named_barrier_sync(1, BAR_THREADS);
        if (tid == 0) s_is_last = atomicAdd(p.ticket, 1u) == (unsigned)grid - 1u;
        named_barrier_sync(1, BAR_THREADS);
        cp_async_wait_all();
        if (s_is_last) {
            __threadfence();
            named_barrier_sync(1, BAR_THREADS);
            for (int b = ew; b < p.R; b += kGemvEpiWarps) {
                if (p.active && !p.active[b]) continue;
                finalize_draft_seq(p, b, grid, feat_s + ew * kWarpScratchWords, clf_s, lane);
            }
            if (tid == 0) *p.ticket = 0u;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 2 * kGemvBufCols);
    }
}

}  // namespace disco
