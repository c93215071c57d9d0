// Tensor-core draft step for a handful of sequences (1..16 hidden rows): the GEMV-shaped case.
//
//   D[r, v] = sum_k H[r, k] * W[v, k]       r (hidden rows) on the TMEM lanes 0 .. R-1,
//                                           v (up to 256 vocabulary rows of a tile) on the TMEM columns
//
// One tcgen05.mma costs about 128 cycles whatever its N (measured: the same for N = 16 and N = 224), so
// the vocabulary has to be the wide operand: a CTA's whole slab of ceil(V / #SM) rows is one or two MMAs
// wide, 4 * d / 64 MMAs deep, a few microseconds that hide under the HBM stream.  (With the vocabulary on
// the lanes and N = 16 the MMAs alone took as long as HBM needs for the slab.)
//
//   * one CTA per SM and slab; the slab is cut into tiles of up to 256 rows (one for the 32000-row
//     head, two for the 49152-row one);
//   * the hidden rows are the A operand: loaded once after the dependency wait, one 8- or 16-row box per
//     k-block, and they stay.  The MMA reads 128 rows from each box's start: what lies behind (further
//     boxes, the ring) only feeds accumulator lanes nobody reads;
//   * warp 0 producer (TMA, 128-byte swizzle; ring of LM-head stages as deep as shared memory allows,
//     filled before the dependency wait), warp 1 MMA issuer (M = 128, N = tile rows, K = 16, two
//     256-column TMEM buffers), warps 2-9 epilogue;
//   * epilogue: all hidden rows sit in TMEM lane quadrant 0, which two of the eight warps may read: they
//     copy the tile's logits to shared memory (row r by lane r), then all eight warps fold them 32 at a time, one
//     logit per lane (soft-max statistics, top-10 and arg-max in parallel, warp_fold_block);
//   * per-CTA records, ticket, last-CTA second phase and classifier exactly as in the streaming kernel.
#pragma once

#include "umma_tail.cuh"

namespace disco {

constexpr int kGemvEpiWarps = 8;
constexpr int kGemvDumpWarps = kGemvEpiWarps / 4;   // epilogue warps that may read TMEM lane quadrant 0
constexpr int kGemvThreads = (2 + kGemvEpiWarps) * 32;
constexpr int kGemvMaxRows = 16;
constexpr int kGemvMaxStages = 16;
constexpr int kGemvRowStride = 256 + 4;   // floats per hidden row in the logit staging area (padded: no bank conflicts)

struct GemvParams {
    TailParams t;     // V, d, R and everything the fused epilogue needs (scratch, classifier, outputs)
    int TR;           // vocabulary rows per CTA (slab)
    int tiles;        // ceil(TR / 256)
    int TRt;          // vocabulary rows per tile
    int TRN;          // rows of the LM-head box = N of the MMA (TRt rounded up to 16, <= 256)
    int b_bytes;      // bytes of one ring stage (TRN * 128, a multiple of 1024)
    int h_rows;       // rows of the hidden-state box (8 or 16)
    int stages;       // ring depth (2 .. kGemvMaxStages)
};

// Shared memory besides the ring: the resident hidden rows, barriers, the logit staging area, records,
// second-phase scratch, classifier.
inline size_t gemv_fixed_smem_bytes(int RK, int clf_H, int d, int h_rows) {
    size_t b = 1024;                                             // alignment
    b += (size_t)((d + kUmmaBK - 1) / kUmmaBK) * h_rows * 128;   // hidden rows
    b += 512;                                                    // barriers, TMEM address
    b += (size_t)RK * kGemvRowStride * 4;                        // logits of one tile
    b += (size_t)(kGemvEpiWarps * RK + 1) * kRecordWords * 4;    // warp records / finalize staging
    b += kGemvEpiWarps * kWarpScratchWords * 4;                  // second-phase scratch per warp
    b += ((size_t)clf_H * (kNFeat + 2) + 4) * 4;                 // classifier parameters
    return b + 128;
}
inline size_t gemv_smem_bytes(int RK, int clf_H, int d, int h_rows, int stages, int b_bytes) {
    return gemv_fixed_smem_bytes(RK, clf_H, d, h_rows) + (size_t)stages * b_bytes;
}

// RK: compile-time bound on the hidden rows (1, 2, 4, 8 or 16)
template <int RK>
__global__ void __launch_bounds__(kGemvThreads, 1)
umma_gemv_draft_kernel(const __grid_constant__ CUtensorMap tmap_W, const __grid_constant__ CUtensorMap tmap_H,
                       const GemvParams g) {
    extern __shared__ uint8_t smem_dyn[];
    const TailParams& p = g.t;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
    const int KB = (p.d + kUmmaBK - 1) / kUmmaBK;
    const int h_stride = g.h_rows * 128;   // bytes between the k-blocks of the resident hidden rows
    uint8_t* h_tiles = smem;
    uint8_t* w_tiles = smem + KB * h_stride;          // 1024-aligned; at least 16 KB long (host check)
    uint8_t* after = w_tiles + g.stages * g.b_bytes;
    uint64_t* full = reinterpret_cast<uint64_t*>(after);
    uint64_t* empty = full + kGemvMaxStages;
    uint64_t* tmem_full = empty + kGemvMaxStages;
    uint64_t* tmem_empty = tmem_full + 2;
    uint64_t* h_full = tmem_empty + 2;
    uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(h_full + 1);
    float* lg_s = reinterpret_cast<float*>(after + 512);
    float* wstate = lg_s + RK * kGemvRowStride;
    float* feat_s = wstate + (kGemvEpiWarps * RK + 1) * kRecordWords;
    float* clf_s = feat_s + kGemvEpiWarps * kWarpScratchWords;
    __shared__ int s_is_last;

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int grid = gridDim.x;
    const int v_begin = blockIdx.x * g.TR;
    const int v_end = min(p.V, v_begin + g.TR);
    const int tiles = v_begin < p.V ? (v_end - v_begin + g.TRt - 1) / g.TRt : 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < g.stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&tmem_full[b], 1);
            mbar_init(&tmem_empty[b], kGemvDumpWarps);
        }
        mbar_init(h_full, 1);
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
    // A chained draft step (draft phase run on the device) in which no sequence drafts any more has nothing
    // to do: every warp finds that out by itself after the dependency wait (the flags are the predecessor's
    // output).  The LM-head stages requested before the wait are awaited, then the CTA leaves.
    const bool chained = p.chain.alive != nullptr && p.chain.step > 1;

    if (warp == 0) {
        // ------------------------------ producer ------------------------------
        const int total = tiles * KB;
        const uint32_t w_bytes = (uint32_t)g.TRN * 128u;
        const int pre = min(g.stages, total);
        if (lane == 0) {
            // the LM head does not depend on the preceding kernel: the whole ring is requested at once
            for (int n = 0; n < pre; ++n) {
                const int tile = n / KB, kb = n - tile * KB;
                mbar_arrive_expect_tx(&full[n], w_bytes);
                tma_load_2d(w_tiles + n * g.b_bytes, &tmap_W, kb * kUmmaBK, v_begin + tile * g.TRt, &full[n]);
            }
        }
        asm volatile("griddepcontrol.wait;" ::: "memory");
        const bool live = !chained || chain_any_live(p.chain, p.R, lane);
        if (lane == 0 && !live) {
            for (int n = 0; n < pre; ++n) mbar_wait(&full[n], 0, p.status);   // nothing may still be landing at exit
        } else if (lane == 0) {
            // the hidden rows, all k-blocks on one barrier; they stay for the whole kernel
            if (total > 0) {
                mbar_arrive_expect_tx(h_full, (uint32_t)(KB * h_stride));
                for (int kb = 0; kb < KB; ++kb) tma_load_2d(h_tiles + kb * h_stride, &tmap_H, kb * kUmmaBK, 0, h_full);
            }
            int stage = pre == g.stages ? 0 : pre, phase = pre == g.stages ? 1 : 0;
            for (int n = pre; n < total; ++n) {
                const int tile = n / KB, kb = n - tile * KB;
                mbar_wait(&empty[stage], phase ^ 1, p.status);
                mbar_arrive_expect_tx(&full[stage], w_bytes);
                tma_load_2d(w_tiles + stage * g.b_bytes, &tmap_W, kb * kUmmaBK, v_begin + tile * g.TRt, &full[stage]);
                if (++stage == g.stages) {
                    stage = 0;
                    phase ^= 1;
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        bool live = true;
        if (chained) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            live = chain_any_live(p.chain, p.R, lane);
        }
        if (lane == 0 && live) {
            int stage = 0, phase = 0;
            const uint32_t idesc = umma_idesc(g.TRN);
            if (tiles > 0) {
                mbar_wait(h_full, 0, p.status);
                tc_fence_after();
            }
            for (int tile = 0; tile < tiles; ++tile) {
                const int buf = tile & 1;
                mbar_wait(&tmem_empty[buf], ((tile >> 1) & 1) ^ 1, p.status);
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * 256;
                for (int kb = 0; kb < KB; ++kb) {
                    mbar_wait(&full[stage], phase, p.status);
                    tc_fence_after();
                    const uint64_t a_desc = umma_smem_desc(h_tiles + kb * h_stride);
                    const uint64_t b_desc = umma_smem_desc(w_tiles + stage * g.b_bytes);
#pragma unroll
                    for (int k = 0; k < kUmmaBK / 16; ++k)  // 16 k-elements = 32 bytes = 2 descriptor units
                        tc_mma_bf16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0);
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
        const int ew = warp - 2;    // 0..7: role in the reductions
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
        const bool live = !chained || chain_any_live(p.chain, p.R, lane);
        if (!live) cp_async_wait_all();
      if (live) {

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
        bool keep_logits[RK];   // rows whose logits go to the optional probs output (never a masked sequence's)
#pragma unroll
        for (int r = 0; r < RK; ++r) keep_logits[r] = p.probs && r < p.R && (!p.active || p.active[r]);

        for (int tile = 0; tile < tiles; ++tile) {
            const int buf = tile & 1;
            const int v0 = v_begin + tile * g.TRt;
            const int ncols = min(g.TRt, v_end - v0);   // further columns belong to the next tile or lie past the slab
            const int nblocks = (ncols + 31) >> 5;
            if (quad == 0) {
                // the one warp that may read lane quadrant 0: row r of the tile's logits goes to shared memory
                mbar_wait(&tmem_full[buf], (tile >> 1) & 1, p.status);
                tc_fence_after();
                for (int c = ew >> 2; c < nblocks; c += kGemvDumpWarps) {   // the quadrant-0 warps share the blocks
                    float z[32];
                    tmem_ld32(tmem_base + buf * 256 + c * 32, z);
                    if (lane < p.R) {
                        float4* dst = reinterpret_cast<float4*>(lg_s + lane * kGemvRowStride + c * 32);
#pragma unroll
                        for (int j = 0; j < 32; j += 4)
                            dst[j >> 2] = make_float4(__fadd_rn(z[j], 0.f), __fadd_rn(z[j + 1], 0.f),
                                                      __fadd_rn(z[j + 2], 0.f), __fadd_rn(z[j + 3], 0.f));
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&tmem_empty[buf]);  // the values are in shared memory: the buffer is free
            }
            named_barrier_sync(1, BAR_THREADS);
            // blocks of 32 logits, one per lane, dealt round-robin to the four warps
            for (int c = ew; c < nblocks; c += kGemvEpiWarps) {
                const int n = min(32, ncols - c * 32);
                const int idx = v0 + c * 32 + lane;
#pragma unroll
                for (int r = 0; r < RK; ++r) {
                    if (r < p.R) {
                        const float val = lane < n ? lg_s[r * kGemvRowStride + c * 32 + lane] : DISCO_NEG_INF;
                        if (keep_logits[r] && lane < n) p.probs[(size_t)r * p.V + idx] = val;
                        warp_fold_block(val, idx, n, lane, st[r], best_v[r], best_i[r], top_v[r],
                                        fold_scratch + r * kRecordWords);
                    }
                }
            }
            if (tile + 1 < tiles) named_barrier_sync(1, BAR_THREADS);  // the staging area is overwritten next
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
            warp_reduce_records(rec, ceil_log2(kGemvEpiWarps));
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
                if (!chain_seq_live(p.chain, p.active, b)) continue;
                finalize_draft_seq(p, b, grid, feat_s + ew * kWarpScratchWords, clf_s, lane);
            }
            if (tid == 0) *p.ticket = 0u;
        }
      }  // live
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace disco
