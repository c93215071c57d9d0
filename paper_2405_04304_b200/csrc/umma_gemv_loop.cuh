// The draft phase of an iteration as ONE persistent kernel, for a handful of sequences (1..4): up to
// sl_max draft steps (Sec. 3: after every draft token the classifier decides whether the next one is
// drafted) without leaving the GPU and without a launch per step.
//
// Each step is the tensor-core GEMV of umma_gemv.cuh (hidden rows on the TMEM lanes, the CTA's whole slab
// of the vocabulary on the columns); what the loop adds:
//   * one CTA per SM stays resident for all steps (cooperative launch: the steps hand over through global
//     memory, so every CTA must be running);
//   * the producer never stops: as soon as the MMAs of step i have released a ring stage it is refilled
//     with the LM head's tiles for step i + 1, while the CTA folds, publishes its record, and the step is
//     decided.  Only the hidden rows of step i + 1 are requested after step i has been decided -- in a
//     decoder they would not exist before;
//   * the A operand is the one 8-row box of hidden rows read 16 times over (zero stride between the 8-row
//     groups of the descriptor): every TMEM lane quadrant holds a copy of each row, so all eight epilogue
//     warps fetch logits, and the MMAs read nothing outside the box (with a non-zero stride they read ring
//     stages that the TMA unit is refilling, which halved their rate);
//   * the step's logits of a CTA (at most 256 per hidden row and tile) are folded by the whole CTA, one
//     logit per thread (cta_fold_tile), into one record per sequence, which is published in stamped
//     16-byte pieces: no fence and no counter between the writer and its reader;
//   * CTA 0 finishes the sequences with all eight epilogue warps (group_merge_partials polls the records
//     of the step until all carry its stamp), records which sequences go on, and publishes the decision
//     "continue / stop" in a stamped word that every CTA polls (bounded);
//   * tiles requested ahead for a step that does not take place are awaited before the CTA leaves.
// Every one of these phases is a chain of dependent instructions on a few warps, so the code is written for
// short chains (values through shared memory and independent comparisons instead of shuffle chains, loads
// of a batch in flight before the first use), not for few instructions.
#pragma once

#include "umma_gemv.cuh"

namespace disco {

constexpr int kLoopMaxSteps = 64;
constexpr unsigned kLoopContinue = 1u, kLoopStop = 2u;
// shared memory of the CTA-wide fold (two copies, used alternately): per-warp reduction slots, the candidates
// of the final ranking (at most the ten largest of each of the eight warps and the row's running ten), and
// the warps' values
constexpr int kFoldCandidates = kGemvEpiWarps * kTopK + kTopK;            // 90
constexpr int kFoldCandidatesPad = 96;                                    // whole batches of 32, the padding is -inf
constexpr int kFoldScratchWords = 64 + kFoldCandidatesPad + kGemvEpiWarps * 32;

struct GemvLoopParams {
    GemvParams g;          // geometry of one step; g.t: shapes, scratch, classifier, outputs of step 1, chain bookkeeping
    int steps;             // sl_max
    int w_rows_per_step;   // the LM head of step i starts (i - 1) * w_rows_per_step rows into the tensor map (0: one head)
    unsigned int* flags;   // [steps] decision of each step: (stamp << 2) | kLoopContinue / kLoopStop
    unsigned int* epoch;   // launches completed so far; the stamp of this launch is that + 1
    float4* records;       // [sequence][CTA] stamped records of 80 bytes; written by this kernel only, starts zeroed
};

__device__ __forceinline__ unsigned int ld_relaxed_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_u32(unsigned int* p, unsigned int v) {
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// The hidden rows of one step (rows row0 .. of the map), all k-blocks on one barrier; they stay for the step.
__device__ __forceinline__ void loop_issue_hidden(uint8_t* h_tiles, int h_stride, int KB, const CUtensorMap* tmap_H, int row0,
                                                  uint64_t* h_full) {
    mbar_arrive_expect_tx(h_full, (uint32_t)(KB * h_stride));
    for (int kb = 0; kb < KB; ++kb) tma_load_2d(h_tiles + kb * h_stride, tmap_H, kb * kUmmaBK, row0, h_full);
}

// A wait that is expected to last microseconds (the MMA issuer between two steps): sleep between the tests so
// that the warp does not compete for issue slots.  Bounded like mbar_wait.
__device__ __forceinline__ bool mbar_wait_idle(uint64_t* bar, uint32_t parity, int* status) {
    const long long t0 = clock64();
    for (int polls = 0;; ++polls) {
        if (mbar_try_wait(bar, parity)) return true;
        __nanosleep(64);
        if ((polls & 255) == 255 && ((status && *reinterpret_cast<volatile int*>(status) == DISCO_ERR_TIMEOUT) ||
                                     clock64() - t0 > kWaitBudgetClocks)) {
            record_status(status, DISCO_ERR_TIMEOUT);
            return false;
        }
    }
}

// Running result of one hidden row over the tiles of a step, in shared memory (16 words):
// m, Z, S, -, the ten largest logits, the arg-max key.
struct RowState {
    float m, Z, S, pad;
    float top[kTopK];
    uint32_t key_lo, key_hi;
};

// Fold the ncols <= 256 logits of one hidden row and tile (z[c], vocabulary index v0 + c) into the row's
// running state, by the eight epilogue warps, one logit per thread:
//   * maximum and arg-max key by warp reductions, then across the warps through shared memory;
//   * e^(z - M) and its first moment by one exponential per thread and shuffle sums;
//   * the ten largest by selection: every warp ranks its 32 logits against each other; the largest of the
//     warps' 10th-largest values (and the row's running 10th) bounds the new 10th from below, so only the
//     warps' top-ten values and the running values at or above it are candidates (a dozen or so, at most
//     90), and the candidates are ranked against each other.
// Two barriers.  sm: kFoldScratchWords words, not the copy the previous call used.  tid: 0 .. 255.
__device__ __forceinline__ void cta_fold_tile(const float* z, int ncols, int v0, RowState* rs, float* sm, int tid) {
    constexpr int BAR_THREADS = kGemvEpiWarps * 32;
    const int lane = tid & 31, w = tid >> 5;
    uint32_t* wred = reinterpret_cast<uint32_t*>(sm);      // [3][8] m bits, key lo, bits of the warp's 10th largest
    float* wsum = sm + 24;                                  // [2][8]
    int* ncand = reinterpret_cast<int*>(sm + 40);           // [1]
    float* cand = sm + 64;                                  // [kFoldCandidatesPad]
    float* wvals = cand + kFoldCandidatesPad;               // [8][32] the warps' values
    const bool valid = tid < ncols;
    const float val = valid ? z[tid] : DISCO_NEG_INF;
    const uint32_t bits = ordered_bits(val);
    const uint32_t mb = __reduce_max_sync(kFullMask, bits);
    // arg-max key of the warp: largest value, lowest index
    const uint32_t klo_mine = valid && bits == mb ? 0xffffffffu - static_cast<uint32_t>(v0 + tid) : 0u;
    const uint32_t klo = __reduce_max_sync(kFullMask, klo_mine);
    const int rank = rank_in_warp(val, lane, wvals + w * 32);
    if (rank == kTopK - 1) wred[16 + w] = bits;             // the warp's 10th largest (-inf with fewer than ten logits)
    if (lane == 0) {
        wred[w] = mb;
        wred[8 + w] = klo;      // 0: the warp holds no logit
    }
    if (tid == 0) *ncand = 0;
    if (tid < kFoldCandidatesPad) cand[tid] = DISCO_NEG_INF;
    named_barrier_sync(1, BAR_THREADS);
    uint32_t Mb = 0u, Klo = 0u, Tb = ordered_bits(rs->top[kTopK - 1]);
#pragma unroll
    for (int k = 0; k < kGemvEpiWarps; ++k) {
        Mb = max(Mb, wred[k]);
        Tb = max(Tb, wred[16 + k]);
    }
#pragma unroll
    for (int k = 0; k < kGemvEpiWarps; ++k) Klo = max(Klo, wred[k] == Mb ? wred[8 + k] : 0u);
    const float M = from_ordered_bits(Mb);
    const float theta = from_ordered_bits(Tb);
    float e = 0.f, et = 0.f;
    if (valid) {
        const float t = val - M;
        e = __expf(t);
        et = e * t;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        e += __shfl_xor_sync(kFullMask, e, off);
        et += __shfl_xor_sync(kFullMask, et, off);
    }
    if (lane == 0) {
        wsum[w] = e;
        wsum[8 + w] = et;
    }
    warp_append(valid && rank < kTopK && val >= theta, val, cand, ncand, kFoldCandidatesPad, lane);
    if (w == 0) {
        const float run = lane < kTopK ? rs->top[lane] : DISCO_NEG_INF;
        warp_append(run >= theta && run > DISCO_NEG_INF, run, cand, ncand, kFoldCandidatesPad, lane);
    }
    named_barrier_sync(1, BAR_THREADS);
    const int n = min(*ncand, kFoldCandidatesPad);   // at most 90 by construction
    if (tid < n) {
        const float x = cand[tid];
        const int r = rank_in_list(cand, n, x, tid);
        if (r < kTopK) rs->top[r] = x;               // entries beyond n were -inf before and stay so
    }
    if (tid == 0 && ncols > 0) {
        float Zt = 0.f, St = 0.f;
#pragma unroll
        for (int k = 0; k < kGemvEpiWarps; ++k) {
            Zt += wsum[k];
            St += wsum[8 + k];
        }
        SoftmaxState st;
        st.m = rs->m, st.Z = rs->Z, st.S = rs->S;
        st.merge(M, Zt, St);
        rs->m = st.m, rs->Z = st.Z, rs->S = st.S;
        // a later tile holds higher indices: it takes the arg-max only with a strictly larger value
        const unsigned long long k_tile = (static_cast<unsigned long long>(Mb) << 32) | Klo;
        const unsigned long long k_run = (static_cast<unsigned long long>(rs->key_hi) << 32) | rs->key_lo;
        if (k_tile > k_run) {
            rs->key_hi = Mb;
            rs->key_lo = Klo;
        }
    }
    // The caller puts a barrier between this call and any reader of the row state that is not one of the
    // threads that wrote it; the scratch copy is reused only by the call after the next.
}

// RK: compile-time bound on the sequences (1, 2 or 4); 8 / RK epilogue warps finish each sequence.
template <int RK>
__global__ void __launch_bounds__(kGemvThreads, 1)
umma_gemv_loop_kernel(const __grid_constant__ CUtensorMap tmap_W, const __grid_constant__ CUtensorMap tmap_H,
                      const GemvLoopParams lp) {
    extern __shared__ uint8_t smem_dyn[];
    const GemvParams& g = lp.g;
    const TailParams& p = g.t;
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
    const int KB = (p.d + kUmmaBK - 1) / kUmmaBK;
    const int h_stride = g.h_rows * 128;
    uint8_t* h_tiles = smem;
    uint8_t* w_tiles = smem + KB * h_stride;
    uint8_t* after = w_tiles + g.stages * g.b_bytes;
    uint64_t* full = reinterpret_cast<uint64_t*>(after);
    uint64_t* empty = full + kGemvMaxStages;
    uint64_t* tmem_full = empty + kGemvMaxStages;
    uint64_t* tmem_empty = tmem_full + 2;
    uint64_t* h_full = tmem_empty + 2;
    uint64_t* go_bar = h_full + 1;
    uint32_t* tmem_base_s = reinterpret_cast<uint32_t*>(go_bar + 1);
    uint32_t* s_code = tmem_base_s + 2;                       // [kLoopMaxSteps] decision of each step, as this CTA saw it
    float* lg_s = reinterpret_cast<float*>(after + 1024);     // [RK][kGemvRowStride] logits of one tile
    RowState* row_s = reinterpret_cast<RowState*>(lg_s + RK * kGemvRowStride);   // [RK]
    float* fold_s = reinterpret_cast<float*>(row_s + RK);     // 2 x kFoldScratchWords, used alternately
    float* group_s = fold_s + 2 * kFoldScratchWords;          // RK x kGroupScratchWords
    float* clf_s = group_s + RK * kGroupScratchWords;
    __shared__ int s_alive;
    __shared__ int s_pos0[4], s_forced[4], s_live[4];         // the finishing CTA's copy of the per-sequence inputs

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int grid = gridDim.x;
    const int B = p.R;
    const int v_begin = blockIdx.x * g.TR;
    const int v_end = min(p.V, v_begin + g.TR);
    const int tiles = v_begin < p.V ? (v_end - v_begin + g.TRt - 1) / g.TRt : 0;
    const int total = tiles * KB;          // LM-head stages of one step

    if (threadIdx.x == 0) {
        for (int s = 0; s < g.stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&tmem_full[b], 1);
            mbar_init(&tmem_empty[b], kGemvEpiWarps);
        }
        mbar_init(h_full, 1);
        mbar_init(go_bar, 1);
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

    if (warp == 0) {
        // ------------------------------ producer ------------------------------
        // One thread requests every LM-head stage of every step.  Its loop keeps running counters (no
        // divisions) and does nothing but test two barriers and issue copies; it sleeps when there is nothing to do.
        if (lane == 0 && total > 0) {
            const uint32_t w_bytes = (uint32_t)g.TRN * 128u;
            int w_step = 0, w_n = 0, w_tile = 0, w_kb = 0;     // the next stage to request: step, stage of the step, tile, k-block
            int w_row = v_begin;                                // first LM-head row of that step's slab in the tensor map
            int w_slot = 0, w_fill = 0;                         // its ring slot, and how often that slot has been filled before
            int ahead_slot = 0, ahead_fill = 0;                 // slot and fill count of the first stage of step w_step
            auto issue_w = [&]() {
                if (w_n == 0) {
                    ahead_slot = w_slot;
                    ahead_fill = w_fill;
                }
                mbar_arrive_expect_tx(&full[w_slot], w_bytes);
                tma_load_2d(w_tiles + w_slot * g.b_bytes, &tmap_W, w_kb * kUmmaBK, w_row + w_tile * g.TRt, &full[w_slot]);
                if (++w_kb == KB) {
                    w_kb = 0;
                    ++w_tile;
                }
                if (++w_n == total) {
                    w_n = 0;
                    w_tile = 0;
                    ++w_step;
                    w_row += lp.w_rows_per_step;
                }
                if (++w_slot == g.stages) {
                    w_slot = 0;
                    ++w_fill;
                }
            };
            // the LM head does not depend on the preceding kernel: the first step's stages are requested at once
            const int pre = min(g.stages, total);
            for (int n = 0; n < pre; ++n) issue_w();
            asm volatile("griddepcontrol.wait;" ::: "memory");
            loop_issue_hidden(h_tiles, h_stride, KB, &tmap_H, 0, h_full);
            int live = 1;                     // steps known to take place
            bool stopped = false;
            const long long t0 = clock64();
            int polls = 0;
            for (;;) {
                bool progress = false;
                // the decision of step `live` (its hidden rows were requested by the thread that read the decision)
                if (live < lp.steps && mbar_try_wait(go_bar, (live - 1) & 1)) {
                    if (s_code[live - 1] != kLoopContinue) {
                        stopped = true;
                        break;
                    }
                    ++live;
                    progress = true;
                }
                // the next LM-head stage: of a step known to take place, or of the one after it (requested ahead)
                if (w_step < lp.steps && w_step <= live) {
                    if (w_fill == 0 || mbar_try_wait(&empty[w_slot], (w_fill - 1) & 1)) {
                        issue_w();
                        progress = true;
                    }
                } else if (w_step >= lp.steps && live >= lp.steps) {
                    break;                    // everything requested, every step known to take place
                }
                if (!progress) __nanosleep(32);   // leave the issue slots to the warps that compute
                if (!progress && (++polls & 1023) == 0) {
                    if (*reinterpret_cast<volatile int*>(p.status) == DISCO_ERR_TIMEOUT ||
                        clock64() - t0 > kWaitBudgetClocks * (long long)lp.steps) {
                        record_status(p.status, DISCO_ERR_TIMEOUT);
                        stopped = true;
                        break;
                    }
                }
            }
            if (stopped) {
                // Stages requested ahead for the step that does not take place (the one after the `live` steps that
                // did: every stage of those has been consumed): its w_n first stages, or all of them if the next
                // stage to request already belongs to the step after it.  Nothing may still be landing at exit.
                const int n_ahead = w_step == live ? w_n : (w_step > live ? total : 0);
                int slot = ahead_slot, fill = ahead_fill;
                for (int n = 0; n < n_ahead; ++n) {
                    mbar_wait(&full[slot], fill & 1, p.status);
                    if (++slot == g.stages) {
                        slot = 0;
                        ++fill;
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0 && total > 0) {
            const uint32_t idesc = umma_idesc(g.TRN);
            int slot = 0, fill = 0, t_global = 0;
            for (int step0 = 0; step0 < lp.steps; ++step0) {
                if (step0 > 0) {
                    if (!mbar_wait_idle(go_bar, (step0 - 1) & 1, p.status)) break;
                    if (s_code[step0 - 1] != kLoopContinue) break;
                }
                if (!mbar_wait(h_full, step0 & 1, p.status)) break;
                tc_fence_after();
                for (int tile = 0; tile < tiles; ++tile, ++t_global) {
                    const int buf = t_global & 1;
                    mbar_wait(&tmem_empty[buf], ((t_global >> 1) & 1) ^ 1, p.status);
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + buf * 256;
                    for (int kb = 0; kb < KB; ++kb) {
                        mbar_wait(&full[slot], fill & 1, p.status);
                        tc_fence_after();
                        // The A operand is the one 8-row box of hidden rows, read 16 times over (zero stride between
                        // the 8-row groups): hidden row r lands on the TMEM lanes r, r + 8, .., r + 120, so every lane
                        // quadrant holds a copy and all epilogue warps can fetch logits; nothing outside the box is read.
                        const uint64_t a_desc = umma_smem_desc(h_tiles + kb * h_stride) & ~(0x3fffull << 32);
                        const uint64_t b_desc = umma_smem_desc(w_tiles + slot * g.b_bytes);
#pragma unroll
                        for (int k = 0; k < kUmmaBK / 16; ++k)
                            tc_mma_bf16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0);
                        tc_commit(&empty[slot]);
                        if (++slot == g.stages) {
                            slot = 0;
                            ++fill;
                        }
                    }
                    tc_commit(&tmem_full[buf]);
                }
            }
        }
    } else {
        // ------------------------------ epilogue ------------------------------
        constexpr int BAR_THREADS = kGemvEpiWarps * 32;
        constexpr int GW = kGemvEpiWarps / RK;      // warps that finish one sequence
        const int ew = warp - 2;
        const int quad = warp & 3;
        const int tid = ew * 32 + lane;
        if (p.clf_H > 0 && blockIdx.x == 0) {       // the finishing CTA stages the classifier
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
        asm volatile("griddepcontrol.wait;" ::: "memory");
        // stamp of this launch: read by every CTA before anything of this launch can advance the word
        const unsigned int launch_stamp = ld_relaxed_u32(lp.epoch) + 1u;
        if (blockIdx.x == 0 && tid < B) {
            s_pos0[tid] = p.chain.pos0[tid];
            s_forced[tid] = p.chain.sl_forced ? p.chain.sl_forced[tid] : 0x7fffffff;
            s_live[tid] = 1;
        }
        cp_async_wait_all();
        int t_global = 0, fold_calls = 0;
        int h_ahead_step = -1;     // (thread 0) step whose hidden rows were requested and not yet used

        for (int step0 = 0; step0 < lp.steps; ++step0) {
            // stamp of this step's records: unique among everything a reader can still find in the buffer
            const uint32_t rec_stamp = (launch_stamp << 6) | (uint32_t)(step0 & 63) | 0x80000000u;
            if (tid < RK) {
                RowState* rs = row_s + tid;
                rs->m = DISCO_NEG_INF, rs->Z = 0.f, rs->S = 0.f, rs->pad = 0.f;
#pragma unroll
                for (int k = 0; k < kTopK; ++k) rs->top[k] = DISCO_NEG_INF;
                rs->key_lo = 0u, rs->key_hi = 0u;
            }
            for (int tile = 0; tile < tiles; ++tile, ++t_global) {
                const int buf = t_global & 1;
                const int v0 = v_begin + tile * g.TRt;
                const int ncols = min(g.TRt, v_end - v0);
                const int nblocks = (ncols + 31) >> 5;
                {
                    // every warp fetches its share of the tile's columns from its own lane quadrant (lane r < 8 of a
                    // quadrant holds hidden row r) and stages them in shared memory, row by row
                    mbar_wait(&tmem_full[buf], (t_global >> 1) & 1, p.status);
                    tc_fence_after();
                    const uint32_t t_quad = tmem_base + buf * 256 + (static_cast<uint32_t>(quad * 32) << 16);
                    for (int c = ew; c < nblocks; c += kGemvEpiWarps) {
                        float z[32];
                        tmem_ld32(t_quad + c * 32, z);
                        if (lane < B) {
                            float4* dst = reinterpret_cast<float4*>(lg_s + lane * kGemvRowStride + c * 32);
#pragma unroll
                            for (int j = 0; j < 32; j += 4)
                                dst[j >> 2] = make_float4(__fadd_rn(z[j], 0.f), __fadd_rn(z[j + 1], 0.f),
                                                          __fadd_rn(z[j + 2], 0.f), __fadd_rn(z[j + 3], 0.f));
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&tmem_empty[buf]);
                }
                named_barrier_sync(1, BAR_THREADS);
                for (int r = 0; r < B; ++r, ++fold_calls)
                    cta_fold_tile(lg_s + r * kGemvRowStride, ncols, v0, row_s + r,
                                  fold_s + (fold_calls & 1) * kFoldScratchWords, tid);
                named_barrier_sync(1, BAR_THREADS);   // the staging area is overwritten by the next tile
            }
            if (tiles == 0) named_barrier_sync(1, BAR_THREADS);   // the cleared row states are visible
            // The MMAs of this step are done with the hidden rows: those of the next step are requested now, ahead
            // of the decision (if the phase stops here they are awaited before the CTA leaves).
            h_ahead_step = -1;
            if (tid == 0 && step0 + 1 < lp.steps && total > 0) {
                loop_issue_hidden(h_tiles, h_stride, KB, &tmap_H, (step0 + 1) * B, h_full);
                h_ahead_step = step0 + 1;
            }
            // ---- the CTA's record of this step for each sequence, in stamped pieces ----
            if (tid < B * kStampedPieces) {
                const int r = tid / kStampedPieces, piece = tid - r * kStampedPieces;
                const RowState* rs = row_s + r;
                float4* dst = lp.records + ((size_t)r * grid + blockIdx.x) * kStampedPieces + piece;
                const float sf = __uint_as_float(rec_stamp);
                float a, b2, c2;
                if (piece == 0) a = rs->m, b2 = rs->Z, c2 = rs->S;
                else if (piece < 4) a = rs->top[3 * piece - 3], b2 = rs->top[3 * piece - 2], c2 = rs->top[3 * piece - 1];
                else a = rs->top[9], b2 = __uint_as_float(rs->key_lo), c2 = __uint_as_float(rs->key_hi);
                store_relaxed_v4(dst, a, b2, c2, sf);
            }
            // ---- CTA 0 finishes the sequences and decides ----
            if (blockIdx.x == 0) {
                if (tid == 0) s_alive = 0;
                named_barrier_sync(1, BAR_THREADS);
                const int b = ew / GW;              // the sequence this warp helps to finish
                const int gt = (ew % GW) * 32 + lane;
                if (b < B) {
                    const bool takes_part = s_live[b] != 0;
                    if (takes_part) {               // uniform over the group
                        const MergedPartials mp =
                            group_merge_partials<GW>(lp.records + (size_t)b * grid * kStampedPieces, grid, rec_stamp,
                                                     p.status, group_s + b * kGroupScratchWords, 2 + b, gt);
                        if (gt < 32) {
                            const size_t at = (size_t)step0 * B;
                            const DraftOutputs o{p.token + at, p.conf + at, p.halt + at,
                                                 p.feats ? p.feats + at * kNFeat : nullptr, p.final_stats, nullptr, 0,
                                                 ChainLink{}};
                            const int Hc = p.clf_H;
                            const bool no_halt = warp_draft_epilogue(
                                mp.st, mp.key, mp.sel, static_cast<float>(s_pos0[b] + step0 + 1), step0 + 1, p.tau,
                                p.sl_max, group_s + b * kGroupScratchWords, clf_s, clf_s + Hc * kNFeat,
                                clf_s + Hc * (kNFeat + 1), clf_s + Hc * (kNFeat + 2), Hc, b, o, lane);
                            if (lane == 0) {
                                // the look-ahead bookkeeping: this CTA finishes every step, so it keeps the flags itself
                                const bool goes_on = s_forced[b] != 0x7fffffff ? (step0 + 1 < s_forced[b]) : no_halt;
                                p.chain.sl[b] = step0 + 1;
                                s_live[b] = goes_on ? 1 : 0;
                                if (goes_on) atomicAdd(&s_alive, 1);
                            }
                        }
                    }
                }
                named_barrier_sync(1, BAR_THREADS);
                if (tid == 0) {
                    const bool last_step = step0 + 1 == lp.steps;
                    const unsigned code = (s_alive > 0 && !last_step) ? kLoopContinue : kLoopStop;
                    // the launch stamp may move on: every CTA has read it (their records of this step were seen)
                    if (code == kLoopStop) *lp.epoch = launch_stamp == 0x00ffffffu ? 0u : launch_stamp;
                    // Nothing in this launch reads what a step wrote except through this word (the outputs are for later
                    // kernels, the records were consumed before the decision): no ordering is needed beside it.
                    st_relaxed_u32(lp.flags + step0, (launch_stamp << 2) | code);
                }
            }
            // ---- every CTA learns the decision ----
            if (tid == 0) {
                unsigned code = 0u;
                const long long t0 = clock64();
                for (int polls = 0;; ++polls) {
                    const unsigned f = ld_relaxed_u32(lp.flags + step0);
                    if ((f >> 2) == launch_stamp) {
                        code = f & 3u;
                        break;
                    }
                    if ((polls & 63) == 63 && (*reinterpret_cast<volatile int*>(p.status) == DISCO_ERR_TIMEOUT ||
                                               clock64() - t0 > kWaitBudgetClocks)) {
                        record_status(p.status, DISCO_ERR_TIMEOUT);
                        code = kLoopStop;
                        break;
                    }
                }
                s_code[step0] = code;
                __threadfence_block();
                mbar_arrive(go_bar);                // the producer and the MMA issuer go on (or leave)
            }
            named_barrier_sync(1, BAR_THREADS);
            if (s_code[step0] != kLoopContinue) break;
        }
        // rows requested for a step that does not take place: their copy must land before the CTA leaves
        if (h_ahead_step >= 0) mbar_wait(h_full, h_ahead_step & 1, p.status);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

inline size_t gemv_loop_fixed_smem_bytes(int RK, int clf_H, int d, int h_rows) {
    size_t b = 1024;                                             // alignment
    b += (size_t)((d + kUmmaBK - 1) / kUmmaBK) * h_rows * 128;   // hidden rows
    b += 1024;                                                   // barriers, TMEM address, decisions
    b += (size_t)RK * kGemvRowStride * 4;                        // logits of one tile
    b += (size_t)RK * sizeof(RowState);                          // running results of the rows
    b += (size_t)2 * kFoldScratchWords * 4;                      // CTA-wide fold, two copies
    b += (size_t)RK * kGroupScratchWords * 4;                    // finishing groups
    b += ((size_t)clf_H * (kNFeat + 2) + 4) * 4;                 // classifier parameters
    return b + 128;
}

}  // namespace disco
