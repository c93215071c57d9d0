// CUDA-core streaming kernel for the logit tails when only a few hidden rows share one pass over
// the LM head (the single-sequence draft step above all).  The projection is then a GEMV: every
// LM-head byte is read once and used for RT fused multiply-adds, so the kernel is built around
// HBM streaming, not around tensor cores.
//
//   * one CTA per slab of consecutive vocabulary rows; a producer warp streams the slab through a
//     ring of shared-memory slots with bulk (TMA-unit) copies signalled on mbarriers;
//   * each ring slot is owned by one consumer warp, which works on up to four vocabulary rows at
//     once: 128-bit shared loads, fp32 FMAs, shuffle reduction; the logits are warp-uniform and
//     go straight into the warp's online soft-max state and its top-10 list (draft step) or its
//     running arg-max (verification);
//   * per-CTA partials go to scratch; the last CTA to take a ticket merges them and runs the
//     fused epilogue (features + halt classifier + stopping rule, or prefix match + bonus token).
//
// More than RT hidden rows are handled by passing over the slab again (correct for any R, but
// the tcgen05 kernel is the one meant for many rows).
#pragma once

#include "common.cuh"

namespace disco {

struct TailParams {
    // projection
    const uint16_t* W;   // bf16 [V, d]
    const uint16_t* H;   // bf16 [R, d]
    int V, d, R;
    int rows_per_cta;    // slab height; grid = ceil(V / rows_per_cta)
    int rps;             // vocabulary rows per ring slot
    int stages;          // ring depth
    uint32_t slot_bytes; // rps * d * 2
    // scratch (context-owned)
    float* part_stats;   // [R][grid][4]   (m, Z, S, -)
    float* part_topv;    // [R][grid][10]
    int* part_topi;      // [R][grid][10]
    unsigned long long* keys;  // [R] packed arg-max keys, zero between calls
    unsigned int* ticket;      // zero between calls
    int* status;
    float* final_stats;  // [R][2] (m, Z) for the optional probs pass
    // draft step
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
    float* probs;
    // verification
    const int32_t* draft_ids;
    const int32_t* row_off;  // null: uniform SL
    int B, SL;
    int32_t* n_accept;
    int32_t* bonus;
    int32_t* target_ids;
};

constexpr int kWarpStateWords = 24;  // m, Z, S, pad, 10 values, 10 indices

inline size_t stream_tail_smem_bytes(int RT, int NW, int d, int stages, uint32_t slot_bytes, int clf_H) {
    size_t b = (size_t)stages * slot_bytes;           // ring
    b += (size_t)RT * d * 2;                          // hidden tile
    b += (size_t)stages * 16;                         // full/empty barriers
    b += (size_t)NW * RT * kWarpStateWords * 4;       // warp states / finalize staging
    b += 64 * 4;                                      // features
    b += ((size_t)clf_H * (kNFeat + 2) + 4) * 4;      // classifier parameters
    return b + 128;
}

// ---------------------------------------------------------------------------------------------
// fused epilogues run by the last CTA
// ---------------------------------------------------------------------------------------------

// Halt classifier of Eq. 2 by one warp: C = sigmoid(w2 . relu(W1 x + b1) + b2).  x (lane < 12) is the
// feature held by that lane; feat_s is 16 words of shared scratch owned by the warp.
__device__ __forceinline__ float warp_halt_classifier(float x, float* feat_s, const float* W1, const float* b1,
                                                      const float* w2, const float* b2p, int Hc, int lane) {
    if (lane < kNFeat) feat_s[lane] = x;
    __syncwarp();
    const float b2 = b2p[0];
    float acc = 0.f;
    for (int j = lane; j < Hc; j += 32) {
        float a = b1[j];
#pragma unroll
        for (int i = 0; i < kNFeat; ++i) a = fmaf(W1[j * kNFeat + i], feat_s[i], a);
        acc = fmaf(w2[j], fmaxf(a, 0.f), acc);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(kFullMask, acc, off);
    __syncwarp();
    return 1.f / (1.f + expf(-(acc + b2)));
}

// Draft step, sequence b: merge the per-CTA partials, form the features of Eq. 2, run the
// classifier and the stopping rule.  Called by all NW consumer warps of the last CTA.
template <int NW>
__device__ void finalize_draft_row(const TailParams& p, int b, int grid, float* stage /*NW*24 words*/,
                                   float* feat_s, const float* clf_s, int warp, int lane) {
    constexpr int BAR_THREADS = NW * 32;
    const int cpw = (grid + NW - 1) / NW;  // CTAs per warp
    const int c0 = min(grid, warp * cpw);
    const int c1 = min(grid, c0 + cpw);
    const size_t base = (size_t)b * grid;

    // issue every global load this warp needs before any of the arithmetic
    const float fpos = static_cast<float>(p.pos[b]);
    const int n_drafted = p.n_drafted[b];
    const int ncand = (c1 - c0) * kTopK;
    const float* tv = p.part_topv + (base + c0) * kTopK;
    const int* ti = p.part_topi + (base + c0) * kTopK;
    float4 q0 = make_float4(DISCO_NEG_INF, 0.f, 0.f, 0.f);
    if (c0 + lane < c1) q0 = __ldcg(reinterpret_cast<const float4*>(p.part_stats) + base + c0 + lane);
    float v0[5];
    int id0[5];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int e = j * 32 + lane;
        const bool ok = e < ncand;
        v0[j] = ok ? __ldcg(tv + e) : DISCO_NEG_INF;
        id0[j] = ok ? __ldcg(ti + e) : kNoIndex;
    }
    v0[4] = DISCO_NEG_INF;
    id0[4] = kNoIndex;

    // stage A: this warp reduces its share of the CTAs
    SoftmaxState st;
    st.init();
    st.merge(q0.x, q0.y, q0.z);
    for (int c = c0 + lane + 32; c < c1; c += 32) {
        const float4 q = __ldcg(reinterpret_cast<const float4*>(p.part_stats) + base + c);
        st.merge(q.x, q.y, q.z);
    }
    warp_merge_softmax(st);

    float run_v;
    int run_i;
    warp_select_top10<5>(v0, id0, lane, run_v, run_i);
    for (int e0 = 32 * 4; e0 < ncand; e0 += 32 * 4) {
        float v[5];
        int id[5];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int e = e0 + j * 32 + lane;
            const bool ok = e < ncand;
            v[j] = ok ? __ldcg(tv + e) : DISCO_NEG_INF;
            id[j] = ok ? __ldcg(ti + e) : kNoIndex;
        }
        v[4] = run_v;
        id[4] = run_i;
        warp_select_top10<5>(v, id, lane, run_v, run_i);
    }
    float* mine = stage + warp * kWarpStateWords;
    if (lane == 0) {
        mine[0] = st.m;
        mine[1] = st.Z;
        mine[2] = st.S;
    }
    if (lane < kTopK) {
        mine[4 + lane] = run_v;
        reinterpret_cast<int*>(mine)[4 + kTopK + lane] = run_i;
    }
    named_barrier_sync(1, BAR_THREADS);

    // stage B: warp 0 merges the NW warp results and runs the epilogue
    if (warp == 0) {
        SoftmaxState g;
        g.init();
        for (int w = lane; w < NW; w += 32)
            g.merge(stage[w * kWarpStateWords], stage[w * kWarpStateWords + 1], stage[w * kWarpStateWords + 2]);
        warp_merge_softmax(g);
        constexpr int E = (NW * kTopK + 31) / 32;
        float v[E];
        int id[E];
#pragma unroll
        for (int j = 0; j < E; ++j) {
            const int e = j * 32 + lane;
            const bool ok = e < NW * kTopK;
            const int w = ok ? e / kTopK : 0, k = ok ? e % kTopK : 0;
            v[j] = ok ? stage[w * kWarpStateWords + 4 + k] : DISCO_NEG_INF;
            id[j] = ok ? reinterpret_cast<const int*>(stage)[w * kWarpStateWords + 4 + kTopK + k] : kNoIndex;
        }
        float top_v;
        int top_i;
        warp_select_top10<E>(v, id, lane, top_v, top_i);

        // features: top-10 probabilities, entropy, position
        const float inv_Z = 1.f / g.Z;
        const float prob = (lane < kTopK && top_i != kNoIndex) ? expf(top_v - g.m) * inv_Z : 0.f;
        const float ent = logf(g.Z) - g.S * inv_Z;
        const float x = lane < kTopK ? prob : (lane == kTopK ? ent : (lane == kTopK + 1 ? fpos : 0.f));
        const float C = warp_halt_classifier(x, feat_s, clf_s, clf_s + p.clf_H * kNFeat, clf_s + p.clf_H * (kNFeat + 1),
                                             clf_s + p.clf_H * (kNFeat + 2), p.clf_H, lane);
        const int tok = __shfl_sync(kFullMask, top_i, 0);
        if (lane == 0) {
            p.token[b] = tok;
            p.conf[b] = C;
            p.halt[b] = ((C < p.tau) || (n_drafted >= p.sl_max)) ? 1 : 0;
            p.final_stats[2 * b] = g.m;
            p.final_stats[2 * b + 1] = g.Z;
        }
        if (p.feats && lane < kNFeat) p.feats[(size_t)b * kNFeat + lane] = x;
    }
    named_barrier_sync(1, BAR_THREADS);
}

// Verification: decode the arg-max keys, match the draft prefix, pick the bonus token.
// One warp per sequence; lane j looks at row j of the sequence.
__device__ __forceinline__ void verify_one_sequence(const unsigned long long* keys, const int32_t* draft_ids,
                                                    const int32_t* row_off, int B, int SL, int R, int b,
                                                    int32_t* n_accept, int32_t* bonus, int32_t* target_ids,
                                                    int* status, int lane) {
    int r0, r1;
    if (row_off) {
        r0 = row_off[b];
        r1 = row_off[b + 1];
    } else {
        r0 = b * (SL + 1);
        r1 = r0 + SL + 1;
    }
    const bool bad = r0 < 0 || r1 <= r0 || r1 > R || (b == 0 && r0 != 0) || (b == B - 1 && r1 != R);
    if (bad) {
        if (lane == 0) {
            record_status(status, DISCO_ERR_INVALID_ARG);
            n_accept[b] = -1;
            bonus[b] = -1;
        }
        return;
    }
    const int sl = r1 - r0 - 1;
    const int32_t* draft = draft_ids + (r0 - b);
    int n_acc = -1, bonus_tok = -1;
    for (int j0 = 0; j0 <= sl; j0 += 32) {
        const int j = j0 + lane;
        int a = -1;
        bool match = false;
        if (j <= sl) {
            a = key_index(__ldcg(keys + r0 + j));
            if (target_ids) target_ids[r0 + j] = a;
            match = (j < sl) && (draft[j] == a);
        }
        if (n_acc < 0) {  // warp-uniform
            const unsigned miss = ~__ballot_sync(kFullMask, match);  // bit set: that row ends the prefix
            const int first = __ffs(miss) - 1;
            if (first >= 0 && j0 + first <= sl) {
                n_acc = j0 + first;
                bonus_tok = __shfl_sync(kFullMask, a, first);
            }
        }
    }
    if (lane == 0) {
        n_accept[b] = n_acc;
        bonus[b] = bonus_tok;
    }
}

// ---------------------------------------------------------------------------------------------
// the streaming kernel
// ---------------------------------------------------------------------------------------------
template <int RT, bool DRAFT, int NW, int KC>
__global__ void __launch_bounds__((NW + 1) * 32, 1) stream_tail_kernel(const __grid_constant__ TailParams p) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    constexpr int BAR_THREADS = NW * 32;
    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const int grid = gridDim.x;
    const uint32_t row_bytes = (uint32_t)p.d * 2u;

    uint8_t* ring = smem_raw;
    uint8_t* htile = ring + (size_t)p.stages * p.slot_bytes;
    uint64_t* full = reinterpret_cast<uint64_t*>(htile + (size_t)RT * row_bytes);
    uint64_t* empty = full + p.stages;
    float* wstate = reinterpret_cast<float*>(empty + p.stages);
    float* feat_s = wstate + NW * RT * kWarpStateWords;
    float* clf_s = feat_s + 64;
    __shared__ int s_is_last;

    const int v0 = blockIdx.x * p.rows_per_cta;
    const int nrows = min(p.V, v0 + p.rows_per_cta) - v0;
    const int nslots = (nrows + p.rps - 1) / p.rps;
    const int nchunks = (p.R + RT - 1) / RT;

    if (tid == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        fence_mbar_init();
    }
    __syncthreads();

    if (warp == NW) {
        // ---------------- producer: stream the slab, once per chunk of hidden rows ----------------
        if (lane == 0) {
            const int total = nchunks * nslots;
            const uint16_t* slab = p.W + (size_t)v0 * p.d;
            int st = 0, round = 0, slot = 0;
            for (int fill = 0; fill < total; ++fill) {
                if (round > 0) mbar_wait(&empty[st], (round - 1) & 1, p.status);
                const int r0 = slot * p.rps;
                const uint32_t bytes = (uint32_t)min(p.rps, nrows - r0) * row_bytes;
                mbar_arrive_expect_tx(&full[st], bytes);
                bulk_g2s(ring + (size_t)st * p.slot_bytes, slab + (size_t)r0 * p.d, bytes, &full[st]);
                if (++st == p.stages) {
                    st = 0;
                    ++round;
                }
                if (++slot == nslots) slot = 0;
            }
        }
        return;
    }

    // -------------------- consumers --------------------
    if (DRAFT) {  // classifier parameters -> shared, asynchronously; only the last CTA reads them
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
    const int n16 = (int)(row_bytes >> 4);  // 16-byte pieces per row
    for (int chunk = 0; chunk < nchunks; ++chunk) {
        named_barrier_sync(1, BAR_THREADS);  // previous chunk's readers of the hidden tile are done
        for (int i = tid; i < RT * n16; i += BAR_THREADS) {
            const int r = i / n16, c = i - r * n16;
            const int row = chunk * RT + r;
            uint4 q = make_uint4(0, 0, 0, 0);
            if (row < p.R) q = __ldg(reinterpret_cast<const uint4*>(p.H + (size_t)row * p.d) + c);
            reinterpret_cast<uint4*>(htile)[i] = q;
        }
        named_barrier_sync(1, BAR_THREADS);

        SoftmaxState st[RT];
        WarpTop10 top[RT];
        float best_v[RT];
        int best_i[RT];
#pragma unroll
        for (int r = 0; r < RT; ++r) {
            st[r].init();
            top[r].init();
            best_v[r] = DISCO_NEG_INF;
            best_i[r] = kNoIndex;
        }

        // With one hidden row and a narrow head the warp keeps its share of h in registers.
        float hreg[KC > 0 ? KC : 1][8];
        if (KC > 0) {
#pragma unroll
            for (int k = 0; k < (KC > 0 ? KC : 1); ++k) {
                const int c = lane + 32 * k;
                uint4 q = make_uint4(0, 0, 0, 0);
                if (c < n16) q = reinterpret_cast<const uint4*>(htile)[c];
                unpack_bf16x8(q, hreg[k]);
            }
        }

        // Each ring slot belongs to one warp (slot s -> warp s % NW), so a warp meets every phase
        // of the barriers it waits on, in order: parity waits can never alias an older phase.
        // Fill f of the stream lands in slot f % stages during round f / stages.
        constexpr int G = 4 / RT;  // vocabulary rows a warp works on at once
        const int f_begin = chunk * nslots, f_end = f_begin + nslots;
        const int round_end = (f_end + p.stages - 1) / p.stages;
        for (int round = f_begin / p.stages; round < round_end; ++round) {
            for (int s = warp; s < p.stages; s += NW) {
                const int f = round * p.stages + s;
                if (f < f_begin || f >= f_end) continue;
                mbar_wait(&full[s], round & 1, p.status);
                const int r0 = (f - f_begin) * p.rps;
                const int nr = min(p.rps, nrows - r0);
                const uint8_t* slot_base = ring + (size_t)s * p.slot_bytes;
                for (int j0 = 0; j0 < nr; j0 += G) {
                    const uint4* wrow[G];
#pragma unroll
                    for (int g = 0; g < G; ++g)
                        wrow[g] = reinterpret_cast<const uint4*>(slot_base + (size_t)min(j0 + g, nr - 1) * row_bytes);
                    float acc[G][RT];
#pragma unroll
                    for (int g = 0; g < G; ++g)
#pragma unroll
                        for (int r = 0; r < RT; ++r) acc[g][r] = 0.f;
                    if (KC > 0) {
#pragma unroll
                        for (int k = 0; k < (KC > 0 ? KC : 1); ++k) {
                            const int c = min(lane + 32 * k, n16 - 1);  // past the row: h is zero there
#pragma unroll
                            for (int g = 0; g < G; ++g) {
                                float wf[8];
                                unpack_bf16x8(wrow[g][c], wf);
#pragma unroll
                                for (int e = 0; e < 8; ++e) acc[g][0] = fmaf(wf[e], hreg[k][e], acc[g][0]);
                            }
                        }
                    } else {
#pragma unroll 2
                        for (int c = lane; c < n16; c += 32) {
                            float hf[RT][8];
#pragma unroll
                            for (int r = 0; r < RT; ++r)
                                unpack_bf16x8(reinterpret_cast<const uint4*>(htile + (size_t)r * row_bytes)[c], hf[r]);
#pragma unroll
                            for (int g = 0; g < G; ++g) {
                                float wf[8];
                                unpack_bf16x8(wrow[g][c], wf);
#pragma unroll
                                for (int r = 0; r < RT; ++r)
#pragma unroll
                                    for (int e = 0; e < 8; ++e) acc[g][r] = fmaf(wf[e], hf[r][e], acc[g][r]);
                            }
                        }
                    }
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1)
#pragma unroll
                        for (int g = 0; g < G; ++g)
#pragma unroll
                            for (int r = 0; r < RT; ++r) acc[g][r] += __shfl_xor_sync(kFullMask, acc[g][r], off);
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        if (j0 + g >= nr) break;
                        const int v = v0 + r0 + j0 + g;
#pragma unroll
                        for (int r = 0; r < RT; ++r) {
                            const float z = __fadd_rn(acc[g][r], 0.f);  // folds -0 into +0
                            if (DRAFT) {
                                st[r].push(z);
                                top[r].offer(z, v, lane);
                                if (p.probs && lane == 0 && chunk * RT + r < p.R)
                                    p.probs[(size_t)(chunk * RT + r) * p.V + v] = z;
                            } else {
                                if (z > best_v[r]) {
                                    best_v[r] = z;
                                    best_i[r] = v;
                                }
                            }
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[s]);  // the slot may be refilled
            }
        }

        // ---- merge the NW warps of this CTA, publish the CTA's partial for each hidden row ----
        if (DRAFT) {
#pragma unroll
            for (int r = 0; r < RT; ++r) {
                float* mine = wstate + (warp * RT + r) * kWarpStateWords;
                if (lane == 0) {
                    mine[0] = st[r].m;
                    mine[1] = st[r].Z;
                    mine[2] = st[r].S;
                }
                if (lane < kTopK) {
                    mine[4 + lane] = top[r].v;
                    reinterpret_cast<int*>(mine)[4 + kTopK + lane] = top[r].i;
                }
            }
            named_barrier_sync(1, BAR_THREADS);
            for (int r = warp; r < RT; r += NW) {
                const int row = chunk * RT + r;
                if (row >= p.R) continue;
                SoftmaxState g;
                g.init();
                for (int w = lane; w < NW; w += 32) {
                    const float* o = wstate + (w * RT + r) * kWarpStateWords;
                    g.merge(o[0], o[1], o[2]);
                }
                warp_merge_softmax(g);
                constexpr int E = (NW * kTopK + 31) / 32;
                float v[E];
                int id[E];
#pragma unroll
                for (int j = 0; j < E; ++j) {
                    const int e = j * 32 + lane;
                    const bool ok = e < NW * kTopK;
                    const int w = ok ? e / kTopK : 0, k = ok ? e % kTopK : 0;
                    const float* o = wstate + (w * RT + r) * kWarpStateWords;
                    v[j] = ok ? o[4 + k] : DISCO_NEG_INF;
                    id[j] = ok ? reinterpret_cast<const int*>(o)[4 + kTopK + k] : kNoIndex;
                }
                float tv;
                int ti;
                warp_select_top10<E>(v, id, lane, tv, ti);
                const size_t slot = (size_t)row * grid + blockIdx.x;
                if (lane == 0) reinterpret_cast<float4*>(p.part_stats)[slot] = make_float4(g.m, g.Z, g.S, 0.f);
                if (lane < kTopK) {
                    p.part_topv[slot * kTopK + lane] = tv;
                    p.part_topi[slot * kTopK + lane] = ti;
                }
            }
        } else {
            unsigned long long* keys_s = reinterpret_cast<unsigned long long*>(wstate);
            if (tid < RT) keys_s[tid] = 0ull;
            named_barrier_sync(1, BAR_THREADS);
            if (lane == 0) {
#pragma unroll
                for (int r = 0; r < RT; ++r)
                    if (best_i[r] != kNoIndex) atomicMax(&keys_s[r], argmax_key(best_v[r], best_i[r]));
            }
            named_barrier_sync(1, BAR_THREADS);
            if (tid < RT && chunk * RT + tid < p.R && keys_s[tid] != 0ull)
                atomicMax(p.keys + chunk * RT + tid, keys_s[tid]);
        }
    }

    // -------------------- ticket: the last CTA runs the fused epilogue --------------------
    __threadfence();
    named_barrier_sync(1, BAR_THREADS);
    if (tid == 0) {
        const unsigned t = atomicAdd(p.ticket, 1u);
        s_is_last = (t == (unsigned)grid - 1u);
    }
    named_barrier_sync(1, BAR_THREADS);
    if (DRAFT) cp_async_wait_all();
    if (!s_is_last) return;
    __threadfence();

    if (DRAFT) {
        named_barrier_sync(1, BAR_THREADS);
        for (int b = 0; b < p.R; ++b) {
            if (p.active && !p.active[b]) continue;
            finalize_draft_row<NW>(p, b, grid, wstate, feat_s, clf_s, warp, lane);
        }
    } else {
        for (int b = warp; b < p.B; b += NW)
            verify_one_sequence(p.keys, p.draft_ids, p.row_off, p.B, p.SL, p.R, b, p.n_accept, p.bonus,
                                p.target_ids, p.status, lane);
        named_barrier_sync(1, BAR_THREADS);
        for (int r = tid; r < p.R; r += BAR_THREADS) p.keys[r] = 0ull;
    }
    if (tid == 0) *p.ticket = 0u;
}

// probs[b, v] currently holds the raw logit; turn it into the soft-max probability.
static __global__ void normalize_probs_kernel(float* probs, const float* final_stats, const uint8_t* active, int V) {
    const int b = blockIdx.y;
    if (active && !active[b]) return;
    const float m = final_stats[2 * b], inv_Z = 1.f / final_stats[2 * b + 1];
    for (int v = blockIdx.x * blockDim.x + threadIdx.x; v < V; v += gridDim.x * blockDim.x)
        probs[(size_t)b * V + v] = expf(probs[(size_t)b * V + v] - m) * inv_Z;
}

}  // namespace disco
