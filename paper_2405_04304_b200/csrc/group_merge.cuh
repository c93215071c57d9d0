// Merging the per-CTA partial records of one sequence with SEVERAL warps (the single-warp merge is
// warp_merge_partials in stream_tail.cuh), and the small ranking helpers it is built from.  Used by the
// persistent draft-phase kernel (its finishing CTA) and by the batched draft step (one finishing group per
// sequence).  These phases are chains of dependent instructions on a few warps, so the code is written for
// short chains (values through shared memory and independent comparisons instead of shuffle chains, the loads
// of a batch in flight before the first use), not for few instructions.
#pragma once

#include "stream_tail.cuh"

namespace disco {

constexpr int kGroupMaxRecords = 160;
constexpr int kGroupMaxCandidates = 128;
// shared memory of one finishing group: cross-warp reduction slots, candidates; at least what the single-warp
// merge needs, which is the fallback for many equal logits
constexpr int kGroupScratchWords = 64 + kGroupMaxCandidates + 16 + kWarpScratchWords;

// Append the values of the lanes with `take` set to a list in shared memory (one atomic per warp).
__device__ __forceinline__ void warp_append(bool take, float v, float* list, int* count, int cap, int lane) {
    const unsigned mask = __ballot_sync(kFullMask, take);
    if (mask == 0u) return;
    int base = 0;
    if (lane == 0) base = atomicAdd(count, __popc(mask));
    base = __shfl_sync(kFullMask, base, 0);
    const int at = base + __popc(mask & ((1u << lane) - 1u));
    if (take && at < cap) list[at] = v;
}

// Rank of x among the n values of a list in shared memory whose tail up to a multiple of 32 is -inf
// (position c is x's own; equal values rank by position).  32 values at a time, all loads of a batch in
// flight before the first comparison.
__device__ __forceinline__ int rank_in_list(const float* list, int n, float x, int c) {
    int r0 = 0, r1 = 0, r2 = 0, r3 = 0;
    for (int t0 = 0; t0 < n; t0 += 32) {
        float4 y[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) y[j] = *reinterpret_cast<const float4*>(list + t0 + 4 * j);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int t = t0 + 4 * j;
            r0 += (y[j].x > x || (y[j].x == x && t < c)) ? 1 : 0;
            r1 += (y[j].y > x || (y[j].y == x && t + 1 < c)) ? 1 : 0;
            r2 += (y[j].z > x || (y[j].z == x && t + 2 < c)) ? 1 : 0;
            r3 += (y[j].w > x || (y[j].w == x && t + 3 < c)) ? 1 : 0;
        }
    }
    return (r0 + r1) + (r2 + r3);
}

// Rank of the lane's value among the warp's 32 (ties: lower lane first).  The values go through 32 words of
// shared memory owned by the warp: eight vector loads and independent comparisons instead of a chain of
// 32 shuffles.
__device__ __forceinline__ int rank_in_warp(float val, int lane, float* warp_vals) {
    warp_vals[lane] = val;
    __syncwarp();
    const int r = rank_in_list(warp_vals, 32, val, lane);
    __syncwarp();
    return r;
}

// Merge the NP <= 160 stamped records of one sequence with a group of GW warps (each thread takes at most
// ceil(160 / (32 GW)) records, and polls them until every 16-byte piece carries the stamp: bounded, status
// gets DISCO_ERR_TIMEOUT): statistics by a two-level reduction; the ten largest logits by selection -- each
// warp ranks its records' largest logits against each other, the largest of the warps' 10th-largest bounds
// the 10th largest logit overall from below, the values at or above it are collected and ranked against
// each other.  The result is valid in the group's first warp (lane k < 10 holds the k-th largest logit).
// More candidates than kGroupMaxCandidates (many equal logits) are left to a single-warp merge of the
// records, which by then are all there.
// sm: kGroupScratchWords words; bar: a named barrier reserved for the group; gt: thread index in the group.
template <int GW>
__device__ __forceinline__ MergedPartials group_merge_partials(const float4* recs, int NP, uint32_t stamp, int* status,
                                                               float* sm, int bar, int gt) {
    constexpr int GT = GW * 32;
    constexpr int PER = (kGroupMaxRecords + GT - 1) / GT;
    const int lane = gt & 31, gw = gt >> 5;
    uint32_t* red_u = reinterpret_cast<uint32_t*>(sm);        // [4][8] m bits, key hi, key lo, bits of the warp's bound
    float* red_f = sm + 32;                                    // [2][8] Z, S
    int* ncand = reinterpret_cast<int*>(sm + 48);              // [1]
    float* res = sm + 52;                                      // [10] (+2)
    float* cand = sm + 64;                                     // [kGroupMaxCandidates]
    float* fallback = cand + kGroupMaxCandidates + 16;         // kWarpScratchWords
    MergedPartials out;
    out.sel = DISCO_NEG_INF;
    float4 q[PER][4];
    {
        bool pend[PER];
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            pend[i] = gt + i * GT < NP;
            q[i][0] = q[i][1] = q[i][2] = q[i][3] = make_float4(0.f, 0.f, 0.f, 0.f);   // Z = 0: empty
        }
        const long long t0 = clock64();
        int polls = 0;
        for (;;) {
            bool any = false;
#pragma unroll
            for (int i = 0; i < PER; ++i) {
                if (pend[i]) {
                    const float4* src = recs + (size_t)(gt + i * GT) * kStampedPieces;
                    float4 raw[kStampedPieces];
#pragma unroll
                    for (int k = 0; k < kStampedPieces; ++k) raw[k] = load_relaxed_v4(src + k);
                    bool good = true;
#pragma unroll
                    for (int k = 0; k < kStampedPieces; ++k) good = good && __float_as_uint(raw[k].w) == stamp;
                    if (good) {
                        pend[i] = false;
                        q[i][0] = make_float4(raw[0].x, raw[0].y, raw[0].z, 0.f);
                        q[i][1] = make_float4(raw[1].x, raw[1].y, raw[1].z, raw[2].x);
                        q[i][2] = make_float4(raw[2].y, raw[2].z, raw[3].x, raw[3].y);
                        q[i][3] = make_float4(raw[3].z, raw[4].x, raw[4].y, raw[4].z);
                    }
                }
                any = any || pend[i];
            }
            if (!any) break;
            if ((++polls & 63) == 0 && (*reinterpret_cast<volatile int*>(status) == DISCO_ERR_TIMEOUT ||
                                        clock64() - t0 > kWaitBudgetClocks)) {
                record_status(status, DISCO_ERR_TIMEOUT);
                break;
            }
        }
    }
    float lm = DISCO_NEG_INF;
    unsigned long long key = 0ull;
    uint32_t bound = ordered_bits(DISCO_NEG_INF);   // the warp's lower bound on the 10th largest logit
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const bool has = q[i][0].y > 0.f;
        if (has) {
            lm = fmaxf(lm, q[i][0].x);
            const unsigned long long k2 = key_from_words(q[i][3].z, q[i][3].w);
            key = k2 > key ? k2 : key;
        }
        // the 10th largest of 32 records' largest logits has ten logits at or above it
        const float head = has ? q[i][1].x : DISCO_NEG_INF;
        const int rank = rank_in_warp(head, lane, fallback + gw * 32);   // (the fallback area is free until it is needed)
        const uint32_t b10 =
            __shfl_sync(kFullMask, ordered_bits(head), __ffs(__ballot_sync(kFullMask, rank == kTopK - 1)) - 1);
        bound = max(bound, b10);
    }
    const uint32_t mb = __reduce_max_sync(kFullMask, ordered_bits(lm));
    const uint32_t khi = __reduce_max_sync(kFullMask, static_cast<uint32_t>(key >> 32));
    const uint32_t klo = __reduce_max_sync(
        kFullMask, static_cast<uint32_t>(key >> 32) == khi ? static_cast<uint32_t>(key & 0xffffffffull) : 0u);
    if (lane == 0) {
        red_u[gw] = mb;
        red_u[8 + gw] = khi;
        red_u[16 + gw] = klo;
        red_u[24 + gw] = bound;
    }
    if (gt == 0) *ncand = 0;
    if (gt < 12) res[gt] = DISCO_NEG_INF;
    for (int c = gt; c < kGroupMaxCandidates; c += GT) cand[c] = DISCO_NEG_INF;
    named_barrier_sync(bar, GT);
    uint32_t Mb = 0u, Khi = 0u, Klo = 0u, Tb = 0u;
#pragma unroll
    for (int w = 0; w < GW; ++w) {
        Mb = max(Mb, red_u[w]);
        Khi = max(Khi, red_u[8 + w]);
        Tb = max(Tb, red_u[24 + w]);
    }
#pragma unroll
    for (int w = 0; w < GW; ++w) Klo = max(Klo, red_u[8 + w] == Khi ? red_u[16 + w] : 0u);
    const float M = from_ordered_bits(Mb);
    const float theta = from_ordered_bits(Tb);
    float Zc = 0.f, Sc = 0.f;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        if (q[i][0].y > 0.f) {
            const float dm = q[i][0].x - M;
            const float e = __expf(dm);
            Zc = fmaf(q[i][0].y, e, Zc);
            Sc = fmaf(e, fmaf(dm, q[i][0].y, q[i][0].z), Sc);
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        Zc += __shfl_xor_sync(kFullMask, Zc, off);
        Sc += __shfl_xor_sync(kFullMask, Sc, off);
    }
    if (lane == 0) {
        red_f[gw] = Zc;
        red_f[8 + gw] = Sc;
    }
    // candidates: every value at or above the bound (the lists are descending: position by position)
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const bool has = q[i][0].y > 0.f;
        const float l[kTopK] = {q[i][1].x, q[i][1].y, q[i][1].z, q[i][1].w, q[i][2].x,
                                q[i][2].y, q[i][2].z, q[i][2].w, q[i][3].x, q[i][3].y};
#pragma unroll
        for (int k = 0; k < kTopK; ++k) {
            const bool take = has && l[k] >= theta && l[k] > DISCO_NEG_INF;
            if (!__any_sync(kFullMask, take)) break;   // warp-uniform: no lane has a k-th value that large
            warp_append(take, l[k], cand, ncand, kGroupMaxCandidates, lane);
        }
    }
    named_barrier_sync(bar, GT);
    float Zt = 0.f, St = 0.f;
#pragma unroll
    for (int w = 0; w < GW; ++w) {
        Zt += red_f[w];
        St += red_f[8 + w];
    }
    out.st.m = M, out.st.Z = Zt, out.st.S = St;
    out.key = (static_cast<unsigned long long>(Khi) << 32) | Klo;
    const int n = *ncand;
    if (n <= kGroupMaxCandidates) {
        for (int c = gt; c < n; c += GT) {
            const float x = cand[c];
            const int r = rank_in_list(cand, n, x, c);
            if (r < kTopK) res[r] = x;
        }
        named_barrier_sync(bar, GT);
        out.sel = lane < kTopK ? res[lane] : DISCO_NEG_INF;
        return out;
    }
    // many equal logits: the single-warp merge of the records (all of which carry the stamp by now)
    if (gw == 0) out = warp_merge_partials(recs, NP, fallback, lane, stamp, status);
    named_barrier_sync(bar, GT);
    return out;
}

}  // namespace disco
