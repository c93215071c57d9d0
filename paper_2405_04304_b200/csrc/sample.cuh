// Sampling at temperature 1 (the paper's Table 6 mode): inverse-CDF draws from probability rows that
// the LM-head kernels have left in global memory, and the accept / resample rule of speculative
// sampling (Leviathan et al., named in Sec. 3 as the verification scheme).
//
// Random numbers are inputs: one uniform in [0, 1) per draw.  Running sums are kept in double precision,
// in vocabulary order, so that a draw depends on the probabilities only and not on how the row is split
// over threads (the split changes the rounding of a double sum in its last bits at most).
#pragma once

#include "common.cuh"

namespace disco {

constexpr int kSampleThreads = 256;

// Inverse-CDF draw by one CTA of kSampleThreads threads: the smallest v whose running sum
// w(0) + .. + w(v) exceeds u * (w(0) + .. + w(V-1)); if rounding leaves none, the last v with w(v) > 0;
// -1 if every weight is zero.  w(v) >= 0 is a callable.  Every thread returns the token.
// sh: kSampleThreads / 32 + 2 doubles of shared memory; total (optional) receives the sum.
template <typename WeightFn>
__device__ __forceinline__ int block_sample_cdf(WeightFn w, int V, double u, double* sh, double* total_out) {
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int chunk = (V + kSampleThreads - 1) / kSampleThreads;
    const int v0 = min(V, t * chunk), v1 = min(V, v0 + chunk);
    double mine = 0.0;
    for (int v = v0; v < v1; ++v) mine += w(v);
    // inclusive scan of the per-thread sums: inside each warp, then over the warp totals
    double incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const double o = __shfl_up_sync(kFullMask, incl, off);
        if (lane >= off) incl += o;
    }
    double* warp_tot = sh;                        // [8]
    int* found = reinterpret_cast<int*>(sh + 8);  // [2]: token, last index with positive weight
    if (lane == 31) warp_tot[warp] = incl;
    if (t == 0) {
        found[0] = -1;
        found[1] = -1;
    }
    __syncthreads();
    double before = 0.0, total = 0.0;
#pragma unroll
    for (int k = 0; k < kSampleThreads / 32; ++k) {
        const double wt = warp_tot[k];
        if (k < warp) before += wt;
        total += wt;
    }
    incl += before;
    const double excl = incl - mine;
    const double target = u * total;
    // exactly one thread holds the crossing (its chunk starts at or below the target and ends above it)
    if (excl <= target && incl > target) {
        double run = excl;
        int tok = -1;
        for (int v = v0; v < v1; ++v) {
            run += w(v);
            if (run > target) {
                tok = v;
                break;
            }
        }
        // the re-walk adds in a different order than the scan: if its last bit falls short, the crossing
        // is the chunk's last entry with weight
        for (int v = v1 - 1; tok < 0 && v >= v0; --v)
            if (w(v) > 0.0) tok = v;
        if (tok >= 0) found[0] = tok;
    }
    // fallback for u next to 1: the last index with positive weight
    int last = -1;
    for (int v = v1 - 1; v >= v0; --v) {
        if (w(v) > 0.0) {
            last = v;
            break;
        }
    }
    if (last >= 0) atomicMax(&found[1], last);
    __syncthreads();
    const int tok = found[0] >= 0 ? found[0] : found[1];
    if (total_out) *total_out = total;
    __syncthreads();  // sh may be reused by the caller
    return tok;
}

// Draft side: token[b] drawn from probs[b, :] with u[b]; p_token[b] = its probability.
// One CTA per sequence; sequences with active[b] == 0 are left untouched.
static __global__ void __launch_bounds__(kSampleThreads)
sample_rows_kernel(const float* __restrict__ probs, const float* __restrict__ u, const uint8_t* __restrict__ active,
                   int V, int32_t* token, float* p_token) {
    __shared__ double sh[kSampleThreads / 32 + 2];
    const int b = blockIdx.x;
    if (active && !active[b]) return;
    const float* y = probs + (size_t)b * V;
    const int tok = block_sample_cdf([&](int v) { return static_cast<double>(__ldcg(y + v)); }, V,
                                     static_cast<double>(u[b]), sh, nullptr);
    if (threadIdx.x == 0) {
        token[b] = tok;
        if (p_token) p_token[b] = tok >= 0 ? y[tok] : 0.f;
    }
}

// Verification side, one CTA per sequence.  Rows r0 .. r1-1 of y_T are the target distributions of the
// sequence (SL + 1 of them); draft token i was drawn from draft_probs[(i * B + b), :].  Token i is
// accepted iff u_accept * y_D(t_i) < y_T(t_i); n = number accepted before the first rejection.  The next
// token is drawn with u_sample[b] from norm(max(0, y_T[n] - y_D[n])) after a rejection, from y_T[SL]
// otherwise; a residual without mass falls back to y_T[n].
struct SpecSampleParams {
    const float* y_T;          // [R, V]
    const float* draft_probs;  // [steps, B, V]
    const int32_t* draft_ids;  // [R - B]
    const int32_t* row_off;    // [B + 1] or null (uniform SL)
    const float* u_accept;     // [R - B]
    const float* u_sample;     // [B]
    int B, SL, R, V;
    int32_t* n_accept;
    int32_t* next_token;
    int* status;
};

static __global__ void __launch_bounds__(kSampleThreads) speculative_sample_kernel(const SpecSampleParams p) {
    __shared__ double sh[kSampleThreads / 32 + 2];
    __shared__ int s_n;
    const int b = blockIdx.x;
    int r0, r1;
    if (p.row_off) {
        r0 = p.row_off[b];
        r1 = p.row_off[b + 1];
    } else {
        r0 = b * (p.SL + 1);
        r1 = r0 + p.SL + 1;
    }
    const bool bad = r0 < 0 || r1 <= r0 || r1 > p.R || (b == 0 && r0 != 0) || (b == p.B - 1 && r1 != p.R);
    if (bad) {
        if (threadIdx.x == 0) {
            record_status(p.status, DISCO_ERR_INVALID_ARG);
            p.n_accept[b] = 0;
            p.next_token[b] = -1;
        }
        return;
    }
    const int sl = r1 - r0 - 1;
    if (threadIdx.x == 0) {
        int n = 0;
        while (n < sl) {
            const int tok = p.draft_ids[r0 - b + n];
            if (tok < 0 || tok >= p.V) {
                record_status(p.status, DISCO_ERR_INVALID_ARG);
                break;
            }
            const double pT = p.y_T[(size_t)(r0 + n) * p.V + tok];
            const double pD = p.draft_probs[((size_t)n * p.B + b) * p.V + tok];
            if (!(static_cast<double>(p.u_accept[r0 - b + n]) * pD < pT)) break;
            ++n;
        }
        s_n = n;
    }
    __syncthreads();
    const int n = s_n;
    const float* yT = p.y_T + (size_t)(r0 + n) * p.V;
    const double us = static_cast<double>(p.u_sample[b]);
    int tok;
    if (n < sl) {
        const float* yD = p.draft_probs + ((size_t)n * p.B + b) * p.V;
        double mass = 0.0;
        tok = block_sample_cdf(
            [&](int v) { return fmax(0.0, static_cast<double>(__ldcg(yT + v)) - static_cast<double>(__ldcg(yD + v))); },
            p.V, us, sh, &mass);
        if (!(mass > 0.0))
            tok = block_sample_cdf([&](int v) { return static_cast<double>(__ldcg(yT + v)); }, p.V, us, sh, nullptr);
    } else {
        tok = block_sample_cdf([&](int v) { return static_cast<double>(__ldcg(yT + v)); }, p.V, us, sh, nullptr);
    }
    if (threadIdx.x == 0) {
        p.n_accept[b] = n;
        p.next_token[b] = tok;
    }
}

}  // namespace disco
