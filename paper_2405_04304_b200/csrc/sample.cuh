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

constexpr int kSampleThreads = 512;
constexpr int kSampleWarps = kSampleThreads / 32;

// Inverse-CDF draw by one CTA of kSampleThreads threads from weights w(v) >= 0, v < V (a callable that
// returns the same value whenever it is asked again): the smallest v whose running sum w(0) + .. + w(v)
// exceeds u * (sum of all); if rounding leaves none, the last v with w(v) > 0; -1 if every weight is zero.
// Every thread returns the token.  Three steps:
//   A  each warp sums one contiguous segment of the row (coalesced reads, four partial sums per lane);
//   B  every thread finds, from the 16 totals, the segment that holds u * total;
//   C  that segment is dealt out again, a few consecutive entries per thread of the whole CTA: sums in
//      vocabulary order, a scan over the CTA, and the thread that holds the crossing walks its entries.
// sh: 40 doubles of shared memory; total (optional) receives the sum.
template <typename WeightFn>
__device__ __forceinline__ int block_sample_cdf(WeightFn w, int V, double u, double* sh, double* total_out) {
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int seg = ((V + kSampleWarps - 1) / kSampleWarps + 31) & ~31;  // entries per warp, whole 32s
    const int s0 = min(V, warp * seg), s1 = min(V, s0 + seg);
    double* warp_tot = sh;                                        // [kSampleWarps] segment totals
    double* piece_tot = sh + kSampleWarps;                        // [kSampleWarps] step C: per-warp sums
    int* found = reinterpret_cast<int*>(sh + 2 * kSampleWarps);   // [2]: token, last index with positive weight
    if (t == 0) {
        found[0] = -1;
        found[1] = -1;
    }
    // A
    double part[4] = {0.0, 0.0, 0.0, 0.0};
    int last = -1;
    for (int v0 = s0 + lane; v0 < s1; v0 += 128) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int v = v0 + 32 * k;
            if (v < s1) {
                const float x = w(v);
                part[k] += static_cast<double>(x);
                if (x > 0.f) last = max(last, v);
            }
        }
    }
    double tot = (part[0] + part[1]) + (part[2] + part[3]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        tot += __shfl_xor_sync(kFullMask, tot, off);
        last = max(last, __shfl_xor_sync(kFullMask, last, off));
    }
    if (lane == 0) warp_tot[warp] = tot;
    __syncthreads();
    if (lane == 0 && last >= 0) atomicMax(&found[1], last);
    // B: the first segment whose running total exceeds the target (the same for every thread)
    double total = 0.0;
#pragma unroll
    for (int k = 0; k < kSampleWarps; ++k) total += warp_tot[k];
    const double target = u * total;
    int win = -1;
    double before = 0.0, run = 0.0;
#pragma unroll
    for (int k = 0; k < kSampleWarps; ++k) {
        const double nxt = run + warp_tot[k];
        if (win < 0 && nxt > target) {
            win = k;
            before = run;
        }
        run = nxt;
    }
    // C
    if (win >= 0) {
        const int c0 = min(V, win * seg), c1 = min(V, c0 + seg);
        const int q = (c1 - c0 + kSampleThreads - 1) / kSampleThreads;   // consecutive entries per thread
        const int p0 = min(c1, c0 + t * q), p1 = min(c1, p0 + q);
        double mine = 0.0;
        int mylast = -1;
        for (int v = p0; v < p1; ++v) {
            const float x = w(v);
            mine += static_cast<double>(x);
            if (x > 0.f) mylast = v;
        }
        double incl = mine;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const double o = __shfl_up_sync(kFullMask, incl, off);
            if (lane >= off) incl += o;
        }
        if (lane == 31) piece_tot[warp] = incl;
        __syncthreads();
        double pre = before;
#pragma unroll
        for (int k = 0; k < kSampleWarps; ++k)
            if (k < warp) pre += piece_tot[k];
        incl += pre;
        const double excl = incl - mine;
        if (excl <= target && incl > target) {   // at most one thread
            double r2 = excl;
            int tok = -1;
            for (int v = p0; v < p1; ++v) {
                r2 += static_cast<double>(w(v));
                if (r2 > target) {
                    tok = v;
                    break;
                }
            }
            found[0] = tok >= 0 ? tok : mylast;
        }
        // the scan adds in another order than step A: if its last bit falls short of the target, the
        // crossing is the segment's last entry with weight
        if (t == kSampleThreads - 1 && !(incl > target)) {
            int sl = -1;
            for (int v = c1 - 1; v >= c0 && sl < 0; --v)
                if (w(v) > 0.f) sl = v;
            found[0] = sl;
        }
    }
    __syncthreads();
    const int tok = found[0] >= 0 ? found[0] : found[1];
    if (total_out) *total_out = total;
    __syncthreads();  // sh may be reused by the caller
    return tok;
}

// Rows of up to kSampleSmemFloats entries are staged in shared memory (one pass over global memory, eight
// loads in flight per thread); longer rows are read from global memory by every step of the draw.
constexpr int kSampleSmemFloats = 50 * 1024;
constexpr int kSampleBatch = 16;
inline size_t sample_smem_bytes(int V) { return V <= kSampleSmemFloats ? (size_t)V * sizeof(float) : 0; }

// Draft side: the row probs[b, :] arrives holding the raw logits left by the LM-head pass; it is turned
// into the distribution y = exp(z - m) / Z in place (m, Z from stats[2b], stats[2b + 1]), then token[b]
// is drawn from it with u[b]; p_token[b] = its probability.  One CTA per sequence; sequences with
// active[b] == 0 are left untouched.  Dynamic shared memory: sample_smem_bytes(V).
static __global__ void __launch_bounds__(kSampleThreads)
sample_rows_kernel(float* __restrict__ probs, const float* __restrict__ stats, const float* __restrict__ u,
                   const uint8_t* __restrict__ active, int V, int use_smem, int32_t* token, float* p_token) {
    extern __shared__ float row_s[];
    __shared__ double sh[40];
    // launched with programmatic stream serialization: resident early, reading only once the LM-head
    // kernel before it has completed
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int b = blockIdx.x;
    if (active && !active[b]) return;
    float* y = probs + (size_t)b * V;
    const float m = stats[2 * b], inv_Z = 1.f / stats[2 * b + 1];
    for (int v0 = threadIdx.x; v0 < V; v0 += kSampleBatch * kSampleThreads) {
        float z[kSampleBatch];
#pragma unroll
        for (int k = 0; k < kSampleBatch; ++k) {
            const int v = v0 + k * kSampleThreads;
            z[k] = v < V ? __ldcg(y + v) : 0.f;
        }
#pragma unroll
        for (int k = 0; k < kSampleBatch; ++k) {
            const int v = v0 + k * kSampleThreads;
            if (v < V) {
                const float pv = __expf(z[k] - m) * inv_Z;
                y[v] = pv;
                if (use_smem) row_s[v] = pv;
            }
        }
    }
    __syncthreads();
    int tok;
    if (use_smem)
        tok = block_sample_cdf([&](int v) { return row_s[v]; }, V, static_cast<double>(u[b]), sh, nullptr);
    else
        tok = block_sample_cdf([&](int v) { return y[v]; }, V, static_cast<double>(u[b]), sh, nullptr);
    if (threadIdx.x == 0) {
        token[b] = tok;
        if (p_token) p_token[b] = tok >= 0 ? y[tok] : 0.f;
    }
}

// Verification side, one CTA per sequence.  Rows r0 .. r1-1 of y_T are the target distributions of the
// sequence (SL + 1 of them); draft token i was drawn from draft_probs[(i * B + b), :].  Token i is
// accepted iff u_accept * y_D(t_i) < y_T(t_i); n = number accepted before the first rejection.  The next
// token is drawn with u_sample[b] from norm(max(0, y_T[n] - y_D[n])) after a rejection, from y_T[SL]
// otherwise; a residual without mass falls back to y_T[n].  Dynamic shared memory: sample_smem_bytes(V).
struct SpecSampleParams {
    const float* y_T;          // [R, V]
    const float* draft_probs;  // [steps, B, V]
    const int32_t* draft_ids;  // [R - B]
    const int32_t* row_off;    // [B + 1] or null (uniform SL)
    const float* u_accept;     // [R - B]
    const float* u_sample;     // [B]
    int B, SL, R, V;
    int use_smem;
    int32_t* n_accept;
    int32_t* next_token;
    int* status;
};

static __global__ void __launch_bounds__(kSampleThreads) speculative_sample_kernel(const SpecSampleParams p) {
    extern __shared__ float row_s[];
    __shared__ double sh[40];
    __shared__ int s_n;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int b = blockIdx.x;
    int r0, r1;
    if (p.row_off) {
        r0 = p.row_off[b];
        r1 = p.row_off[b + 1];
    } else {
        r0 = b * (p.SL + 1);
        r1 = r0 + p.SL + 1;
    }
    const bool bad = r0 < b || r1 <= r0 || r1 > p.R - (p.B - 1 - b) || (b == 0 && r0 != 0) || (b == p.B - 1 && r1 != p.R);
    if (bad) {
        if (threadIdx.x == 0) {
            record_status(p.status, DISCO_ERR_INVALID_ARG);
            p.n_accept[b] = 0;
            p.next_token[b] = -1;
        }
        return;
    }
    const int sl = r1 - r0 - 1;
    // acceptance tests of all positions side by side (one thread each), then the first that fails
    if (threadIdx.x == 0) s_n = sl;
    __syncthreads();
    for (int i = threadIdx.x; i < sl; i += kSampleThreads) {
        const int tok = p.draft_ids[r0 - b + i];
        bool pass = false;
        if (tok < 0 || tok >= p.V) {
            record_status(p.status, DISCO_ERR_INVALID_ARG);
        } else {
            const double pT = p.y_T[(size_t)(r0 + i) * p.V + tok];
            const double pD = p.draft_probs[((size_t)i * p.B + b) * p.V + tok];
            pass = static_cast<double>(p.u_accept[r0 - b + i]) * pD < pT;
        }
        if (!pass) atomicMin(&s_n, i);
    }
    __syncthreads();
    const int n = s_n;
    const float* yT = p.y_T + (size_t)(r0 + n) * p.V;
    const float* yD = n < sl ? p.draft_probs + ((size_t)n * p.B + b) * p.V : nullptr;
    const double us = static_cast<double>(p.u_sample[b]);
    const int V = p.V;
    // weights of the draw: the residual max(0, y_T - y_D) after a rejection, y_T itself otherwise.  The
    // residual is rounded to binary32 (relative error 6e-8, far inside what the draw can resolve).
    if (p.use_smem) {
        for (int v0 = threadIdx.x; v0 < V; v0 += kSampleBatch * kSampleThreads) {
            float a[kSampleBatch], d[kSampleBatch];
#pragma unroll
            for (int k = 0; k < kSampleBatch; ++k) {
                const int v = v0 + k * kSampleThreads;
                a[k] = v < V ? __ldcg(yT + v) : 0.f;
                d[k] = (yD && v < V) ? __ldcg(yD + v) : 0.f;
            }
#pragma unroll
            for (int k = 0; k < kSampleBatch; ++k) {
                const int v = v0 + k * kSampleThreads;
                if (v < V) row_s[v] = yD ? fmaxf(0.f, a[k] - d[k]) : a[k];
            }
        }
        __syncthreads();
    }
    int tok;
    double mass = 0.0;
    if (p.use_smem)
        tok = block_sample_cdf([&](int v) { return row_s[v]; }, V, us, sh, &mass);
    else if (yD)
        tok = block_sample_cdf([&](int v) { return fmaxf(0.f, yT[v] - yD[v]); }, V, us, sh, &mass);
    else
        tok = block_sample_cdf([&](int v) { return yT[v]; }, V, us, sh, &mass);
    if (yD && !(mass > 0.0)) tok = block_sample_cdf([&](int v) { return yT[v]; }, V, us, sh, nullptr);
    if (threadIdx.x == 0) {
        p.n_accept[b] = n;
        p.next_token[b] = tok;
    }
}

// Bulk feature extraction (App. D): per position the total-variation distance TV(y^D, y^T) =
// (1/2) sum_v |y^D_v - y^T_v| of the two distributions (rows of y_D and y_T) and the accepted label
// (draft arg-max equals target arg-max).  One CTA per position.
static __global__ void __launch_bounds__(256)
tv_label_kernel(const float* __restrict__ y_D, const float* __restrict__ y_T, const int32_t* __restrict__ token_D,
                const int32_t* __restrict__ token_T, int V, float* tv, uint8_t* label) {
    __shared__ double part[8];
    const int n = blockIdx.x;
    const float* a = y_D + (size_t)n * V;
    const float* b = y_T + (size_t)n * V;
    double s = 0.0;
    for (int v0 = threadIdx.x; v0 < V; v0 += kSampleBatch * 256) {
        float x[kSampleBatch], y[kSampleBatch];
#pragma unroll
        for (int k = 0; k < kSampleBatch; ++k) {
            const int v = v0 + k * 256;
            x[k] = v < V ? __ldcg(a + v) : 0.f;
            y[k] = v < V ? __ldcg(b + v) : 0.f;
        }
#pragma unroll
        for (int k = 0; k < kSampleBatch; ++k) s += static_cast<double>(fabsf(x[k] - y[k]));
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(kFullMask, s, off);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < 8; ++w) t += part[w];
        tv[n] = static_cast<float>(0.5 * t);
        label[n] = token_D[n] == token_T[n] ? 1 : 0;
    }
}

}  // namespace disco
