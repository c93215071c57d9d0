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

// Step C of the draw below, also used on its own: entries [c0, c1) hold the crossing of `target` (the running
// sum before c0 is `before`).  They are dealt out, a few consecutive entries per thread of the whole CTA: sums in
// vocabulary order, a scan over the CTA, and the thread that holds the crossing walks its entries and writes
// the token to found[0].  piece_tot: kSampleWarps doubles of shared memory.  Ends without a barrier.
template <typename WeightFn>
__device__ __forceinline__ void block_cdf_walk(WeightFn w, int c0, int c1, double before, double target,
                                               double* piece_tot, int* found) {
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int q = (c1 - c0 + kSampleThreads - 1) / kSampleThreads;   // consecutive entries per thread
    const int p0 = min(c1, c0 + t * q), p1 = min(c1, p0 + q);
    // (eight entries at a time, their loads in flight together; the first eight stay in registers for the walk)
    constexpr int kKeep = 8;
    float first[kKeep] = {};
    double mine = 0.0;
    int mylast = -1;
    for (int v0 = p0; v0 < p1; v0 += kKeep) {
        float x[kKeep];
#pragma unroll
        for (int k = 0; k < kKeep; ++k) x[k] = v0 + k < p1 ? w(v0 + k) : 0.f;
#pragma unroll
        for (int k = 0; k < kKeep; ++k) {
            mine += static_cast<double>(x[k]);
            if (x[k] > 0.f) mylast = v0 + k;
            if (v0 == p0) first[k] = x[k];
        }
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
#pragma unroll
        for (int k = 0; k < kKeep; ++k) {
            if (tok < 0 && p0 + k < p1) {
                r2 += static_cast<double>(first[k]);
                if (r2 > target) tok = p0 + k;
            }
        }
        for (int v = p0 + kKeep; v < p1 && tok < 0; ++v) {
            r2 += static_cast<double>(w(v));
            if (r2 > target) tok = v;
        }
        found[0] = tok >= 0 ? tok : mylast;
    }
    // the scan adds in another order than the totals were: if its last bit falls short of the target, the
    // crossing is the range's last entry with weight
    if (t == kSampleThreads - 1 && !(incl > target)) {
        int sl = -1;
        for (int v = c1 - 1; v >= c0 && sl < 0; --v)
            if (w(v) > 0.f) sl = v;
        found[0] = sl;
    }
}

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
    if (win >= 0) block_cdf_walk(w, min(V, win * seg), min(V, min(V, win * seg) + seg), before, target, piece_tot, found);
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

// Verification side.  y_T arrives holding the raw logits of the R target rows (m, Z of row r in stats[2r],
// stats[2r + 1]) and leaves holding the distributions y = exp(z - m) / Z.  Rows r0 .. r1-1 belong to one
// sequence (SL + 1 of them); draft token i was drawn from draft_probs[(i * B + b), :].  Token i is accepted iff
// u_accept * y_D(t_i) < y_T(t_i); n = number accepted before the first rejection.  The next token is drawn with
// u_sample[b] from norm(max(0, y_T[n] - y_D[n])) after a rejection, from y_T[SL] otherwise; a residual without
// mass falls back to y_T[n].  With R = B (no draft tokens) this is a plain draw from each row.
//
// One launch does all of it: CTA (r, s) owns segment s of row r.  It works out n of its sequence itself (a few
// loads), normalises its segment, and, on the row the draw is from, leaves the sums of its segment's weights
// in scratch memory.  The last CTA of a sequence to finish (a ticket per sequence, zeroed by the host before
// the call) picks the segment that holds u * total and walks it.  The acceptance test reads raw logits while
// other CTAs normalise: the SL entries it reads are left raw by their owners and normalised by the last CTA.
constexpr int kSampleMaxSegments = 16;
struct SampleRowsParams {
    float* y_T;                // [R, V]
    const float* stats;        // [R][2]
    const float* draft_probs;  // [steps, B, V] (null when R == B)
    const int32_t* draft_ids;  // [R - B]
    const int32_t* row_off;    // [B + 1] or null (uniform SL)
    const float* u_accept;     // [R - B]
    const float* u_sample;     // [B]
    int B, SL, R, V;
    int SEG, seg_len;          // segments per row (<= kSampleMaxSegments) and their length (a multiple of 4)
    int32_t* n_accept;
    int32_t* next_token;
    double* seg_tot;           // scratch [B][kSampleMaxSegments][2]: weights of the draw, the row itself
    int32_t* seg_last;         // scratch, same shape: last index with positive weight (-1: none)
    unsigned int* tickets;     // [B], zero at launch
    int* status;
};

static __global__ void __launch_bounds__(kSampleThreads) sample_rows_fused_kernel(const SampleRowsParams p) {
    __shared__ double sh[40];
    __shared__ double red[4][kSampleWarps];
    __shared__ int s_b, s_n, s_skip, s_last, s_lastpos[2];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const int r = blockIdx.x / p.SEG, s = blockIdx.x - r * p.SEG;
    const int V = p.V;
    // malformed offsets are reported once per sequence, by the first CTA of row b
    if (p.row_off && r < p.B && s == 0 && t == 0) {
        const int b = r, r0 = p.row_off[b], r1 = p.row_off[b + 1];
        if (r0 < b || r1 <= r0 || r1 > p.R - (p.B - 1 - b) || (b == 0 && r0 != 0) || (b == p.B - 1 && r1 != p.R)) {
            record_status(p.status, DISCO_ERR_INVALID_ARG);
            p.n_accept[b] = 0;
            p.next_token[b] = -1;
        }
    }
    if (t == 0) {
        s_b = p.row_off ? -1 : r / (p.SL + 1);
        s_skip = -1;
        s_lastpos[0] = s_lastpos[1] = -1;
    }
    __syncthreads();
    if (p.row_off) {
        for (int b = t; b < p.B; b += kSampleThreads)
            if (p.row_off[b] <= r && r < p.row_off[b + 1]) s_b = b;
        __syncthreads();
    }
    const int b = s_b;
    if (b < 0) return;
    int r0, r1;
    if (p.row_off) {
        r0 = p.row_off[b];
        r1 = p.row_off[b + 1];
        if (r0 < b || r1 <= r0 || r1 > p.R - (p.B - 1 - b) || (b == 0 && r0 != 0) || (b == p.B - 1 && r1 != p.R)) return;
    } else {
        r0 = b * (p.SL + 1);
        r1 = r0 + p.SL + 1;
    }
    const int sl = r1 - r0 - 1;
    // (loads that wait for nothing are issued first: the uniform of the draw, this CTA's first logits)
    const float u_draw = p.u_sample[b];
    float* y = p.y_T + (size_t)r * V;
    const float m = p.stats[2 * r], inv_Z = 1.f / p.stats[2 * r + 1];
    const int v_lo = min(V, s * p.seg_len), v_hi = min(V, v_lo + p.seg_len);
    float z_first[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int v = v_lo + t + k * kSampleThreads;
        z_first[k] = v < v_hi ? __ldcg(y + v) : 0.f;
    }
    // acceptance tests of all positions side by side, then the first that fails
    if (t == 0) s_n = sl;
    __syncthreads();
    int my_tok = -1;          // position t (the first this thread tests): its token and target probability
    float my_pv = 0.f;
    for (int i = t; i < sl; i += kSampleThreads) {
        const int tok = p.draft_ids[r0 - b + i];
        bool pass = false;
        if (tok < 0 || tok >= V) {
            record_status(p.status, DISCO_ERR_INVALID_ARG);
        } else {
            const int row = r0 + i;
            const float pv = expf(__ldcg(p.y_T + (size_t)row * V + tok) - p.stats[2 * row]) * (1.f / p.stats[2 * row + 1]);
            const double pD = p.draft_probs[((size_t)i * p.B + b) * V + tok];
            pass = static_cast<double>(p.u_accept[r0 - b + i]) * pD < static_cast<double>(pv);
            if (row == r) s_skip = tok;      // this entry stays raw until every reader is done
            if (i == t) {
                my_tok = tok;
                my_pv = pv;
            }
        }
        if (!pass) atomicMin(&s_n, i);
    }
    __syncthreads();
    const int n = s_n, skip = s_skip;
    const bool draw_row = r == r0 + n;
    const float* yD = (draw_row && n < sl) ? p.draft_probs + ((size_t)n * p.B + b) * V : nullptr;
    double acc_w = 0.0, acc_y = 0.0;
    int last_w = -1, last_y = -1;
    for (int v0 = v_lo + t; v0 < v_hi; v0 += 8 * kSampleThreads) {
        float z[8], d[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int v = v0 + k * kSampleThreads;
            z[k] = v0 == v_lo + t ? z_first[k] : (v < v_hi ? __ldcg(y + v) : 0.f);
            d[k] = (yD && v < v_hi) ? __ldg(yD + v) : 0.f;
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int v = v0 + k * kSampleThreads;
            if (v < v_hi) {
                const float pv = expf(z[k] - m) * inv_Z;
                if (v != skip) y[v] = pv;
                if (draw_row) {
                    const float w = yD ? fmaxf(0.f, pv - d[k]) : pv;
                    acc_w += static_cast<double>(w);
                    acc_y += static_cast<double>(pv);
                    if (w > 0.f) last_w = max(last_w, v);
                    if (pv > 0.f) last_y = max(last_y, v);
                }
            }
        }
    }
    if (draw_row) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            acc_w += __shfl_xor_sync(kFullMask, acc_w, off);
            acc_y += __shfl_xor_sync(kFullMask, acc_y, off);
            last_w = max(last_w, __shfl_xor_sync(kFullMask, last_w, off));
            last_y = max(last_y, __shfl_xor_sync(kFullMask, last_y, off));
        }
        if (lane == 0) {
            red[0][warp] = acc_w;
            red[1][warp] = acc_y;
            atomicMax(&s_lastpos[0], last_w);
            atomicMax(&s_lastpos[1], last_y);
        }
        __syncthreads();
        if (t == 0) {
            double tw = 0.0, ty = 0.0;
            for (int k = 0; k < kSampleWarps; ++k) {
                tw += red[0][k];
                ty += red[1][k];
            }
            const size_t at = ((size_t)b * kSampleMaxSegments + s) * 2;
            p.seg_tot[at] = tw;
            p.seg_tot[at + 1] = ty;
            p.seg_last[at] = s_lastpos[0];
            p.seg_last[at + 1] = s_lastpos[1];
        }
    }
    // ticket: the last CTA of the sequence finishes it
    __threadfence();
    __syncthreads();
    if (t == 0) s_last = atomicAdd(p.tickets + b, 1u) == (unsigned)((r1 - r0) * p.SEG) - 1u;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // the entries the acceptance tests read (the first kSampleThreads positions' values are still in registers)
    if (t < sl && my_tok >= 0) p.y_T[(size_t)(r0 + t) * V + my_tok] = my_pv;
    for (int i = t + kSampleThreads; i < sl; i += kSampleThreads) {
        const int tok = p.draft_ids[r0 - b + i];
        if (tok >= 0 && tok < V) {
            const int row = r0 + i;
            float* e = p.y_T + (size_t)row * V + tok;
            *e = expf(__ldcg(e) - p.stats[2 * row]) * (1.f / p.stats[2 * row + 1]);
        }
    }
    __syncthreads();
    // the draw: the segment that holds u * total, then a walk through it
    const float* yn = p.y_T + (size_t)(r0 + n) * V;
    const float* yDn = n < sl ? p.draft_probs + ((size_t)n * p.B + b) * V : nullptr;
    // (the segments' sums are fetched side by side: a loop of dependent global loads would cost a round trip each)
    double* tot = &red[0][0];                                  // [kSampleMaxSegments][2], free again
    int* lastp = reinterpret_cast<int*>(&red[2][0]);           // the same shape
    static_assert(2 * kSampleMaxSegments <= 2 * kSampleWarps, "the sums fit the reduction area");
    if (t < 2 * p.SEG) {
        tot[t] = __ldcg(p.seg_tot + (size_t)b * kSampleMaxSegments * 2 + t);
        lastp[t] = __ldcg(p.seg_last + (size_t)b * kSampleMaxSegments * 2 + t);
    }
    __syncthreads();
    double total = 0.0;
    for (int k = 0; k < p.SEG; ++k) total += tot[2 * k];
    int which = 0;
    if (yDn && !(total > 0.0)) {     // a residual without mass: the row itself
        which = 1;
        total = 0.0;
        for (int k = 0; k < p.SEG; ++k) total += tot[2 * k + 1];
    }
    const double target = static_cast<double>(u_draw) * total;
    int win = -1, lastpos = -1;
    double before = 0.0, run = 0.0;
    for (int k = 0; k < p.SEG; ++k) {
        const double nxt = run + tot[2 * k + which];
        if (win < 0 && nxt > target) {
            win = k;
            before = run;
        }
        run = nxt;
        lastpos = max(lastpos, lastp[2 * k + which]);
    }
    int* found = reinterpret_cast<int*>(sh + 2 * kSampleWarps);
    if (t == 0) found[0] = -1;
    __syncthreads();
    if (win >= 0) {
        const int c0 = min(V, win * p.seg_len), c1 = min(V, c0 + p.seg_len);
        if (yDn && which == 0)
            block_cdf_walk([&](int v) { return fmaxf(0.f, __ldcg(yn + v) - __ldg(yDn + v)); }, c0, c1, before, target,
                           sh + kSampleWarps, found);
        else
            block_cdf_walk([&](int v) { return __ldcg(yn + v); }, c0, c1, before, target, sh + kSampleWarps, found);
    }
    __syncthreads();
    if (t == 0) {
        p.n_accept[b] = n;
        p.next_token[b] = found[0] >= 0 ? found[0] : lastpos;
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
