// CPU oracle for the DISCO per-iteration logit tails (arXiv 2405.04304).
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
// CUDA library is checked against.  It is compiled into liboracle.so and may be
// loaded only by the test-suite, by the smoke check and by the benchmark's CPU
// baseline leg.  The product library never links, loads or calls it, and the
// two share no source.
//
// Every function writes out the definition it cites, one step after another,
// in double precision, with the full probability vector materialised.  Nothing
// is blocked, fused or reordered.  Host pointers everywhere; bf16 values arrive
// as raw 16-bit patterns (the upper half of an IEEE binary32).
//
// Pins (tests that fix each function to something other than itself) are in
// tests/test_oracle_pins.py.  Unpinned: nothing in this file.  (Behaviour of a
// *trained* classifier, its tuned threshold and SL_max are not reproduced at
// all: the paper prints neither weights nor values.)

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <thread>
#include <vector>

namespace {

// bf16 -> double.  Exact: bf16 is the top 16 bits of a binary32.
inline double bf16_value(uint16_t bits) {
    uint32_t u = static_cast<uint32_t>(bits) << 16;
    float f;
    std::memcpy(&f, &u, sizeof f);
    return static_cast<double>(f);
}

constexpr int ORACLE_OK = 0;
constexpr int ORACLE_BAD_ARG = -1;

}  // namespace

extern "C" {

// LM-head projection (Sec. 3: the "probability vector of the draft model" is
// the soft-max of these logits; Sec. 2: the target scores all SL+1 positions in
// one pass).   z[r,v] = sum_{j=0}^{d-1} W[v,j] * H[r,j],  j ascending, double.
// W is [V,d] row-major, H is [R,d] row-major, z is [R,V] row-major.
// nthreads > 1 splits the vocabulary rows between threads; every z[r,v] is
// still the same single ascending sum, so the result does not depend on it.
int oracle_project(const uint16_t* W, const uint16_t* H, int V, int d, int R,
                   double* z, int nthreads) {
    if (!W || !H || !z || V <= 0 || d <= 0 || R < 0) return ORACLE_BAD_ARG;
    auto slab = [&](int v0, int v1) {
        for (int r = 0; r < R; ++r)
            for (int v = v0; v < v1; ++v) {
                double acc = 0.0;
                for (int j = 0; j < d; ++j)
                    acc += bf16_value(W[(size_t)v * d + j]) * bf16_value(H[(size_t)r * d + j]);
                z[(size_t)r * V + v] = acc;
            }
    };
    if (nthreads <= 1) {
        slab(0, V);
    } else {
        std::vector<std::thread> pool;
        for (int t = 0; t < nthreads; ++t) {
            int v0 = (int)((long long)V * t / nthreads);
            int v1 = (int)((long long)V * (t + 1) / nthreads);
            pool.emplace_back(slab, v0, v1);
        }
        for (auto& th : pool) th.join();
    }
    return ORACLE_OK;
}

// Greedy token (temperature 0, Sec. 4 "greedy decoding"): the smallest index
// attaining the maximum.  *gap receives the distance between the largest and
// the second largest logit (0 on an exact tie, +inf when V == 1); the tests use
// it to find positions where fp32 and fp64 may legitimately disagree.
int oracle_argmax(const double* z, int V, int32_t* best, double* gap) {
    if (!z || !best || V <= 0) return ORACLE_BAD_ARG;
    int b = 0;
    for (int v = 1; v < V; ++v)
        if (z[v] > z[b]) b = v;
    double second = -std::numeric_limits<double>::infinity();
    for (int v = 0; v < V; ++v)
        if (v != b && z[v] > second) second = z[v];
    *best = b;
    if (gap) *gap = (V == 1) ? std::numeric_limits<double>::infinity() : z[b] - second;
    return ORACLE_OK;
}

// Soft-max at temperature 1 of the raw logits (Sec. 3, y^D_i):
// y_v = exp(z_v - m) / sum_u exp(z_u - m),  m = max_u z_u.
int oracle_softmax(const double* z, int V, double* y) {
    if (!z || !y || V <= 0) return ORACLE_BAD_ARG;
    double m = z[0];
    for (int v = 1; v < V; ++v) m = std::max(m, z[v]);
    double denom = 0.0;
    for (int v = 0; v < V; ++v) denom += std::exp(z[v] - m);
    for (int v = 0; v < V; ++v) y[v] = std::exp(z[v] - m) / denom;
    return ORACLE_OK;
}

// Top_k of Eq. 2: the k largest probabilities, descending.  Equal values keep
// the lower index first.  If V < k the tail is padded with value 0, index -1.
int oracle_topk(const double* y, int V, int k, double* vals, int32_t* ids) {
    if (!y || !vals || V <= 0 || k <= 0) return ORACLE_BAD_ARG;
    std::vector<int32_t> order(V);
    for (int v = 0; v < V; ++v) order[v] = v;
    std::stable_sort(order.begin(), order.end(),
                     [&](int32_t a, int32_t b) { return y[a] > y[b]; });
    for (int i = 0; i < k; ++i) {
        if (i < V) {
            vals[i] = y[order[i]];
            if (ids) ids[i] = order[i];
        } else {
            vals[i] = 0.0;
            if (ids) ids[i] = -1;
        }
    }
    return ORACLE_OK;
}

// Ent of Eq. 2: Shannon entropy of the whole vector, natural logarithm;
// a zero probability contributes nothing.
int oracle_entropy(const double* y, int V, double* ent) {
    if (!y || !ent || V <= 0) return ORACLE_BAD_ARG;
    double e = 0.0;
    for (int v = 0; v < V; ++v)
        if (y[v] > 0.0) e -= y[v] * std::log(y[v]);
    *ent = e;
    return ORACLE_OK;
}

// Feature vector of Eq. 2:  x = Concat(Top_k(y), Ent(y), i)  ->  k + 2 numbers.
int oracle_features(const double* y, int V, int k, int32_t pos, double* x) {
    if (!x) return ORACLE_BAD_ARG;
    int rc = oracle_topk(y, V, k, x, nullptr);
    if (rc) return rc;
    rc = oracle_entropy(y, V, &x[k]);
    if (rc) return rc;
    x[k + 1] = static_cast<double>(pos);
    return ORACLE_OK;
}

// FFN of Eq. 2, read as the "shallow 2-layer FFN" of Sec. 4: two linear layers
// nfeat -> H -> 1 with a ReLU between them and a logistic output, so that C is
// a likelihood in (0,1) of the draft token being accepted (Sec. 1).
// W1 is [H,nfeat] row-major.
int oracle_classifier(const double* x, int nfeat, const float* W1, const float* b1,
                      const float* w2, const float* b2, int H, double* C) {
    if (!x || !W1 || !b1 || !w2 || !b2 || !C || H <= 0 || nfeat <= 0) return ORACLE_BAD_ARG;
    double s = static_cast<double>(b2[0]);
    for (int j = 0; j < H; ++j) {
        double a = static_cast<double>(b1[j]);
        for (int i = 0; i < nfeat; ++i) a += static_cast<double>(W1[(size_t)j * nfeat + i]) * x[i];
        if (a < 0.0) a = 0.0;
        s += static_cast<double>(w2[j]) * a;
    }
    *C = 1.0 / (1.0 + std::exp(-s));
    return ORACLE_OK;
}

// One draft step for B independent sequences (Sec. 3): project, soft-max,
// greedy token, features, classifier, then the stopping rule
//     halt = (C < tau)  or  (n_drafted >= SL_max).
// C == tau continues.  The comparison is taken on C rounded to binary32, the
// precision in which the library holds C and tau.  Sequences with active[b]==0
// are skipped and their outputs left untouched.
// Outputs (any may be null except token): token[B], conf[B], halt[B],
// feats[B,k+2], probs[B,V], gap[B] (top-2 logit gap), topk_ids[B,k].
int oracle_draft_step(const uint16_t* W_D, const uint16_t* h_D, int V, int d, int B,
                      const int32_t* pos, const int32_t* n_drafted, const uint8_t* active,
                      const float* W1, const float* b1, const float* w2, const float* b2, int H,
                      int k, float tau, int sl_max,
                      int32_t* token, double* conf, uint8_t* halt, double* feats,
                      double* probs, double* gap, int32_t* topk_ids, int nthreads) {
    if (!W_D || !h_D || !pos || !n_drafted || !token || V <= 0 || d <= 0 || B < 0 || k <= 0)
        return ORACLE_BAD_ARG;
    std::vector<double> z(V), y(V), x(k + 2);
    for (int b = 0; b < B; ++b) {
        if (active && !active[b]) continue;
        int rc = oracle_project(W_D, h_D + (size_t)b * d, V, d, 1, z.data(), nthreads);
        if (rc) return rc;
        rc = oracle_argmax(z.data(), V, &token[b], gap ? &gap[b] : nullptr);
        if (rc) return rc;
        rc = oracle_softmax(z.data(), V, y.data());
        if (rc) return rc;
        rc = oracle_features(y.data(), V, k, pos[b], x.data());
        if (rc) return rc;
        if (topk_ids) {
            std::vector<double> tmp(k);
            oracle_topk(y.data(), V, k, tmp.data(), topk_ids + (size_t)b * k);
        }
        double C = 0.0;
        rc = oracle_classifier(x.data(), k + 2, W1, b1, w2, b2, H, &C);
        if (rc) return rc;
        if (conf) conf[b] = C;
        if (halt) halt[b] = (static_cast<float>(C) < tau) || (n_drafted[b] >= sl_max) ? 1 : 0;
        if (feats) std::copy(x.begin(), x.end(), feats + (size_t)b * (k + 2));
        if (probs) std::copy(y.begin(), y.end(), probs + (size_t)b * V);
    }
    return ORACLE_OK;
}

// Rule-based stopping test of App. F ("ppl SL-opt"): the confidence in the tokens drafted so far in
// this iteration is their perplexity  ppl_n = exp(-(1/n) sum_{j<=n} ln y_j(t_j)),  lower = more
// confident;  halt = (ppl_n > ppl_max) or (n_drafted >= SL_max).  nll_sum[b] carries the sum over the
// earlier tokens of the iteration and receives this token's term.  The comparison is taken on ppl
// rounded to binary32 (the library's precision).
int oracle_draft_step_ppl(const uint16_t* W_D, const uint16_t* h_D, int V, int d, int B,
                          const int32_t* n_drafted, const uint8_t* active, double* nll_sum, float ppl_max,
                          int sl_max, int32_t* token, double* ppl, uint8_t* halt, double* gap, int nthreads) {
    if (!W_D || !h_D || !n_drafted || !nll_sum || !token || V <= 0 || d <= 0 || B < 0) return ORACLE_BAD_ARG;
    std::vector<double> z(V), y(V);
    for (int b = 0; b < B; ++b) {
        if (active && !active[b]) continue;
        if (n_drafted[b] < 1) return ORACLE_BAD_ARG;
        int rc = oracle_project(W_D, h_D + (size_t)b * d, V, d, 1, z.data(), nthreads);
        if (rc) return rc;
        rc = oracle_argmax(z.data(), V, &token[b], gap ? &gap[b] : nullptr);
        if (rc) return rc;
        rc = oracle_softmax(z.data(), V, y.data());
        if (rc) return rc;
        nll_sum[b] += -std::log(y[token[b]]);
        const double perp = std::exp(nll_sum[b] / n_drafted[b]);
        if (ppl) ppl[b] = perp;
        if (halt) halt[b] = (static_cast<float>(perp) > ppl_max) || (n_drafted[b] >= sl_max) ? 1 : 0;
    }
    return ORACLE_OK;
}

// Acceptance at temperature 0 (Sec. 3, rejection sampling "with zero
// temperature"; Fig. 1): draft token j+1 is accepted iff it equals the target's
// greedy token at row j and every earlier draft token was accepted.
//   n = |longest matching prefix|,  bonus = target token at row n.
int oracle_accept_prefix(const int32_t* draft, const int32_t* target, int SL,
                         int32_t* n_accept, int32_t* bonus) {
    if (SL < 0 || !target || !n_accept || !bonus || (SL > 0 && !draft)) return ORACLE_BAD_ARG;
    int n = 0;
    while (n < SL && draft[n] == target[n]) ++n;
    *n_accept = n;
    *bonus = target[n];
    return ORACLE_OK;
}

// Verification tail for B sequences with ragged look-ahead (Sec. 2, Sec. 3).
// Sequence b owns rows row_off[b] .. row_off[b+1]-1 of H_T (SL_b + 1 rows) and
// draft ids draft_ids[row_off[b]-b .. row_off[b+1]-b-2] (SL_b of them).
// target_ids[R] and gap[R] are optional.
int oracle_verify_ragged(const uint16_t* W_T, const uint16_t* H_T, int V, int d,
                         const int32_t* draft_ids, const int32_t* row_off, int B,
                         int32_t* n_accept, int32_t* bonus, int32_t* target_ids, double* gap,
                         int nthreads) {
    if (!W_T || !H_T || !row_off || !n_accept || !bonus || V <= 0 || d <= 0 || B < 0)
        return ORACLE_BAD_ARG;
    std::vector<double> z(V);
    for (int b = 0; b < B; ++b) {
        int r0 = row_off[b], r1 = row_off[b + 1];
        int SL = r1 - r0 - 1;
        if (SL < 0) return ORACLE_BAD_ARG;
        std::vector<int32_t> a(SL + 1);
        for (int r = r0; r < r1; ++r) {
            int rc = oracle_project(W_T, H_T + (size_t)r * d, V, d, 1, z.data(), nthreads);
            if (rc) return rc;
            rc = oracle_argmax(z.data(), V, &a[r - r0], gap ? &gap[r] : nullptr);
            if (rc) return rc;
            if (target_ids) target_ids[r] = a[r - r0];
        }
        int rc = oracle_accept_prefix(draft_ids ? draft_ids + (r0 - b) : nullptr, a.data(), SL,
                                      &n_accept[b], &bonus[b]);
        if (rc) return rc;
    }
    return ORACLE_OK;
}

// Uniform look-ahead: every sequence has SL draft tokens and SL+1 rows.
int oracle_verify(const uint16_t* W_T, const uint16_t* H_T, int V, int d,
                  const int32_t* draft_ids, int B, int SL,
                  int32_t* n_accept, int32_t* bonus, int32_t* target_ids, double* gap,
                  int nthreads) {
    if (B < 0 || SL < 0) return ORACLE_BAD_ARG;
    std::vector<int32_t> off(B + 1);
    for (int b = 0; b <= B; ++b) off[b] = b * (SL + 1);
    return oracle_verify_ragged(W_T, H_T, V, d, draft_ids, off.data(), B, n_accept, bonus,
                                target_ids, gap, nthreads);
}

// ---------------------------------------------------------------------------
// Sampling at temperature 1 (the paper's second evaluated mode, Table 6;
// speculative sampling of Leviathan et al., which Sec. 3 names as the
// verification scheme).  Random numbers are inputs: the caller passes uniforms.
// ---------------------------------------------------------------------------

// Inverse-CDF draw from non-negative weights w[V] with a uniform u in [0, 1):
// the smallest v whose running sum w_0 + .. + w_v exceeds u * (w_0 + .. + w_{V-1}).
// Rounding can leave no such v for u next to 1: then the last v with w_v > 0.
// total (optional) receives the sum.  All weights zero: *token = -1.
int oracle_sample_cdf(const double* w, int V, double u, int32_t* token, double* total) {
    if (!w || !token || V <= 0) return ORACLE_BAD_ARG;
    double sum = 0.0;
    for (int v = 0; v < V; ++v) sum += w[v];
    if (total) *total = sum;
    const double target = u * sum;
    double run = 0.0;
    int last = -1;
    for (int v = 0; v < V; ++v) {
        run += w[v];
        if (w[v] > 0.0) last = v;
        if (run > target) {
            *token = v;
            return ORACLE_OK;
        }
    }
    *token = last;
    return ORACLE_OK;
}

// Draft step with a sampled token: as oracle_draft_step, except that the token
// is drawn from y^D = softmax(W_D h) with u[b] instead of being the arg-max.
// Features, classifier and stopping rule are unchanged (they look at y^D, not
// at the token).  p_token[b] = y^D(token); probs[B,V] = y^D (needed later by the
// verification's residual distribution).
int oracle_draft_step_sample(const uint16_t* W_D, const uint16_t* h_D, int V, int d, int B,
                             const int32_t* pos, const int32_t* n_drafted, const uint8_t* active,
                             const float* W1, const float* b1, const float* w2, const float* b2, int H,
                             int k, float tau, int sl_max, const double* u,
                             int32_t* token, double* p_token, double* conf, uint8_t* halt, double* feats,
                             double* probs, int nthreads) {
    if (!W_D || !h_D || !pos || !n_drafted || !token || !u || V <= 0 || d <= 0 || B < 0 || k <= 0)
        return ORACLE_BAD_ARG;
    std::vector<double> z(V), y(V), x(k + 2);
    for (int b = 0; b < B; ++b) {
        if (active && !active[b]) continue;
        int rc = oracle_project(W_D, h_D + (size_t)b * d, V, d, 1, z.data(), nthreads);
        if (rc) return rc;
        rc = oracle_softmax(z.data(), V, y.data());
        if (rc) return rc;
        rc = oracle_sample_cdf(y.data(), V, u[b], &token[b], nullptr);
        if (rc) return rc;
        if (p_token) p_token[b] = y[token[b]];
        rc = oracle_features(y.data(), V, k, pos[b], x.data());
        if (rc) return rc;
        double C = 0.0;
        rc = oracle_classifier(x.data(), k + 2, W1, b1, w2, b2, H, &C);
        if (rc) return rc;
        if (conf) conf[b] = C;
        if (halt) halt[b] = (static_cast<float>(C) < tau) || (n_drafted[b] >= sl_max) ? 1 : 0;
        if (feats) std::copy(x.begin(), x.end(), feats + (size_t)b * (k + 2));
        if (probs) std::copy(y.begin(), y.end(), probs + (size_t)b * V);
    }
    return ORACLE_OK;
}

// One sequence of speculative sampling, given the distributions themselves:
// yT[(SL+1), V] target rows, yD[SL, V] draft rows, draft tokens t[SL], uniforms
// ua[SL] (one per draft token) and us (one for the token that ends the
// iteration).  Draft token i is accepted iff ua_i * yD_i(t_i) < yT_i(t_i), i.e.
// with probability min(1, yT_i(t_i) / yD_i(t_i)); n = number accepted before the
// first rejection.  The next token is drawn with us from
//     norm(max(0, yT_n - yD_n))   if n < SL (a rejection at position n),
//     yT_SL                       if every draft token was accepted;
// a residual that is zero everywhere (yT_n == yD_n, where a rejection cannot
// happen except through rounding) falls back to yT_n.
int oracle_speculative_sample(const double* yT, const double* yD, const int32_t* t, int SL, int V,
                              const double* ua, double us, int32_t* n_accept, int32_t* next_token) {
    if (!yT || !n_accept || !next_token || SL < 0 || V <= 0) return ORACLE_BAD_ARG;
    if (SL > 0 && (!yD || !t || !ua)) return ORACLE_BAD_ARG;
    int n = 0;
    while (n < SL) {
        const int tok = t[n];
        if (tok < 0 || tok >= V) return ORACLE_BAD_ARG;
        const double pT = yT[(size_t)n * V + tok], pD = yD[(size_t)n * V + tok];
        if (!(ua[n] * pD < pT)) break;
        ++n;
    }
    *n_accept = n;
    std::vector<double> w(V);
    const double* rowT = yT + (size_t)n * V;
    if (n < SL) {
        const double* rowD = yD + (size_t)n * V;
        double mass = 0.0;
        for (int v = 0; v < V; ++v) {
            w[v] = std::max(0.0, rowT[v] - rowD[v]);
            mass += w[v];
        }
        if (!(mass > 0.0)) std::copy(rowT, rowT + V, w.begin());
    } else {
        std::copy(rowT, rowT + V, w.begin());
    }
    return oracle_sample_cdf(w.data(), V, us, next_token, nullptr);
}

// Verification tail with sampling for B sequences with ragged look-ahead: rows
// as in oracle_verify_ragged; the target distributions are yT_r = softmax(W_T
// H_T[r]).  The draft distributions arrive as binary32 (what a draft step
// hands over) in step-major order: draft_probs[(i * B + b) * V + v] is the
// distribution from which token i of sequence b was drawn.  ua is packed like
// draft_ids (one uniform per draft token), us[B] has one uniform per sequence.
// y_T (optional, [R, V]) receives the target distributions.
int oracle_verify_sample(const uint16_t* W_T, const uint16_t* H_T, int V, int d,
                         const int32_t* draft_ids, const float* draft_probs, const int32_t* row_off, int B,
                         const double* ua, const double* us, int32_t* n_accept, int32_t* next_token,
                         double* y_T, int nthreads) {
    if (!W_T || !H_T || !row_off || !us || !n_accept || !next_token || V <= 0 || d <= 0 || B < 0)
        return ORACLE_BAD_ARG;
    std::vector<double> z(V);
    for (int b = 0; b < B; ++b) {
        const int r0 = row_off[b], r1 = row_off[b + 1];
        const int SL = r1 - r0 - 1;
        if (SL < 0) return ORACLE_BAD_ARG;
        if (SL > 0 && (!draft_ids || !draft_probs || !ua)) return ORACLE_BAD_ARG;
        std::vector<double> yT((size_t)(SL + 1) * V), yD((size_t)SL * V);
        for (int r = r0; r < r1; ++r) {
            int rc = oracle_project(W_T, H_T + (size_t)r * d, V, d, 1, z.data(), nthreads);
            if (rc) return rc;
            rc = oracle_softmax(z.data(), V, yT.data() + (size_t)(r - r0) * V);
            if (rc) return rc;
        }
        for (int i = 0; i < SL; ++i)
            for (int v = 0; v < V; ++v) yD[(size_t)i * V + v] = draft_probs[((size_t)i * B + b) * V + v];
        if (y_T) std::copy(yT.begin(), yT.end(), y_T + (size_t)r0 * V);
        int rc = oracle_speculative_sample(yT.data(), yD.data(), draft_ids ? draft_ids + (r0 - b) : nullptr, SL, V,
                                           ua ? ua + (r0 - b) : nullptr, us[b], &n_accept[b], &next_token[b]);
        if (rc) return rc;
    }
    return ORACLE_OK;
}

// ---------------------------------------------------------------------------
// Bulk feature extraction for classifier training (App. D, Sec. 4 "SL classifier
// training"): for N positions at once, the features of Eq. 2 of the draft AND of
// the target distribution, the accepted/rejected label and the total-variation
// distance between the two distributions.
// ---------------------------------------------------------------------------

// Total variation distance TV(p, q) = (1/2) * sum_v |p_v - q_v|.
int oracle_total_variation(const double* p, const double* q, int V, double* tv) {
    if (!p || !q || !tv || V <= 0) return ORACLE_BAD_ARG;
    double s = 0.0;
    for (int v = 0; v < V; ++v) s += std::fabs(p[v] - q[v]);
    *tv = 0.5 * s;
    return ORACLE_OK;
}

// Position n (0 <= n < N) has a draft hidden state H_D[n] and a target hidden state H_T[n] (both models
// have seen the same prefix: the prompt plus the target's own tokens) and the position counter pos[n].
//   y^D = softmax(W_D H_D[n]),  y^T = softmax(W_T H_T[n])
//   feats_D[n] = Concat(Top_k(y^D), Ent(y^D), pos[n]),  feats_T[n] likewise from y^T
//   label[n]   = 1 iff arg-max y^D == arg-max y^T        (the draft token "resembles" the target token:
//                token equality, the criterion of greedy verification)
//   tv[n]      = TV(y^D, y^T)
// token_D, token_T, gap_D, gap_T (top-2 logit gaps) are optional.
int oracle_extract_features(const uint16_t* W_D, const uint16_t* H_D, int d_D,
                            const uint16_t* W_T, const uint16_t* H_T, int d_T, int V, int N,
                            const int32_t* pos, int k,
                            double* feats_D, double* feats_T, double* tv, uint8_t* label,
                            int32_t* token_D, int32_t* token_T, double* gap_D, double* gap_T, int nthreads) {
    if (!W_D || !H_D || !W_T || !H_T || !pos || !feats_D || !feats_T || !tv || !label || V <= 0 || d_D <= 0 ||
        d_T <= 0 || N < 0 || k <= 0)
        return ORACLE_BAD_ARG;
    std::vector<double> z(V), yD(V), yT(V);
    for (int n = 0; n < N; ++n) {
        int32_t tD = -1, tT = -1;
        int rc = oracle_project(W_D, H_D + (size_t)n * d_D, V, d_D, 1, z.data(), nthreads);
        if (rc) return rc;
        rc = oracle_argmax(z.data(), V, &tD, gap_D ? &gap_D[n] : nullptr);
        if (rc) return rc;
        rc = oracle_softmax(z.data(), V, yD.data());
        if (rc) return rc;
        rc = oracle_project(W_T, H_T + (size_t)n * d_T, V, d_T, 1, z.data(), nthreads);
        if (rc) return rc;
        rc = oracle_argmax(z.data(), V, &tT, gap_T ? &gap_T[n] : nullptr);
        if (rc) return rc;
        rc = oracle_softmax(z.data(), V, yT.data());
        if (rc) return rc;
        rc = oracle_features(yD.data(), V, k, pos[n], feats_D + (size_t)n * (k + 2));
        if (rc) return rc;
        rc = oracle_features(yT.data(), V, k, pos[n], feats_T + (size_t)n * (k + 2));
        if (rc) return rc;
        rc = oracle_total_variation(yD.data(), yT.data(), V, &tv[n]);
        if (rc) return rc;
        label[n] = tD == tT ? 1 : 0;
        if (token_D) token_D[n] = tD;
        if (token_T) token_T[n] = tT;
    }
    return ORACLE_OK;
}

// ---------------------------------------------------------------------------
// One whole speculative iteration with the look-ahead decided on the fly (Sec. 3:
// "immediately after generating any draft token" the classifier decides whether
// the draft model generates the next token or the target takes over; never more
// than SL_max draft tokens).
// ---------------------------------------------------------------------------

// Draft phase.  Sequence b drafts token i = 1, 2, ... from the hidden state
// h_D[i-1, b] (h_D is [SL_max, B, d]: the draft model's body is not part of this
// path, its outputs are given).  The token's position feature is pos0[b] + i,
// where pos0[b] counts the tokens generated before this iteration, and its
// n_drafted is i.  After token i:
//   * sl_forced == null: the stopping rule of oracle_draft_step decides
//     (classifier below tau, or i == SL_max);
//   * sl_forced != null: the policy is overruled and sequence b drafts exactly
//     min(sl_forced[b], SL_max) tokens (sl_forced[b] >= 1); the classifier still
//     runs and its outputs are reported.
// tau <= 0 is the static policy (SL = SL_max); tau > 1 gives SL = 1.
// Outputs are step-major [SL_max, B] (feats [SL_max, B, k+2]); entries of steps a
// sequence did not take are left untouched.  sl[b] = tokens drafted.
int oracle_draft_loop(const uint16_t* W_D, const uint16_t* h_D, int V, int d, int B,
                      const int32_t* pos0, const float* W1, const float* b1, const float* w2,
                      const float* b2, int H, int k, float tau, int sl_max, const int32_t* sl_forced,
                      int32_t* token, double* conf, uint8_t* halt, double* feats, double* gap,
                      int32_t* sl, int nthreads) {
    if (!W_D || !h_D || !pos0 || !token || !sl || V <= 0 || d <= 0 || B < 0 || sl_max < 1 || k <= 0)
        return ORACLE_BAD_ARG;
    for (int b = 0; b < B; ++b) {
        if (sl_forced && sl_forced[b] < 1) return ORACLE_BAD_ARG;
        sl[b] = 0;
        for (int i = 1; i <= sl_max; ++i) {
            const size_t at = (size_t)(i - 1) * B + b;   // step-major slot of (step i, sequence b)
            const int32_t pos = pos0[b] + i, n_drafted = i;
            uint8_t stop = 0;
            int rc = oracle_draft_step(W_D, h_D + at * d, V, d, 1, &pos, &n_drafted, nullptr, W1, b1, w2, b2, H,
                                       k, tau, sl_max, &token[at], conf ? &conf[at] : nullptr, &stop,
                                       feats ? feats + at * (k + 2) : nullptr, nullptr,
                                       gap ? &gap[at] : nullptr, nullptr, nthreads);
            if (rc) return rc;
            if (halt) halt[at] = stop;
            sl[b] = i;
            if (sl_forced ? (i >= sl_forced[b]) : (stop != 0)) break;
        }
    }
    return ORACLE_OK;
}

// Verification of the tokens the draft phase produced, in the fixed-shape layout
// the SL_max footnote of Sec. 3 points to: H_T is [B, SL_max+1, d] (row j of
// sequence b is the target hidden state that predicts the token after draft
// token j; only rows 0 .. sl[b] are looked at), the draft tokens are
// draft[b * stride_b + j * stride_j], j < sl[b].  n_accept, bonus as in
// oracle_accept_prefix.  target_ids / gap are [B, SL_max+1]; entries beyond
// sl[b] are left untouched.
int oracle_verify_padded(const uint16_t* W_T, const uint16_t* H_T, int V, int d, int B, int sl_max,
                         const int32_t* sl, const int32_t* draft, long long stride_b, long long stride_j,
                         int32_t* n_accept, int32_t* bonus, int32_t* target_ids, double* gap,
                         int nthreads) {
    if (!W_T || !H_T || !sl || !n_accept || !bonus || V <= 0 || d <= 0 || B < 0 || sl_max < 0)
        return ORACLE_BAD_ARG;
    std::vector<double> z(V);
    for (int b = 0; b < B; ++b) {
        const int SL = sl[b];
        if (SL < 0 || SL > sl_max || (SL > 0 && !draft)) return ORACLE_BAD_ARG;
        std::vector<int32_t> a(SL + 1), t(SL);
        for (int j = 0; j < SL; ++j) t[j] = draft[(long long)b * stride_b + (long long)j * stride_j];
        for (int j = 0; j <= SL; ++j) {
            const size_t row = (size_t)b * (sl_max + 1) + j;
            int rc = oracle_project(W_T, H_T + row * d, V, d, 1, z.data(), nthreads);
            if (rc) return rc;
            rc = oracle_argmax(z.data(), V, &a[j], gap ? &gap[row] : nullptr);
            if (rc) return rc;
            if (target_ids) target_ids[row] = a[j];
        }
        int rc = oracle_accept_prefix(SL ? t.data() : nullptr, a.data(), SL, &n_accept[b], &bonus[b]);
        if (rc) return rc;
    }
    return ORACLE_OK;
}

// The iteration: draft phase, then verification of what it drafted.
//   draft_ids == null: the target checks the tokens the draft phase produced
//                      (token[j, b], the real loop);
//   draft_ids != null: [B, SL_max] ids offered to the target instead (the synthetic
//                      workloads plant the target's own tokens there, corrupted with a
//                      given probability, to set the acceptance rate).
int oracle_iteration(const uint16_t* W_D, const uint16_t* h_D, int d_D, const uint16_t* W_T,
                     const uint16_t* H_T, int d_T, int V, int B, const int32_t* pos0,
                     const float* W1, const float* b1, const float* w2, const float* b2, int H, int k,
                     float tau, int sl_max, const int32_t* sl_forced, const int32_t* draft_ids,
                     int32_t* token, double* conf, uint8_t* halt, double* feats, double* gap_D,
                     int32_t* sl, int32_t* n_accept, int32_t* bonus, int32_t* target_ids, double* gap_T,
                     int nthreads) {
    int rc = oracle_draft_loop(W_D, h_D, V, d_D, B, pos0, W1, b1, w2, b2, H, k, tau, sl_max, sl_forced,
                               token, conf, halt, feats, gap_D, sl, nthreads);
    if (rc) return rc;
    if (draft_ids)
        return oracle_verify_padded(W_T, H_T, V, d_T, B, sl_max, sl, draft_ids, sl_max, 1, n_accept, bonus,
                                    target_ids, gap_T, nthreads);
    return oracle_verify_padded(W_T, H_T, V, d_T, B, sl_max, sl, token, 1, B, n_accept, bonus, target_ids,
                                gap_T, nthreads);
}

int oracle_hardware_threads() { return (int)std::thread::hardware_concurrency(); }

}  // extern "C"
