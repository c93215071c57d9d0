// CUDA-core streaming kernel for the logit tails when only a few hidden rows share one pass over
// the LM head (the single-sequence draft step above all).  The projection is then a GEMV: every
// LM-head byte is read once and used for RT fused multiply-adds, so the kernel is built around
// HBM streaming, not around tensor cores.
//
//   * one CTA per slab of consecutive vocabulary rows; a producer warp streams the slab through a
//     ring of shared-memory slots with bulk (TMA-unit) copies signalled on mbarriers;
//   * each ring slot is owned by one consumer warp, which works on up to four vocabulary rows at
//     once: 128-bit shared loads, fp32 FMAs, shuffle reduction; the logits are warp-uniform and
//     go straight into the warp's online soft-max state, its top-10 values and its running arg-max;
//   * per-CTA partials (64-byte records) go to scratch; the last CTA to take a ticket merges them
//     and runs the fused epilogue (features + halt classifier + stopping rule, or prefix match +
//     bonus token).
//
// The LM head is never written by this library, so the kernel starts streaming it before it waits
// (griddepcontrol.wait) for the preceding kernel of the stream; everything that kernel may have
// produced (hidden states, scratch) is touched only after the wait.
//
// More than RT hidden rows are handled by passing over the slab again (correct for any R, but
// the tcgen05 kernel is the one meant for many rows).
#pragma once

#include "common.cuh"

namespace disco {

// Verification in the fixed-shape layout (the SL_max footnote of Sec. 3): every sequence owns SL + 1 rows
// (SL = the cap), of which the first sl[b] + 1 count; sl[b] is device memory that the draft phase wrote.
// Draft token j of sequence b is ids[b * stride_b + j * stride_j].
struct VerifyPadded {
    const int32_t* sl;        // [B]; null: not this mode
    long long stride_b, stride_j;
    int32_t* row_off_out;     // [B + 1] or null: exclusive prefix sums of sl[b] + 1 (offsets of the packed rows)
    const int32_t* pos0;      // [B] tokens generated before this iteration (with pos_next)
    int32_t* pos_next;        // [B] or null: pos0[b] + n_accept[b] + 1, the next iteration's pos0 (may be pos0 itself)
    const int32_t* packed_off;  // [B + 1] or null.  Non-null: the hidden rows were packed before the projection (row_off of
                                // the packed rows, computed on the device): the keys of sequence b start at packed_off[b],
                                // while its outputs keep the fixed-shape layout
};

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
    float4* part_rec;          // [R][grid] records: (m, Z, S, -), top-10 logits descending, arg-max key
    unsigned long long* keys;  // [R] packed arg-max keys, zero between calls
    unsigned int* ticket;      // zero between calls
    int* status;
    float* final_stats;  // [R][2] (m, Z) for the optional probs pass
    // draft step
    const int32_t* pos;
    const int32_t* n_drafted;
    const uint8_t* active;
    ChainLink chain;     // alive != null: this launch is one step of a draft phase chained on the device
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
    float* nll_sum;      // non-null: perplexity rule instead of the classifier (tau is then the perplexity bound)
    int stats_only;      // 1: arg-max and soft-max statistics only (pos, n_drafted, classifier unused); 2: token and
                         // features only (classifier, n_drafted unused)
    // sampled draft step (non-null u_draw): the token is drawn from the soft-max by the second phase, from the
    // per-CTA sums and the one slab of logits (in probs) that holds u * total; at most 160 CTAs
    const float* u_draw;  // [B] uniforms in [0, 1)
    float* p_token;       // [B] or null: probability of the drawn token
    // words that the kernel after this one counts in (the tickets of a verification with sampling): cleared here
    unsigned int* clear_words;
    int clear_n;
    int slab_rows;        // vocabulary rows per CTA (the slab of record c starts at c * slab_rows)
    // verification
    const int32_t* draft_ids;
    const int32_t* row_off;  // null: uniform SL
    int B, SL;
    int32_t* n_accept;
    int32_t* bonus;
    int32_t* target_ids;
    VerifyPadded padded;     // sl != null: fixed-shape rows, per-sequence look-ahead read from the device
};

constexpr int kRecordWords = 16;  // one partial record: m, Z, S, -, 10 logits, key (2 words)
// Shared scratch owned by one warp in the second phase: 16 words for the features of Eq. 2, then the
// work area of warp_merge_partials (a pool of whole records, the candidate list, the ten results).
constexpr int kMergePoolRecords = 16;
constexpr int kMergeCandidates = 64;
constexpr int kWarpScratchWords = 16 + kMergePoolRecords * 12 + kMergeCandidates + 16;

inline size_t stream_tail_smem_bytes(int RT, int NW, int d, int stages, uint32_t slot_bytes, int clf_H) {
    size_t b = (size_t)stages * slot_bytes;           // ring
    b += (size_t)RT * d * 2;                          // hidden tile
    b += (size_t)stages * 16;                         // full/empty barriers
    b += (size_t)(NW * RT + 1) * kRecordWords * 4;    // warp records / finalize staging (+ carry)
    b += (size_t)NW * kWarpScratchWords * 4;          // second-phase scratch per warp
    b += ((size_t)clf_H * (kNFeat + 2) + 4) * 4;      // classifier parameters
    return b + 128;
}

// ---------------------------------------------------------------------------------------------
// partial records
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned long long key_from_words(float lo, float hi) {
    return (static_cast<unsigned long long>(__float_as_uint(hi)) << 32) | __float_as_uint(lo);
}

// One partial record held by a lane: statistics, arg-max key and a descending list of 16 values
// (the ten logits of the record, then -inf).
struct LaneRecord {
    float m, Z, S;
    unsigned long long key;
    float l[16];
    __device__ __forceinline__ void clear() {
        m = DISCO_NEG_INF;
        Z = 0.f;
        S = 0.f;
        key = 0ull;
#pragma unroll
        for (int k = 0; k < 16; ++k) l[k] = DISCO_NEG_INF;
    }
    __device__ __forceinline__ void set(const float4& q, const float4& a, const float4& b, const float4& c) {
        clear();
        if (q.y > 0.f) {
            m = q.x, Z = q.y, S = q.z;
            key = key_from_words(c.z, c.w);
            l[0] = a.x, l[1] = a.y, l[2] = a.z, l[3] = a.w, l[4] = b.x, l[5] = b.y, l[6] = b.z, l[7] = b.w;
            l[8] = c.x, l[9] = c.y;
        }
    }
    // Fold another record into this one, inside the lane: statistics, key, and the two descending
    // lists merged by a bitonic network (max(a[i], b[15 - i]) holds the 16 largest as a bitonic sequence).
    __device__ __forceinline__ void absorb(const LaneRecord& o) {
        if (!(o.Z > 0.f)) return;
        SoftmaxState st;
        st.m = m, st.Z = Z, st.S = S;
        st.merge(o.m, o.Z, o.S);
        m = st.m, Z = st.Z, S = st.S;
        key = o.key > key ? o.key : key;
#pragma unroll
        for (int i = 0; i < 16; ++i) l[i] = fmaxf(l[i], o.l[15 - i]);
#pragma unroll
        for (int stride = 8; stride > 0; stride >>= 1) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                if ((i & stride) == 0) {
                    const float hi = fmaxf(l[i], l[i + stride]);
                    const float lo = fminf(l[i], l[i + stride]);
                    l[i] = hi;
                    l[i + stride] = lo;
                }
            }
        }
    }
};

// Reduce the records held by the lanes of a warp (lanes without one hold a cleared record).  Afterwards
// the low lanes hold the merged statistics, the largest key and, in l[0..9], the ten largest logits.
//   * statistics: one integer max-reduction for the reference maximum, one exponential per lane, then
//     shuffle sums (much shorter than a butterfly of pairwise merges);
//   * lists: a bitonic merge network across lanes: max(a[i], partner[15 - i]) keeps the 16 largest of
//     two descending lists as a bitonic sequence, four compare-exchange stages sort it again.
// `levels` = ceil(log2(number of lanes that may hold a record)): lanes 0 .. 2^levels - 1 end up with the
// result (lane 0 always does).
__device__ __forceinline__ void warp_reduce_records(LaneRecord& r, int levels) {
    const uint32_t mbits = __reduce_max_sync(kFullMask, ordered_bits(r.m));
    const float M = from_ordered_bits(mbits);
    float Zc = 0.f, Sc = 0.f;
    if (r.Z > 0.f) {
        const float dm = r.m - M;
        const float e = __expf(dm);
        Zc = r.Z * e;
        Sc = e * (r.S + dm * r.Z);
    }
#pragma unroll 1
    for (int lv = 0; lv < levels; ++lv) {
        const int off = 1 << lv;
        Zc += __shfl_xor_sync(kFullMask, Zc, off);
        Sc += __shfl_xor_sync(kFullMask, Sc, off);
        const unsigned long long k2 = __shfl_xor_sync(kFullMask, r.key, off);
        r.key = k2 > r.key ? k2 : r.key;
        float o[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) o[i] = __shfl_xor_sync(kFullMask, r.l[15 - i], off);
#pragma unroll
        for (int i = 0; i < 16; ++i) r.l[i] = fmaxf(r.l[i], o[i]);
#pragma unroll
        for (int stride = 8; stride > 0; stride >>= 1) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                if ((i & stride) == 0) {
                    const float hi = fmaxf(r.l[i], r.l[i + stride]);
                    const float lo = fminf(r.l[i], r.l[i + stride]);
                    r.l[i] = hi;
                    r.l[i + stride] = lo;
                }
            }
        }
    }
    r.m = M;
    r.Z = Zc;
    r.S = Sc;
}

__device__ __forceinline__ int ceil_log2(int n) { return n <= 1 ? 0 : 32 - __clz(n - 1); }

// Result of merging the partial records of one sequence: statistics and key in every lane, the k-th
// largest logit in lane k < 10 (-inf elsewhere).
struct MergedPartials {
    SoftmaxState st;
    unsigned long long key;
    float sel;
    float zs[5];   // up to 160 records: sum of e^(z - m) over the slab of record j * 32 + lane (0 if none)
};

// Stamped records (80 bytes): five 16-byte pieces, each three payload words and the stamp of the launch
// that wrote it: (m, Z, S | l0 l1 l2 | l3 l4 l5 | l6 l7 l8 | l9, key lo, key hi).  A 16-byte piece is
// written and read as one access, so a reader that finds the current stamp in a piece holds that
// piece's payload of this launch, whatever the order in which the pieces travel: no fence, barrier or
// counter lies between writer and reader (a fence at GPU scope costs about 1.5 us here).  The buffer is
// written by nothing else and starts zeroed; the stamp is never zero.
constexpr int kStampedPieces = 5;
__device__ __forceinline__ void store_relaxed_v4(float4* p, float a, float b, float c, float d) {
    asm volatile("st.relaxed.gpu.global.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ float4 load_relaxed_v4(const float4* p) {
    float4 v;
    asm volatile("ld.relaxed.gpu.global.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "l"(p)
                 : "memory");
    return v;
}
__device__ __forceinline__ void store_stamped_record(float4* rec, float m, float Z, float S, const float (&l)[kTopK],
                                                     unsigned long long key, uint32_t stamp) {
    const float sf = __uint_as_float(stamp);
    store_relaxed_v4(rec, m, Z, S, sf);
    store_relaxed_v4(rec + 1, l[0], l[1], l[2], sf);
    store_relaxed_v4(rec + 2, l[3], l[4], l[5], sf);
    store_relaxed_v4(rec + 3, l[6], l[7], l[8], sf);
    store_relaxed_v4(rec + 4, l[9], __uint_as_float(static_cast<uint32_t>(key & 0xffffffffull)),
                     __uint_as_float(static_cast<uint32_t>(key >> 32)), sf);
}

// Merge the NP partial records of one sequence (consecutive) by one warp.
// stamp == 0: plain 64-byte records, complete before the call.  stamp != 0: stamped 80-byte records that
// other CTAs of this launch are still writing; wait (bounded, status gets DISCO_ERR_TIMEOUT) until each
// carries the stamp.
// Up to 160 records take one L2 round trip, five per lane, and the ten largest logits are found by
// selection instead of a merge tree: the tenth largest of the lanes' largest logits is a lower bound
// on the tenth largest overall; the few records whose head reaches it are copied whole to a pool in
// shared memory, the pool's values at or above the bound become candidates, and the candidates are
// ranked against each other.  More than 160 records, more than kMergePoolRecords such records or more
// than kMergeCandidates candidates (many equal logits) fall back to pairwise list merges.
// scratch: kWarpScratchWords - 16 words owned by the warp, 16-byte aligned.
// want_top10 = false: statistics and key only (sel = -inf).
__device__ __forceinline__ MergedPartials warp_merge_partials(const float4* recs, int NP, float* scratch, int lane,
                                                              uint32_t stamp = 0u, int* status = nullptr,
                                                              bool want_top10 = true) {
    constexpr int kPerLane = 5;
    MergedPartials out;
    bool fast = NP <= 32 * kPerLane;
    if (fast) {
        float4 q[kPerLane][4];
        if (stamp) {
            bool pend[kPerLane];
#pragma unroll
            for (int j = 0; j < kPerLane; ++j) {
                pend[j] = j * 32 + lane < NP;
                q[j][0] = q[j][1] = q[j][2] = q[j][3] = make_float4(0.f, 0.f, 0.f, 0.f);  // Z = 0: empty
            }
            const long long t0 = clock64();
            int polls = 0;
            for (;;) {
                // the pieces of up to three pending records are requested before any is looked at (more in
                // flight would not fit the registers): two L2 round trips per poll of the lane's five records
                bool any = false;
#pragma unroll
                for (int j0 = 0; j0 < kPerLane; j0 += 3) {
                    float4 raw[3][kStampedPieces];
#pragma unroll
                    for (int jj = 0; jj < 3; ++jj) {
                        const int j = j0 + jj;
                        if (j < kPerLane && pend[j]) {
                            const float4* src = recs + (size_t)(j * 32 + lane) * kStampedPieces;
#pragma unroll
                            for (int i = 0; i < kStampedPieces; ++i) raw[jj][i] = load_relaxed_v4(src + i);
                        }
                    }
#pragma unroll
                    for (int jj = 0; jj < 3; ++jj) {
                        const int j = j0 + jj;
                        if (j < kPerLane) {
                            if (pend[j]) {
                                bool good = true;
#pragma unroll
                                for (int i = 0; i < kStampedPieces; ++i)
                                    good = good && __float_as_uint(raw[jj][i].w) == stamp;
                                if (good) {
                                    pend[j] = false;
                                    q[j][0] = make_float4(raw[jj][0].x, raw[jj][0].y, raw[jj][0].z, 0.f);
                                    q[j][1] = make_float4(raw[jj][1].x, raw[jj][1].y, raw[jj][1].z, raw[jj][2].x);
                                    q[j][2] = make_float4(raw[jj][2].y, raw[jj][2].z, raw[jj][3].x, raw[jj][3].y);
                                    q[j][3] = make_float4(raw[jj][3].z, raw[jj][4].x, raw[jj][4].y, raw[jj][4].z);
                                }
                            }
                            any = any || pend[j];
                        }
                    }
                }
                if (!__any_sync(kFullMask, any)) break;
                if ((++polls & 63) == 0 && (*reinterpret_cast<volatile int*>(status) == DISCO_ERR_TIMEOUT ||
                                            clock64() - t0 > kWaitBudgetClocks)) {
                    record_status(status, DISCO_ERR_TIMEOUT);
                    break;
                }
            }
        } else {
#pragma unroll
            for (int j = 0; j < kPerLane; ++j) {
                const int c = j * 32 + lane;
                if (c < NP) {
                    const float4* src = recs + (size_t)c * 4;
                    q[j][0] = __ldcg(src), q[j][1] = __ldcg(src + 1), q[j][2] = __ldcg(src + 2), q[j][3] = __ldcg(src + 3);
                } else {
                    q[j][0] = q[j][1] = q[j][2] = q[j][3] = make_float4(0.f, 0.f, 0.f, 0.f);  // Z = 0: empty
                }
            }
        }
        float4* pool = reinterpret_cast<float4*>(scratch);                  // kMergePoolRecords x 3 float4
        float* cand = scratch + kMergePoolRecords * 12;                     // kMergeCandidates
        float* res = cand + kMergeCandidates;                               // kTopK
        if (lane < kTopK) res[lane] = DISCO_NEG_INF;
        // reference maximum, key and largest logit of the lane's records
        float lm = DISCO_NEG_INF, head = DISCO_NEG_INF;
        unsigned long long key = 0ull;
#pragma unroll
        for (int j = 0; j < kPerLane; ++j) {
            if (q[j][0].y > 0.f) {
                lm = fmaxf(lm, q[j][0].x);
                head = fmaxf(head, q[j][1].x);
                const unsigned long long k2 = key_from_words(q[j][3].z, q[j][3].w);
                key = k2 > key ? k2 : key;
            }
        }
        // statistics: one max-reduction, the exponentials of all records side by side, shuffle sums
        const float M = from_ordered_bits(__reduce_max_sync(kFullMask, ordered_bits(lm)));
        float Zc = 0.f, Sc = 0.f;
#pragma unroll
        for (int j = 0; j < kPerLane; ++j) {
            out.zs[j] = 0.f;
            if (q[j][0].y > 0.f) {
                const float dm = q[j][0].x - M;
                const float e = __expf(dm);
                out.zs[j] = q[j][0].y * e;
                Zc += out.zs[j];
                Sc = fmaf(e, fmaf(dm, q[j][0].y, q[j][0].z), Sc);
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            Zc += __shfl_xor_sync(kFullMask, Zc, off);
            Sc += __shfl_xor_sync(kFullMask, Sc, off);
        }
        const uint32_t khi = __reduce_max_sync(kFullMask, static_cast<uint32_t>(key >> 32));
        const uint32_t klo = __reduce_max_sync(
            kFullMask, static_cast<uint32_t>(key >> 32) == khi ? static_cast<uint32_t>(key & 0xffffffffull) : 0u);
        out.st.m = M, out.st.Z = Zc, out.st.S = Sc;
        out.key = (static_cast<unsigned long long>(khi) << 32) | klo;
        if (!want_top10) {
            out.sel = DISCO_NEG_INF;
            return out;
        }
        // threshold: the head of rank 9 among the 32 lanes' heads (ties broken by lane)
        int rank = 0;
#pragma unroll
        for (int s2 = 0; s2 < 32; ++s2) {
            const float o = __shfl_sync(kFullMask, head, s2);
            rank += (o > head || (o == head && s2 < lane)) ? 1 : 0;
        }
        const unsigned who = __ballot_sync(kFullMask, rank == kTopK - 1);
        const float theta = __shfl_sync(kFullMask, head, __ffs(who) - 1);
        // records whose largest logit reaches the threshold go to the pool, whole
        const unsigned lt = (1u << lane) - 1u;
        int nrec = 0;
#pragma unroll
        for (int j = 0; j < kPerLane; ++j) {
            const bool qual = q[j][0].y > 0.f && q[j][1].x >= theta && q[j][1].x > DISCO_NEG_INF;
            const unsigned mask = __ballot_sync(kFullMask, qual);
            const int slot = nrec + __popc(mask & lt);
            if (qual && slot < kMergePoolRecords) {
                pool[slot * 3] = q[j][1];
                pool[slot * 3 + 1] = q[j][2];
                pool[slot * 3 + 2] = make_float4(q[j][3].x, q[j][3].y, DISCO_NEG_INF, DISCO_NEG_INF);
            }
            nrec += __popc(mask);
        }
        fast = nrec <= kMergePoolRecords;
        int n = 0;
        if (fast) {
            __syncwarp();
            // pool values at or above the threshold become candidates (the pool's padding is -inf)
            const float* pv = reinterpret_cast<const float*>(pool);
            for (int i0 = 0; i0 < nrec * 12; i0 += 32) {
                const int i = i0 + lane;
                const float v = i < nrec * 12 ? pv[i] : DISCO_NEG_INF;
                const bool qual = v >= theta && v > DISCO_NEG_INF;
                const unsigned mask = __ballot_sync(kFullMask, qual);
                const int slot = n + __popc(mask & lt);
                if (qual && slot < kMergeCandidates) cand[slot] = v;
                n += __popc(mask);
            }
            fast = n <= kMergeCandidates;
        }
        if (fast) {
            const int n4 = (n + 3) & ~3;
            if (lane < n4 - n) cand[n + lane] = DISCO_NEG_INF;  // pad to whole float4s
            __syncwarp();
            // rank the candidates against each other; ranks 0..9 are the result
            for (int idx = lane; idx < n; idx += 32) {
                const float x = cand[idx];
                int r = 0;
                for (int t = 0; t < n4; t += 4) {
                    const float4 y = *reinterpret_cast<const float4*>(cand + t);
                    r += (y.x > x || (y.x == x && t < idx)) ? 1 : 0;
                    r += (y.y > x || (y.y == x && t + 1 < idx)) ? 1 : 0;
                    r += (y.z > x || (y.z == x && t + 2 < idx)) ? 1 : 0;
                    r += (y.w > x || (y.w == x && t + 3 < idx)) ? 1 : 0;
                }
                if (r < kTopK) res[r] = x;
            }
            __syncwarp();
            out.sel = lane < kTopK ? res[lane] : DISCO_NEG_INF;
            __syncwarp();
            return out;
        }
        __syncwarp();
    }
    // general case: pairwise merges of descending lists
    LaneRecord r;
    r.clear();
    const long long t0 = clock64();
    int polls = 0;
#pragma unroll 1
    for (int c0 = 0; c0 < NP; c0 += 32) {
        const int c = c0 + lane;
        if (c < NP) {
            LaneRecord o;
            if (stamp) {
                const float4* src = recs + (size_t)c * kStampedPieces;
                for (;;) {
                    const float4 a = load_relaxed_v4(src), b = load_relaxed_v4(src + 1), c2 = load_relaxed_v4(src + 2),
                                 d = load_relaxed_v4(src + 3), e = load_relaxed_v4(src + 4);
                    if (__float_as_uint(a.w) == stamp && __float_as_uint(b.w) == stamp && __float_as_uint(c2.w) == stamp &&
                        __float_as_uint(d.w) == stamp && __float_as_uint(e.w) == stamp) {
                        o.set(make_float4(a.x, a.y, a.z, 0.f), make_float4(b.x, b.y, b.z, c2.x),
                              make_float4(c2.y, c2.z, d.x, d.y), make_float4(d.z, e.x, e.y, e.z));
                        break;
                    }
                    if ((++polls & 63) == 0 && (*reinterpret_cast<volatile int*>(status) == DISCO_ERR_TIMEOUT ||
                                                clock64() - t0 > kWaitBudgetClocks)) {
                        record_status(status, DISCO_ERR_TIMEOUT);
                        o.clear();
                        break;
                    }
                }
            } else {
                const float4* src = recs + (size_t)c * 4;
                o.set(__ldcg(src), __ldcg(src + 1), __ldcg(src + 2), __ldcg(src + 3));
            }
            r.absorb(o);
        }
    }
    warp_reduce_records(r, 5);
    out.st.m = r.m, out.st.Z = r.Z, out.st.S = r.S;
    out.key = __shfl_sync(kFullMask, r.key, 0);
    out.sel = DISCO_NEG_INF;
#pragma unroll
    for (int k = 0; k < kTopK; ++k) {
        const float v = __shfl_sync(kFullMask, r.l[k], 0);
        out.sel = (lane == k) ? v : out.sel;
    }
    return out;
}

// Lane 0 holds (m, Z, S, key); lane k < 10 holds the k-th logit: write them as one record.
__device__ __forceinline__ void warp_store_record(float* rec, const SoftmaxState& st, unsigned long long key, float sel,
                                                  int lane) {
    if (lane == 0) {
        rec[0] = st.m;
        rec[1] = st.Z;
        rec[2] = st.S;
        rec[3] = 0.f;
        rec[14] = __uint_as_float(static_cast<uint32_t>(key & 0xffffffffull));
        rec[15] = __uint_as_float(static_cast<uint32_t>(key >> 32));
    }
    if (lane < kTopK) rec[4 + lane] = sel;
}

// Store the reduced record that lane 0 holds (the other lanes may hold partial results).
__device__ __forceinline__ void warp_store_record(float* rec, const LaneRecord& r, int lane) {
    float sel = DISCO_NEG_INF;
#pragma unroll
    for (int k = 0; k < kTopK; ++k) {
        const float v = __shfl_sync(kFullMask, r.l[k], 0);
        sel = (lane == k) ? v : sel;
    }
    SoftmaxState st;
    st.m = r.m, st.Z = r.Z, st.S = r.S;
    warp_store_record(rec, st, r.key, sel, lane);
}

// ---------------------------------------------------------------------------------------------
// fused epilogues
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

// Features of Eq. 2 from merged statistics, then classifier and stopping rule; one warp.
// sel: lane k < 10 holds the k-th largest logit.  Returns (lane 0) whether the sequence drafts on.
struct DraftOutputs {
    int32_t* token;
    float* conf;
    uint8_t* halt;
    float* feats;
    float* final_stats;
    float* nll_sum;  // non-null: perplexity rule (App. F) instead of the classifier
    int stats_only;  // 1: arg-max and soft-max statistics only (rows of a verification with sampling);
                     // 2: token and features, no classifier (bulk feature extraction)
    ChainLink chain; // draft phase chained on the device: the look-ahead bookkeeping goes with the halt flag
};
__device__ __forceinline__ bool warp_draft_epilogue(const SoftmaxState& st, unsigned long long key, float sel, float fpos,
                                                    int n_drafted, float tau, int sl_max, float* feat_s, const float* W1,
                                                    const float* b1, const float* w2, const float* b2, int Hc, int b,
                                                    const DraftOutputs& o, int lane) {
    if (o.stats_only == 1) {
        if (lane == 0) {
            if (o.token) o.token[b] = key_index(key);
            o.final_stats[2 * b] = st.m;
            o.final_stats[2 * b + 1] = st.Z;
        }
        return false;
    }
    if (o.nll_sum) {
        // Perplexity rule: the greedy token attains the largest logit, so -ln y(token) = ln Z.  The caller
        // keeps the running sum over the tokens drafted in this iteration; halt when the perplexity of
        // that run exceeds the bound (here passed in tau) or the cap is reached.
        if (lane == 0) {
            const float nll = o.nll_sum[b] + logf(st.Z);
            const float ppl = expf(nll / static_cast<float>(n_drafted));
            o.nll_sum[b] = nll;
            o.token[b] = key_index(key);
            o.conf[b] = ppl;
            o.halt[b] = ((ppl > tau) || (n_drafted >= sl_max)) ? 1 : 0;
            o.final_stats[2 * b] = st.m;
            o.final_stats[2 * b + 1] = st.Z;
        }
        return false;
    }
    const float inv_Z = 1.f / st.Z;
    const float prob = (lane < kTopK && sel > DISCO_NEG_INF) ? __expf(sel - st.m) * inv_Z : 0.f;
    const float ent = __logf(st.Z) - st.S * inv_Z;
    const float x = lane < kTopK ? prob : (lane == kTopK ? ent : (lane == kTopK + 1 ? fpos : 0.f));
    if (o.stats_only == 2) {
        if (lane == 0) {
            if (o.token) o.token[b] = key_index(key);
            o.final_stats[2 * b] = st.m;
            o.final_stats[2 * b + 1] = st.Z;
        }
        if (o.feats && lane < kNFeat) o.feats[(size_t)b * kNFeat + lane] = x;
        return false;
    }
    const float C = warp_halt_classifier(x, feat_s, W1, b1, w2, b2, Hc, lane);
    bool goes_on = false;
    if (lane == 0) {
        const bool halt = (C < tau) || (n_drafted >= sl_max);
        o.token[b] = key_index(key);
        o.conf[b] = C;
        o.halt[b] = halt ? 1 : 0;
        goes_on = chain_record(o.chain, b, halt);
        o.final_stats[2 * b] = st.m;
        o.final_stats[2 * b + 1] = st.Z;
    }
    if (o.feats && lane < kNFeat) o.feats[(size_t)b * kNFeat + lane] = x;
    return goes_on;   // lane 0: the sequence drafts another token after this one
}

// Inverse-CDF draw of one token by one warp, after warp_merge_partials: the records are in vocabulary
// order (record c = the slab of rows [c * slab_rows, (c + 1) * slab_rows)), so the running sums of their
// scaled Z locate the slab that holds u * Z; inside it the logits (row `logits` of the probs buffer, still
// unnormalised) are exponentiated again, summed a contiguous piece per lane, scanned, and the lane that
// holds the crossing walks its piece.  Returns the token (every lane) and its probability.
__device__ __forceinline__ int warp_draw_token(const MergedPartials& mp, int NP, int slab_rows, int V,
                                               const float* logits, float u, int lane, float* p_out) {
    const float target = u * mp.st.Z;
    // inclusive running sums in record order: a scan per group of 32 records, groups in sequence
    float base = 0.f, my_before = 0.f;
    int my_c = -1, last_c = -1;
#pragma unroll
    for (int j = 0; j < 5; ++j) {
        float incl = mp.zs[j];
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const float o = __shfl_up_sync(kFullMask, incl, off);
            if (lane >= off) incl += o;
        }
        incl += base;
        const float excl = incl - mp.zs[j];
        if (my_c < 0 && mp.zs[j] > 0.f && excl <= target && incl > target) {
            my_c = j * 32 + lane;
            my_before = excl;
        }
        if (mp.zs[j] > 0.f) last_c = j * 32 + lane;
        base = __shfl_sync(kFullMask, incl, 31);
    }
    // the first record that crosses; rounding next to u = 1: the last record with mass
    const unsigned who = __ballot_sync(kFullMask, my_c >= 0);
    int c;
    float before;
    if (who) {
        const int src = __ffs(who) - 1;
        c = __shfl_sync(kFullMask, my_c, src);
        before = __shfl_sync(kFullMask, my_before, src);
    } else {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) last_c = max(last_c, __shfl_xor_sync(kFullMask, last_c, off));
        c = last_c;
        before = DISCO_NEG_INF;   // nothing crosses: the walk below ends at the slab's last entry with mass
    }
    if (c < 0 || c >= NP) {
        if (p_out) *p_out = 0.f;
        return -1;
    }
    const int v0 = c * slab_rows, v1 = min(V, v0 + slab_rows);
    const int piece = (v1 - v0 + 31) / 32;
    const int p0 = min(v1, v0 + lane * piece), p1 = min(v1, p0 + piece);
    float mine = 0.f;
    for (int v = p0; v < p1; ++v) mine += __expf(__ldcg(logits + v) - mp.st.m);
    float incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const float o = __shfl_up_sync(kFullMask, incl, off);
        if (lane >= off) incl += o;
    }
    incl += before;
    const bool cross = (incl - mine) <= target && incl > target;
    unsigned w2 = __ballot_sync(kFullMask, cross);
    // the re-summed slab may fall short of the record's sum in its last bit: then the last lane with mass
    if (!w2) {
        const unsigned has = __ballot_sync(kFullMask, mine > 0.f);
        w2 = has ? (1u << (31 - __clz(has))) : 1u;
    }
    const int owner = __ffs(w2) - 1;
    int tok = -1;
    float pe = 0.f;
    if (lane == owner) {
        float run = incl - mine;
        for (int v = p0; v < p1; ++v) {
            const float e = __expf(__ldcg(logits + v) - mp.st.m);
            if (e > 0.f) {   // remember the last entry with mass in case the sum never crosses
                tok = v;
                pe = e;
            }
            run += e;
            if (run > target) break;
        }
    }
    tok = __shfl_sync(kFullMask, tok, owner);
    pe = __shfl_sync(kFullMask, pe, owner);
    if (p_out) *p_out = pe / mp.st.Z;
    return tok;
}

// Draft step, sequence b, in the last CTA, by ONE warp (the warps take different sequences): merge the
// per-CTA records, then features, classifier and stopping rule.
// feat16: kWarpScratchWords words of shared memory owned by the calling warp.
__device__ __forceinline__ void finalize_draft_seq(const TailParams& p, int b, int grid, float* feat16, const float* clf_s,
                                                   int lane) {
    // issued early: hidden behind the merge
    const float fpos = p.chain.alive ? static_cast<float>(p.chain.pos0[b] + p.chain.step)
                                     : (p.pos ? static_cast<float>(p.pos[b]) : 0.f);
    const int n_drafted = p.chain.alive ? p.chain.step : (p.n_drafted ? p.n_drafted[b] : 0);
    const MergedPartials mp =
        warp_merge_partials(p.part_rec + (size_t)b * grid * 4, grid, feat16 + 16, lane, 0u, nullptr, p.stats_only != 1);
    const int Hc = p.clf_H;
    const SoftmaxState st = mp.st;
    const DraftOutputs o{p.token, p.conf, p.halt, p.feats, p.final_stats, p.nll_sum, p.stats_only, p.chain};
    warp_draft_epilogue(st, mp.key, mp.sel, fpos, n_drafted, p.tau, p.sl_max, feat16, clf_s, clf_s + Hc * kNFeat,
                        clf_s + Hc * (kNFeat + 1), clf_s + Hc * (kNFeat + 2), Hc, b, o, lane);
    if (p.u_draw) {   // the greedy token is replaced by a draw from the distribution
        float pt = 0.f;
        const int tok = warp_draw_token(mp, grid, p.slab_rows, p.V, p.probs + (size_t)b * p.V, p.u_draw[b], lane, &pt);
        if (lane == 0) {
            p.token[b] = tok;
            if (p.p_token) p.p_token[b] = pt;
        }
    }
}

// Verification: decode the arg-max keys, match the draft prefix, pick the bonus token.
// One warp per sequence; lane j looks at row j of the sequence.  Three row layouts: packed rows with
// offsets (row_off), a uniform look-ahead SL, or the fixed-shape layout with the look-ahead read from
// device memory (pad.sl).
__device__ __forceinline__ void verify_one_sequence(const unsigned long long* keys, const int32_t* draft_ids,
                                                    const int32_t* row_off, int B, int SL, int R, int b,
                                                    int32_t* n_accept, int32_t* bonus, int32_t* target_ids,
                                                    int* status, int lane, const VerifyPadded& pad) {
    int r0, r1;
    int out0 = -1;            // first row of the sequence in target_ids when that differs from its first key row
    long long id0, idj = 1;
    bool bad;
    if (pad.sl) {
        const int s = __ldcg(pad.sl + b);
        out0 = b * (SL + 1);
        r0 = pad.packed_off ? __ldcg(pad.packed_off + b) : out0;
        r1 = r0 + s + 1;
        id0 = (long long)b * pad.stride_b;
        idj = pad.stride_j;
        bad = s < 0 || s > SL || r0 < 0 || r1 > R;
    } else {
        if (row_off) {
            r0 = row_off[b];
            r1 = row_off[b + 1];
        } else {
            r0 = b * (SL + 1);
            r1 = r0 + SL + 1;
        }
        id0 = r0 - b;
        // every sequence owns at least one row, so row_off[b] >= b and R - row_off[b+1] >= B - 1 - b: offsets that
        // break this would put the sequence's draft ids (which start at r0 - b) outside the [R - B] array
        bad = r0 < b || r1 <= r0 || r1 > R - (B - 1 - b) || (b == 0 && r0 != 0) || (b == B - 1 && r1 != R);
    }
    if (bad) {
        if (lane == 0) {
            record_status(status, DISCO_ERR_INVALID_ARG);
            n_accept[b] = -1;
            bonus[b] = -1;
        }
        return;
    }
    const int sl = r1 - r0 - 1;
    int n_acc = -1, bonus_tok = -1;
    for (int j0 = 0; j0 <= sl; j0 += 32) {
        const int j = j0 + lane;
        int a = -1;
        bool match = false;
        if (j <= sl) {
            a = key_index(__ldcg(keys + r0 + j));
            if (target_ids) target_ids[(out0 >= 0 ? out0 : r0) + j] = a;
            match = (j < sl) && (__ldcg(draft_ids + id0 + j * idj) == a);
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
        if (pad.sl && pad.pos_next) pad.pos_next[b] = pad.pos0[b] + n_acc + 1;   // n_acc accepted tokens and the bonus token
    }
}

// Fixed-shape verification: offsets of the packed rows, row_off[b] = sum over b' < b of (sl[b'] + 1), for the
// caller's next stage.  One warp.
__device__ __forceinline__ void warp_write_row_offsets(const VerifyPadded& pad, int B, int SL, int lane) {
    if (!pad.sl || !pad.row_off_out) return;
    int base = 0;
    for (int b0 = 0; b0 < B; b0 += 32) {
        const int b = b0 + lane;
        int rows = 0;
        if (b < B) rows = min(max(__ldcg(pad.sl + b), 0), SL) + 1;
        int incl = rows;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int o = __shfl_up_sync(kFullMask, incl, off);
            if (lane >= off) incl += o;
        }
        if (b < B) pad.row_off_out[b] = base + incl - rows;
        base += __shfl_sync(kFullMask, incl, 31);
    }
    if (lane == 0) pad.row_off_out[B] = base;
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
    float* wstate = reinterpret_cast<float*>(empty + p.stages);  // 16-byte aligned
    float* feat_s = wstate + (NW * RT + 1) * kRecordWords;
    float* clf_s = feat_s + NW * kWarpScratchWords;
    __shared__ int s_is_last;

    const int v0 = blockIdx.x * p.rows_per_cta;
    const int nrows = min(p.V, v0 + p.rows_per_cta) - v0;
    const int nslots = (nrows + p.rps - 1) / p.rps;
    const int nchunks = (p.R + RT - 1) / RT;

    // the next kernel of the stream may start its own prologue now
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

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
    if (DRAFT && p.clf_H > 0) {  // classifier parameters -> shared, asynchronously; only the last CTA reads them
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
    // from here on the kernel reads the hidden states and writes scratch and outputs: the preceding
    // kernel of the stream must have finished
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (blockIdx.x == 0)
        for (int i = tid; i < p.clear_n; i += BAR_THREADS) p.clear_words[i] = 0u;

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

        // Running state of this warp per hidden row, and the block of logits not folded into it yet:
        // the warp-uniform logit of the cnt-th vocabulary row this warp meets is parked in lane cnt % 32.
        SoftmaxState st[RT];
        float top_v[RT], best_v[RT], blk_v[RT];
        int best_i[RT];
        int blk_idx = 0, cnt = 0;
#pragma unroll
        for (int r = 0; r < RT; ++r) {
            st[r].init();
            top_v[r] = DISCO_NEG_INF;
            best_v[r] = DISCO_NEG_INF;
            best_i[r] = kNoIndex;
            blk_v[r] = DISCO_NEG_INF;
        }
        // scratch for the rank scatter: the warp's record slots (written for good only after the loop)
        float* fold_scratch = wstate + (warp * RT) * kRecordWords + 4;
        // rows whose logits go to the optional probs output: none of a masked sequence's outputs is written
        bool keep_logits[RT];
#pragma unroll
        for (int r = 0; r < RT; ++r) {
            const int row = chunk * RT + r;
            keep_logits[r] = DRAFT && p.probs && row < p.R && (!p.active || p.active[row]);
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
                        const bool mine = lane == (cnt & 31);
                        if (mine) blk_idx = v;
#pragma unroll
                        for (int r = 0; r < RT; ++r) {
                            const float z = __fadd_rn(acc[g][r], 0.f);  // folds -0 into +0
                            if (mine) blk_v[r] = z;
                            if (keep_logits[r] && lane == 0) p.probs[(size_t)(chunk * RT + r) * p.V + v] = z;
                        }
                        if ((++cnt & 31) == 0) {  // 32 logits parked: fold them
#pragma unroll
                            for (int r = 0; r < RT; ++r) {
                                warp_fold_block(blk_v[r], blk_idx, 32, lane, st[r], best_v[r], best_i[r], top_v[r],
                                                fold_scratch + r * kRecordWords);
                                blk_v[r] = DISCO_NEG_INF;
                            }
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[s]);  // the slot may be refilled
            }
        }

        if (cnt & 31) {  // the last, partial block
#pragma unroll
            for (int r = 0; r < RT; ++r)
                warp_fold_block(blk_v[r], blk_idx, cnt & 31, lane, st[r], best_v[r], best_i[r], top_v[r],
                                fold_scratch + r * kRecordWords);
        }

        // ---- merge the NW warps of this CTA, publish the CTA's result for each hidden row ----
        if (DRAFT) {
#pragma unroll
            for (int r = 0; r < RT; ++r) {
                const unsigned long long key = best_i[r] != kNoIndex ? argmax_key(best_v[r], best_i[r]) : 0ull;
                warp_store_record(wstate + (warp * RT + r) * kRecordWords, st[r], key, top_v[r], lane);
            }
            named_barrier_sync(1, BAR_THREADS);
            for (int r = warp; r < RT; r += NW) {
                const int row = chunk * RT + r;
                if (row >= p.R) continue;
                // the records of hidden row r sit RT records apart; lane w < NW takes warp w's
                LaneRecord rec;
                rec.clear();
                if (lane < NW) {
                    const float4* sr = reinterpret_cast<const float4*>(wstate + (lane * RT + r) * kRecordWords);
                    rec.set(sr[0], sr[1], sr[2], sr[3]);
                }
                warp_reduce_records(rec, ceil_log2(NW));
                warp_store_record(reinterpret_cast<float*>(p.part_rec + ((size_t)row * grid + blockIdx.x) * 4), rec, lane);
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
        for (int b = warp; b < p.R; b += NW) {
            if (!chain_seq_live(p.chain, p.active, b)) continue;
            finalize_draft_seq(p, b, grid, feat_s + warp * kWarpScratchWords, clf_s, lane);
        }
        named_barrier_sync(1, BAR_THREADS);
    } else {
        for (int b = warp; b < p.B; b += NW)
            verify_one_sequence(p.keys, p.draft_ids, p.row_off, p.B, p.SL, p.R, b, p.n_accept, p.bonus,
                                p.target_ids, p.status, lane, p.padded);
        if (warp == 0) warp_write_row_offsets(p.padded, p.B, p.SL, lane);
        named_barrier_sync(1, BAR_THREADS);
        for (int r = tid; r < p.R; r += BAR_THREADS) p.keys[r] = 0ull;
    }
    if (tid == 0) *p.ticket = 0u;
}

// Fixed-shape verification with many rows: the rows that count (the first sl[b] + 1 of each sequence's SL + 1) are
// copied next to each other, so that the projection does not pay for the padding.  Block (b, j) copies row j of
// sequence b to packed row off[b] + j, where off[b] = sum over b' < b of (sl[b'] + 1) (every block sums what it
// needs itself; block (0, 0) also writes all B + 1 offsets, off[B] = the number of packed rows).
// grid = (SL + 1, B), 128 threads.
struct PackParams {
    const uint16_t* H;    // bf16 [B, SL + 1, d]
    uint16_t* packed;     // bf16 [<= B * (SL + 1), d]
    const int32_t* sl;    // [B]
    int32_t* off;         // [B + 1]
    int32_t* off_user;    // [B + 1] or null: a second copy for the caller
    int B, SL, d;
};
static __global__ void __launch_bounds__(128) pack_rows_kernel(const PackParams p) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    __shared__ int s_part[4];
    const int j = blockIdx.x, b = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    auto rows_of = [&](int q) { return min(max(__ldcg(p.sl + q), 0), p.SL) + 1; };
    if (j == 0 && b == 0) {   // all offsets, by one warp
        if (warp == 0) {
            int base = 0;
            for (int q0 = 0; q0 < p.B; q0 += 32) {
                const int q = q0 + lane;
                const int rows = q < p.B ? rows_of(q) : 0;
                int incl = rows;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int t = __shfl_up_sync(kFullMask, incl, o);
                    if (lane >= o) incl += t;
                }
                if (q < p.B) {
                    p.off[q] = base + incl - rows;
                    if (p.off_user) p.off_user[q] = base + incl - rows;
                }
                base += __shfl_sync(kFullMask, incl, 31);
            }
            if (lane == 0) {
                p.off[p.B] = base;
                if (p.off_user) p.off_user[p.B] = base;
            }
        }
    }
    if (j >= rows_of(b)) return;   // a padding row (uniform over the block)
    int part = 0;
    for (int q = threadIdx.x; q < b; q += blockDim.x) part += rows_of(q);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(kFullMask, part, o);
    if (lane == 0) s_part[warp] = part;
    __syncthreads();
    const int dst = s_part[0] + s_part[1] + s_part[2] + s_part[3] + j;
    const uint4* src = reinterpret_cast<const uint4*>(p.H + ((size_t)b * (p.SL + 1) + j) * p.d);
    uint4* out = reinterpret_cast<uint4*>(p.packed + (size_t)dst * p.d);
    for (int c = threadIdx.x; c < p.d / 8; c += blockDim.x) out[c] = __ldg(src + c);
}

// probs[b, v] currently holds the raw logit; turn it into the soft-max probability.
static __global__ void normalize_probs_kernel(float* probs, const float* final_stats, const uint8_t* active, int V) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int b = blockIdx.y;
    if (active && !active[b]) return;
    const float m = final_stats[2 * b], inv_Z = 1.f / final_stats[2 * b + 1];
    for (int v = blockIdx.x * blockDim.x + threadIdx.x; v < V; v += gridDim.x * blockDim.x)
        probs[(size_t)b * V + v] = expf(probs[(size_t)b * V + v] - m) * inv_Z;
}

}  // namespace disco
