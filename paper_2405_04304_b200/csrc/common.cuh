// Shared device helpers of the DISCO logit-tail kernels: PTX wrappers (mbarrier, bulk copy),
// ordered keys for deterministic arg-max, online soft-max state, warp-resident top-10 lists.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "disco.h"

namespace disco {

constexpr int kTopK = DISCO_TOPK;
constexpr int kNFeat = DISCO_NFEAT;
constexpr unsigned kFullMask = 0xffffffffu;
constexpr int kNoIndex = 0x7fffffff;

// Bounded-wait budget: a wait gives up after this many clock ticks (about 0.05 s by default).  A device
// variable, one copy per translation unit, so that a test can shorten it (disco_test_hooks) and make a wait
// run out without anything hanging.
constexpr long long kDefaultWaitBudgetClocks = 100000000ll;
static __device__ long long g_wait_budget_clocks = kDefaultWaitBudgetClocks;
#define kWaitBudgetClocks (*reinterpret_cast<volatile long long*>(&g_wait_budget_clocks))

// ------------------------------------------------------------------------------------------
// status word
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void record_status(int* status, int code) {
    if (status) atomicCAS(status, 0, code);
}

// ------------------------------------------------------------------------------------------
// draft steps chained on the device (the draft phase of an iteration as one enqueue, Sec. 3: after every
// draft token the classifier decides whether the next one is drafted)
// ------------------------------------------------------------------------------------------
// A launch with alive != null is draft step `step` (1-based) of such a chain: the position feature of
// sequence b is pos0[b] + step, its n_drafted is step, and it takes part iff it is still drafting (every
// sequence at step 1; alive[b] afterwards, as the step before left it).  When a sequence has been finished
// the launch records sl[b] = step and alive[b] = 0 if it stops here (the stopping rule, or the forced
// look-ahead sl_forced[b] when that is given), 1 otherwise.  alive and sl are written by the predecessor
// launch: they are read and written past L1 only, after the dependency wait.
struct ChainLink {
    uint8_t* alive;            // [B] library scratch; null: a plain draft step
    int32_t* sl;               // [B] tokens drafted so far
    const int32_t* pos0;       // [B] tokens generated before this iteration
    const int32_t* sl_forced;  // [B] or null
    int step;
};

__device__ __forceinline__ bool chain_seq_live(const ChainLink& c, const uint8_t* active, int b) {
    if (c.alive) return c.step == 1 || __ldcg(c.alive + b) != 0;
    return !active || active[b] != 0;
}
// Warp-collective: does any of the B sequences still draft?  (Always true outside a chain and at step 1.)
__device__ __forceinline__ bool chain_any_live(const ChainLink& c, int B, int lane) {
    if (!c.alive || c.step == 1) return true;
    bool any = false;
    for (int b = lane; b < B; b += 32) any = any || __ldcg(c.alive + b) != 0;
    return __any_sync(0xffffffffu, any);
}
// By the thread that has just written sequence b's halt flag.  Returns whether the sequence drafts on.
__device__ __forceinline__ bool chain_record(const ChainLink& c, int b, bool halt) {
    if (!c.alive) return !halt;
    const bool stop = c.sl_forced ? (c.step >= c.sl_forced[b]) : halt;
    __stcg(c.sl + b, c.step);
    __stcg(c.alive + b, static_cast<uint8_t>(stop ? 0 : 1));
    return !stop;
}

// ------------------------------------------------------------------------------------------
// shared-memory barriers and bulk (TMA-unit) copies
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}

__device__ __forceinline__ void fence_mbar_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)),
                 "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Wait for the phase with the given parity to complete.  Never spins without bound: after
// kWaitBudgetClocks it records DISCO_ERR_TIMEOUT and returns false; the caller carries on
// (its results are then meaningless, but every later wait is bounded in the same way).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, int* status) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        // Once any wait in the grid has run out, all others give up at once.  (The status word is global
        // memory, a round trip of about a thousand cycles: it is looked at between batches of polls, never
        // ahead of a poll that may succeed.)
        if (status && *reinterpret_cast<volatile int*>(status) == DISCO_ERR_TIMEOUT) return false;
        if (clock64() - t0 > kWaitBudgetClocks) {
            record_status(status, DISCO_ERR_TIMEOUT);
            return false;
        }
    }
}

// Contiguous global -> shared copy by the TMA unit; completion is counted in bytes on `bar`.
// Both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src_gmem, uint32_t bytes,
                                         uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            smem_addr(dst_smem)),
        "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar))
        : "memory");
}

__device__ __forceinline__ void named_barrier_sync(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// 4-byte asynchronous copy global -> shared (classifier parameters)
__device__ __forceinline__ void cp_async4(void* dst_smem, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_addr(dst_smem)), "l"(src)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// ------------------------------------------------------------------------------------------
// numerics
// ------------------------------------------------------------------------------------------
#define DISCO_NEG_INF (-__int_as_float(0x7f800000))

// Monotone map float -> uint32 (larger float, larger key); -0 must have been folded into +0.
__device__ __forceinline__ uint32_t ordered_bits(float x) {
    uint32_t u = __float_as_uint(x);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float from_ordered_bits(uint32_t k) {
    uint32_t u = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
    return __uint_as_float(u);
}
// 64-bit key whose maximum is "largest value, then lowest index".  Key 0 means "nothing yet".
__device__ __forceinline__ unsigned long long argmax_key(float x, int idx) {
    return (static_cast<unsigned long long>(ordered_bits(x)) << 32) |
           static_cast<unsigned long long>(0xffffffffu - static_cast<uint32_t>(idx));
}
__device__ __forceinline__ int key_index(unsigned long long key) {
    return static_cast<int>(0xffffffffu - static_cast<uint32_t>(key & 0xffffffffull));
}

__device__ __forceinline__ void unpack_bf16x8(const uint4& q, float (&f)[8]) {
    f[0] = __uint_as_float(q.x << 16);
    f[1] = __uint_as_float(q.x & 0xffff0000u);
    f[2] = __uint_as_float(q.y << 16);
    f[3] = __uint_as_float(q.y & 0xffff0000u);
    f[4] = __uint_as_float(q.z << 16);
    f[5] = __uint_as_float(q.z & 0xffff0000u);
    f[6] = __uint_as_float(q.w << 16);
    f[7] = __uint_as_float(q.w & 0xffff0000u);
}

// Soft-max statistics of a set of logits z_i:  m = max, Z = sum e^{z_i-m}, S = sum e^{z_i-m}(z_i-m).
// Entropy = ln Z - S/Z;  probability of logit z = e^{z-m}/Z.
struct SoftmaxState {
    float m, Z, S;
    __device__ __forceinline__ void init() {
        m = DISCO_NEG_INF;
        Z = 0.f;
        S = 0.f;
    }
    __device__ __forceinline__ void push(float z) {
        if (z > m) {
            if (Z > 0.f) {
                const float dm = m - z;
                const float e = __expf(dm);
                S = e * (S + dm * Z);
                Z = Z * e + 1.f;
            } else {
                Z = 1.f;
                S = 0.f;
            }
            m = z;
        } else {
            const float t = z - m;
            const float e = __expf(t);
            Z += e;
            S = fmaf(e, t, S);
        }
    }
    __device__ __forceinline__ void merge(float m2, float Z2, float S2) {
        if (!(Z2 > 0.f)) return;
        if (!(Z > 0.f)) {
            m = m2;
            Z = Z2;
            S = S2;
            return;
        }
        const float M = fmaxf(m, m2);
        const float d1 = m - M, d2 = m2 - M;
        const float e1 = __expf(d1), e2 = __expf(d2);
        S = e1 * (S + d1 * Z) + e2 * (S2 + d2 * Z2);
        Z = Z * e1 + Z2 * e2;
        m = M;
    }
};

// A block of up to 32 logits of one hidden row, one per lane (lanes >= n hold -inf), folded into the
// warp's running state in one go: soft-max statistics by an integer max-reduction, one exponential per
// lane and shuffle sums; arg-max by a ballot (lanes hold ascending vocabulary indices, so the lowest
// lane wins ties); top-10 by rank counting (every candidate counts how many others beat it and writes
// itself to that position).  top_v: lane k < 10 holds the k-th largest value so far.  scratch: 10
// floats of shared memory owned by the warp.
__device__ __forceinline__ void warp_fold_block(float val, int idx, int n, int lane, SoftmaxState& st, float& best_v,
                                                int& best_i, float& top_v, float* scratch) {
    const uint32_t bits = ordered_bits(val);
    const uint32_t mbits = __reduce_max_sync(kFullMask, bits);
    const float M = from_ordered_bits(mbits);
    // arg-max of the block
    const int lead = __ffs(__ballot_sync(kFullMask, bits == mbits)) - 1;
    const int lead_idx = __shfl_sync(kFullMask, idx, lead);
    if (M > best_v) {
        best_v = M;
        best_i = lead_idx;
    }
    // statistics of the block, then merged into the running state
    float e = 0.f, et = 0.f;
    if (lane < n) {
        const float t = val - M;
        e = __expf(t);
        et = e * t;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        e += __shfl_xor_sync(kFullMask, e, off);
        et += __shfl_xor_sync(kFullMask, et, off);
    }
    st.merge(M, e, et);
    // ranks among the block's candidates and the ten values kept so far (which win ties)
    const float old_v = top_v;  // lanes >= 10 hold -inf
    int rank_new = 0, rank_old = lane;
#pragma unroll 8
    for (int k = 0; k < 32; ++k) {
        const float vk = __shfl_sync(kFullMask, val, k);
        rank_new += (vk > val) || (vk == val && k < lane);
        rank_old += vk > old_v;
    }
#pragma unroll
    for (int k = 0; k < kTopK; ++k) {
        const float ok = __shfl_sync(kFullMask, old_v, k);
        rank_new += ok >= val;
    }
    if (lane < kTopK) scratch[lane] = DISCO_NEG_INF;  // positions nobody claims stay empty
    __syncwarp();
    if (lane < n && rank_new < kTopK) scratch[rank_new] = val;
    if (lane < kTopK && old_v > DISCO_NEG_INF && rank_old < kTopK) scratch[rank_old] = old_v;
    __syncwarp();
    top_v = lane < kTopK ? scratch[lane] : DISCO_NEG_INF;
    __syncwarp();
}

// Ten largest values seen so far, descending, in the registers of one thread.
struct RegTop10 {
    float t[kTopK];
    __device__ __forceinline__ void init() {
#pragma unroll
        for (int k = 0; k < kTopK; ++k) t[k] = DISCO_NEG_INF;
    }
    __device__ __forceinline__ void push(float z) {
        float carry = z;
#pragma unroll
        for (int k = 0; k < kTopK; ++k) {
            const float hi = fmaxf(t[k], carry);
            carry = fminf(t[k], carry);
            t[k] = hi;
        }
    }
    // Two values at once.  With a >= b the (k+1)-th largest of the list and {a, b} is
    //     max(t[k], min(t[k-1], a), min(t[k-2], b))          (t[-1] = t[-2] = +inf),
    // the merge rule of two descending lists: three min/max per slot for two values instead of four, no
    // carry chain, and the outer maximum is one three-input instruction.
    __device__ __forceinline__ void push2(float z0, float z1) {
        const float a = fmaxf(z0, z1), b = fminf(z0, z1);
#pragma unroll
        for (int k = kTopK - 1; k >= 2; --k) t[k] = max3(t[k], fminf(t[k - 1], a), fminf(t[k - 2], b));
        t[1] = max3(t[1], fminf(t[0], a), b);
        t[0] = fmaxf(t[0], a);
    }
    // Merge with another descending list of ten: both lists laid end to end, the other one reversed, fall
    // then rise (a bitonic sequence of 32 with -inf in the middle); the half-cleaner of distance 16 leaves the 16
    // largest in 16 slots, four of them by a comparison and the rest by position, and four more distances sort
    // them.  A chain of five min/max instead of the hundred of ten insertions; what only feeds slots 10 .. 15 of
    // the result is dead code.
    __device__ __forceinline__ void merge(const float (&o)[kTopK]) {
        static_assert(kTopK == 10, "the network below is written for lists of ten");
        float L[16];
#pragma unroll
        for (int i = 0; i < 6; ++i) L[i] = t[i];
        L[6] = fmaxf(t[6], o[9]);
        L[7] = fmaxf(t[7], o[8]);
        L[8] = fmaxf(t[8], o[7]);
        L[9] = fmaxf(t[9], o[6]);
#pragma unroll
        for (int i = 10; i < 16; ++i) L[i] = o[15 - i];
#pragma unroll
        for (int s = 8; s >= 1; s >>= 1) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                if ((i & s) == 0) {
                    const float hi = fmaxf(L[i], L[i + s]), lo = fminf(L[i], L[i + s]);
                    L[i] = hi;
                    L[i + s] = lo;
                }
            }
        }
#pragma unroll
        for (int k = 0; k < kTopK; ++k) t[k] = L[k];
    }
    static __device__ __forceinline__ float max3(float x, float y, float z) {
        float d;
        asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(x), "f"(y), "f"(z));
        return d;
    }
};

}  // namespace disco
