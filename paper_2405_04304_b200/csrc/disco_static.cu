// disco_draft_step_static: the draft step for callers that cannot allocate device memory.
//
// The regular entry points take their scratch (per-CTA partial results, a ticket counter, a status
// word) from a context that disco_create allocates with cudaMalloc.  Some hosts of this library are
// not allowed to do that: a serving process whose device memory is carved up and capped by another
// component that hands out no allocator, or a decode loop that cannot afford the device-wide
// synchronisation a cudaMalloc may imply.  For them this file keeps the scratch in a fixed-size
// __device__ array that is part of the library image: every GPU that loads the library holds those
// bytes until the process exits, and nothing here calls cudaMalloc, cudaFree or any allocating routine.
//
// The kernel is the same CUDA-core streaming kernel the context-based call uses for a handful of
// sequences; only where its scratch lives differs.
#include <cuda_runtime.h>

#include <algorithm>
#include <mutex>

#include "disco.h"
#include "stream_tail.cuh"

using namespace disco;

namespace {

constexpr int kWarps = 16;
constexpr int kMaxB = DISCO_STATIC_MAX_BATCH;
constexpr int kMaxGrid = DISCO_STATIC_MAX_GRID;
constexpr size_t kHeadBytes = 256;  // ticket @0, status @64, final (m, Z) per sequence @128
constexpr size_t kRecordBytes = (size_t)kMaxB * kMaxGrid * 64;  // one 64-byte partial record per (sequence, CTA)
constexpr size_t kScratchBytes = kHeadBytes + kRecordBytes;

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress; it is NOT a
// device address and must never be handed to a kernel as one.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
struct DeviceSetup {
    bool ready;
    unsigned char* scratch;  // device address of g_static_scratch on this device
    int sm_count;
    size_t smem_optin;
    size_t dyn_limit[3];
};
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mu;   // first calls from several host threads take turns at the set-up

template <int RT, int KC>
bool configure(DeviceSetup& s, int slot) {
    auto kern = stream_tail_kernel<RT, true, kWarps, KC>;
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, kern) != cudaSuccess) return false;
    const size_t limit = s.smem_optin - fa.sharedSizeBytes;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)limit) != cudaSuccess)
        return false;
    s.dyn_limit[slot] = std::min(s.dyn_limit[slot], limit);   // the slot starts at the device's opt-in maximum
    return true;
}

// Once per device, with that device current: resolve the device address of the scratch array and
// raise the shared-memory limit of the kernels.
int setup_device(int dev) {
    std::lock_guard<std::mutex> lock(g_setup_mu);
    DeviceSetup& s = g_setup[dev];
    if (s.ready) return DISCO_OK;
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return DISCO_ERR_CUDA;
    int sm = 0, optin = 0;
    if (cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
        return DISCO_ERR_CUDA;
    s.scratch = static_cast<unsigned char*>(ptr);
    s.sm_count = sm;
    s.smem_optin = (size_t)optin;
    s.dyn_limit[0] = s.dyn_limit[1] = s.dyn_limit[2] = s.smem_optin;
    bool ok = configure<1, 3>(s, 0) && configure<1, 4>(s, 0) && configure<1, 0>(s, 0);
    s.dyn_limit[1] = s.smem_optin;
    ok = ok && configure<2, 0>(s, 1);
    s.dyn_limit[2] = s.smem_optin;
    ok = ok && configure<4, 0>(s, 2);
    if (!ok) return DISCO_ERR_CUDA;
    s.ready = true;
    return DISCO_OK;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" int disco_draft_step_static(int V, int d_draft, const void* W_D, const void* h_D, int B,
                                       const int32_t* pos, const int32_t* n_drafted, const uint8_t* active,
                                       const disco_clf* clf, float tau, int sl_max, int32_t* token, float* conf,
                                       uint8_t* halt, float* feats, void* stream) {
    if (!W_D || !h_D || !pos || !n_drafted || !token || !conf || !halt || !clf) return DISCO_ERR_INVALID_ARG;
    if (!clf->W1 || !clf->b1 || !clf->w2 || !clf->b2 || clf->H < 1 || clf->H > DISCO_MAX_CLF_HIDDEN)
        return DISCO_ERR_INVALID_ARG;
    if (!aligned16(W_D) || !aligned16(h_D)) return DISCO_ERR_INVALID_ARG;
    if (V < 1 || d_draft < 8 || (d_draft % 8) || B < 1 || sl_max < 1) return DISCO_ERR_INVALID_ARG;
    if (d_draft > 16384) return DISCO_ERR_UNSUPPORTED_SHAPE;
    if (B > kMaxB) return DISCO_ERR_STATIC_LIMIT;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return DISCO_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return DISCO_ERR_STATIC_LIMIT;
    int rc = setup_device(dev);
    if (rc) return rc;
    const DeviceSetup& s = g_setup[dev];
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    // launch geometry: one CTA per slab of vocabulary rows, slots of about 6 KB in the shared-memory ring
    const int RT = B == 1 ? 1 : (B == 2 ? 2 : 4);
    const uint32_t row_bytes = (uint32_t)d_draft * 2u;
    const int rpc = std::max(1, std::min((V + s.sm_count - 1) / s.sm_count, 2048));
    const int grid = (V + rpc - 1) / rpc;
    if (grid > kMaxGrid) return DISCO_ERR_STATIC_LIMIT;
    const int rps = std::min(std::max(1, 6144 / (int)row_bytes), rpc);
    const uint32_t slot_bytes = (uint32_t)rps * row_bytes;
    const size_t fixed = stream_tail_smem_bytes(RT, kWarps, d_draft, 0, 0, clf->H);
    const size_t limit = s.dyn_limit[RT == 1 ? 0 : (RT == 2 ? 1 : 2)];
    if (limit <= fixed + 2048) return DISCO_ERR_UNSUPPORTED_SHAPE;
    long long stages = (long long)((limit - 2048 - fixed) / (slot_bytes + 16));
    stages = std::min<long long>(stages, 2 * kWarps);
    if (stages > kWarps) stages -= stages % kWarps;
    if (stages < 2) return DISCO_ERR_UNSUPPORTED_SHAPE;
    const size_t smem = stream_tail_smem_bytes(RT, kWarps, d_draft, (int)stages, slot_bytes, clf->H);

    TailParams p{};
    p.W = static_cast<const uint16_t*>(W_D);
    p.H = static_cast<const uint16_t*>(h_D);
    p.V = V;
    p.d = d_draft;
    p.R = B;
    p.B = B;
    p.rows_per_cta = rpc;
    p.rps = rps;
    p.stages = (int)stages;
    p.slot_bytes = slot_bytes;
    p.ticket = reinterpret_cast<unsigned int*>(s.scratch);
    p.status = reinterpret_cast<int*>(s.scratch + 64);
    p.final_stats = reinterpret_cast<float*>(s.scratch + 128);
    p.part_rec = reinterpret_cast<float4*>(s.scratch + kHeadBytes);
    p.keys = nullptr;
    p.pos = pos;
    p.n_drafted = n_drafted;
    p.active = active;
    p.clf_W1 = clf->W1;
    p.clf_b1 = clf->b1;
    p.clf_w2 = clf->w2;
    p.clf_b2 = clf->b2;
    p.clf_H = clf->H;
    p.tau = tau;
    p.sl_max = sl_max;
    p.token = token;
    p.conf = conf;
    p.halt = halt;
    p.feats = feats;
    p.probs = nullptr;

    // The array keeps whatever the previous call left.  The ticket has to start at zero; the partial
    // results are fully rewritten by every call before they are read.
    if (cudaMemsetAsync(s.scratch, 0, 128, st) != cudaSuccess) return DISCO_ERR_CUDA;
    const dim3 block((kWarps + 1) * 32);
    if (RT == 1) {
        if (d_draft <= 768) stream_tail_kernel<1, true, kWarps, 3><<<grid, block, smem, st>>>(p);
        else if (d_draft <= 1024) stream_tail_kernel<1, true, kWarps, 4><<<grid, block, smem, st>>>(p);
        else stream_tail_kernel<1, true, kWarps, 0><<<grid, block, smem, st>>>(p);
    } else if (RT == 2) {
        stream_tail_kernel<2, true, kWarps, 0><<<grid, block, smem, st>>>(p);
    } else {
        stream_tail_kernel<4, true, kWarps, 0><<<grid, block, smem, st>>>(p);
    }
    return cudaGetLastError() == cudaSuccess ? DISCO_OK : DISCO_ERR_CUDA;
}
