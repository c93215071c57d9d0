// Host side of the C ABI declared in include/disco.h: context, argument checks, kernel selection
// and launches.  No PyTorch types; plain pointers and sizes only.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>

#include "disco.h"
#include "stream_tail.cuh"
#include "umma_tail.cuh"
#include "sample.cuh"
#include "umma_gemv.cuh"
#include "umma_gemv_loop.cuh"

using namespace disco;

namespace {

constexpr int kStreamWarps = 16;     // consumer warps of the streaming kernel
constexpr int kMaxHidden = 16384;    // widest hidden dimension the kernels accept
constexpr int kSlotTargetBytes = 6144;

constexpr int kMaxDevices = 64;

// One-time, per-device configuration of one kernel (its dynamic shared-memory limit).  Every template
// instance of a launcher owns one of these; the lock makes first calls from several host threads, and
// contexts on several devices, safe.
struct KernelSetup {
    std::mutex mu;
    bool done[kMaxDevices] = {};
    size_t dyn_limit[kMaxDevices] = {};
};

struct StreamPlan {
    int rows_per_cta, grid, rps, stages;
    uint32_t slot_bytes;
    size_t smem;
    bool ok;
};

}  // namespace

struct disco_ctx {
    int device;
    int V, d_draft, d_target, max_batch, max_rows, clf_hidden;
    int sm_count;
    size_t smem_optin;
    int path;
    int pdl;  // launch the streaming kernel with programmatic stream serialization (DISCO_PDL=0 turns it off)
    long long launches;
    cudaStream_t last_stream;  // stream of the most recent enqueue (disco_last_device_status waits for it only)
    unsigned int test_stamp_skew;  // disco_test_hooks
    // scratch for cross-block reductions
    int part_rows;  // rows the partial buffers can hold
    int max_grid;
    unsigned long long* keys;
    unsigned int* ticket;
    int* status;
    float* final_stats;
    uint8_t* chain_alive;          // [max_batch] draft phase on the device: which sequences still draft
    double* sample_seg_tot;        // verification with sampling: [max_batch][kSampleMaxSegments][2] sums of weights
    int32_t* sample_seg_last;      //   the same shape: last index with positive weight
    unsigned int* sample_tickets;  //   [max_batch]
    void* pack_rows;               // fixed-shape verification with many rows: the rows that count, packed
    int32_t* pack_off;             // [max_batch + 1] their offsets; the last entry is the row count
    void* loop_rec;                // persistent draft-phase kernel: stamped 80-byte records, [4][CTA]; written by nothing else
    void* part_rec;                // draft step: 64-byte partial records, [sequence][CTA]
    void* stamped_rec;             // batched draft step: stamped 80-byte records, [sequence][CTA]; written by nothing else
    int part_slots;                // partials per row the buffers can hold
    void* encode_tiled;            // cuTensorMapEncodeTiled, resolved through the runtime
    // device staging for the *_host entry points
    void* stage_hidden;
    void* stage_hidden_draft;      // disco_iteration_host: the draft hidden states of all steps
    cudaStream_t copy_stream;      // disco_iteration_host: the target hidden states travel beside the draft phase
    cudaEvent_t copy_done;
    // Small inputs and outputs of the *_host entry points live in pinned host memory that the GPU maps:
    // the kernels read and write it in place, so a host call costs one copy (the hidden states), one
    // launch and one synchronisation.  *_h: host address, *_d: the same memory as the device sees it.
    int32_t *stage_int_h, *stage_int_d;    // pos | n_drafted | token | draft_ids | row_off | n_accept | bonus | target_ids
    float *stage_float_h, *stage_float_d;  // conf | feats
    uint8_t *stage_byte_h, *stage_byte_d;  // active | halt
};

namespace {

// With DISCO_DEBUG set in the environment, failed CUDA runtime calls are reported on stderr.
inline bool cuda_ok(cudaError_t e, const char* what) {
    if (e == cudaSuccess) return true;
    static const bool verbose = std::getenv("DISCO_DEBUG") != nullptr;
    if (verbose) std::fprintf(stderr, "[disco] %s: %s\n", what, cudaGetErrorString(e));
    return false;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Raise a kernel's dynamic shared-memory limit once per device: to `bytes`, or (bytes == 0) to all that the
// device allows beside the kernel's static shared memory.  *limit receives the value in force.
template <typename Kern>
bool raise_smem_limit(const disco_ctx* c, KernelSetup& ks, Kern kern, size_t bytes, size_t* limit) {
    if (c->device < 0 || c->device >= kMaxDevices) return false;
    std::lock_guard<std::mutex> lock(ks.mu);
    if (!ks.done[c->device]) {
        size_t want = bytes;
        if (want == 0) {
            cudaFuncAttributes fa;
            if (!cuda_ok(cudaFuncGetAttributes(&fa, kern), "cudaFuncGetAttributes")) return false;
            want = c->smem_optin - fa.sharedSizeBytes;
        }
        if (!cuda_ok(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)want),
                     "cudaFuncSetAttribute"))
            return false;
        ks.dyn_limit[c->device] = want;
        ks.done[c->device] = true;
    }
    if (limit) *limit = ks.dyn_limit[c->device];
    return true;
}

StreamPlan plan_stream(const disco_ctx* c, int V, int d, int RT, int clf_H) {
    StreamPlan pl{};
    const uint32_t row_bytes = (uint32_t)d * 2u;
    int rpc = (V + c->sm_count - 1) / c->sm_count;
    rpc = std::max(1, std::min(rpc, 2048));
    pl.rows_per_cta = rpc;
    pl.grid = (V + rpc - 1) / rpc;
    int rps = std::max(1, kSlotTargetBytes / (int)row_bytes);
    rps = std::min(rps, rpc);
    pl.rps = rps;
    pl.slot_bytes = (uint32_t)rps * row_bytes;
    const size_t fixed = stream_tail_smem_bytes(RT, kStreamWarps, d, 0, 0, clf_H);
    const size_t budget = c->smem_optin > 2048 ? c->smem_optin - 2048 : 0;
    if (budget <= fixed) return pl;
    long long stages = (long long)((budget - fixed) / (pl.slot_bytes + 16));
    stages = std::min<long long>(stages, 2 * kStreamWarps);
    if (stages > kStreamWarps) stages -= stages % kStreamWarps;  // slots are dealt round-robin to the warps
    if (stages < 2) return pl;
    pl.stages = (int)stages;
    pl.smem = stream_tail_smem_bytes(RT, kStreamWarps, d, pl.stages, pl.slot_bytes, clf_H);
    pl.ok = true;
    return pl;
}

template <int RT, bool DRAFT, int KC>
int launch_stream(disco_ctx* c, TailParams& p, const StreamPlan& pl, cudaStream_t st) {
    auto kern = stream_tail_kernel<RT, DRAFT, kStreamWarps, KC>;
    static KernelSetup setup;
    size_t dyn_limit = 0;
    if (!raise_smem_limit(c, setup, kern, 0, &dyn_limit)) return DISCO_ERR_CUDA;
    if (pl.smem > dyn_limit) return DISCO_ERR_UNSUPPORTED_SHAPE;
    // Programmatic dependent launch: the kernel may start while the preceding kernel of the stream is
    // still in its tail; it streams the LM head (never written by this library) and waits with
    // griddepcontrol.wait before it touches anything else.
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)pl.grid);
    cfg.blockDim = dim3((kStreamWarps + 1) * 32);
    cfg.dynamicSmemBytes = pl.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = c->pdl ? 1 : 0;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, p);
    c->launches += 1;
    return cuda_ok(e, "stream_tail_kernel launch") ? DISCO_OK : DISCO_ERR_CUDA;
}

template <bool DRAFT>
int run_stream(disco_ctx* c, TailParams& p, int clf_H, cudaStream_t st) {
    const int RT = p.R == 1 ? 1 : (p.R == 2 ? 2 : 4);
    const StreamPlan pl = plan_stream(c, p.V, p.d, RT, clf_H);
    if (!pl.ok) return DISCO_ERR_UNSUPPORTED_SHAPE;
    if (DRAFT && (pl.grid > c->max_grid || p.R > c->part_rows)) return DISCO_ERR_WORKSPACE;
    p.rows_per_cta = pl.rows_per_cta;
    p.slab_rows = pl.rows_per_cta;
    p.rps = pl.rps;
    p.stages = pl.stages;
    p.slot_bytes = pl.slot_bytes;
    switch (RT) {
        case 1:  // one hidden row: the warp can hold its share of h in registers (32 * 8 * KC values)
            if (p.d <= 768) return launch_stream<1, DRAFT, 3>(c, p, pl, st);
            if (p.d <= 1024) return launch_stream<1, DRAFT, 4>(c, p, pl, st);
            return launch_stream<1, DRAFT, 0>(c, p, pl, st);
        case 2: return launch_stream<2, DRAFT, 0>(c, p, pl, st);
        default: return launch_stream<4, DRAFT, 0>(c, p, pl, st);
    }
}


// ------------------------------------------------------------------------------------------------
// tcgen05 path
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// bf16 [rows, d] row-major, boxes of box_rows x 64 elements, 128-byte swizzle, zero fill out of bounds
bool encode_bf16_2d(const disco_ctx* c, CUtensorMap* map, const void* base, int rows, int d, int box_rows) {
    if (!c->encode_tiled) return false;
    const cuuint64_t gdim[2] = {(cuuint64_t)d, (cuuint64_t)rows};
    const cuuint64_t gstride[1] = {(cuuint64_t)d * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kUmmaBK, (cuuint32_t)box_rows};
    const cuuint32_t estride[2] = {1, 1};
    const CUresult r = reinterpret_cast<EncodeTiledFn>(c->encode_tiled)(
        map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estride,
        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool umma_possible(const disco_ctx* c, int R) {
    const int MT = (R + 127) / 128;
    return c->encode_tiled != nullptr && MT <= c->sm_count;
}

// Launch the tcgen05 kernel for R hidden rows of width d against the LM head W [V, d].
template <bool DRAFT, bool STATS = false>
int launch_umma(disco_ctx* c, const void* W, const void* H, int d, int R, float* probs,
                const DraftFinalParams* draft_final, const UmmaParams* fused, cudaStream_t st,
                const int32_t* dev_R = nullptr) {
    UmmaParams p{};
    if (fused) p = *fused;  // verification finished by the main kernel's last CTA
    p.V = c->V;
    p.d = d;
    p.R = R;
    p.MT = (R + 127) / 128;
    p.CN = c->sm_count / p.MT;
    // Vocabulary rows per tile: up to 256 for verification (its epilogue is a compare per logit); the
    // draft step's epilogue is heavy (soft-max, top-10), so it gets several small tiles per CTA and
    // the epilogue of one tile runs under the loads of the next.
    const int tile_target = (DRAFT && !STATS) ? (R <= 128 ? 128 : 256) : 256;
    p.TPC = std::max(1, (c->V + tile_target * p.CN - 1) / (tile_target * p.CN));
    p.TR = (c->V + p.CN * p.TPC - 1) / (p.CN * p.TPC);
    p.TRN = std::max(16, (p.TR + 15) / 16 * 16);
    p.dev_R = dev_R;
    if (dev_R) p.TRN = 256;   // the kernel derives the tiling from the device-side row count; the box is the largest tile
    p.a_rows = p.MT > 1 ? 128 : std::max(8, (R + 7) / 8 * 8);
    // Draft step with few rows: copies of the rows fill the other TMEM lane quadrants, so that the
    // epilogue (heavy there) runs on every warp scheduler.  Verification's epilogue is a compare per
    // logit and keeps the smaller stage instead.
    p.rep = (DRAFT && !STATS && R <= 64) ? (R <= 32 ? 4 : 2) : 1;   // (measured: no gain for the statistics-only epilogue)
    p.rows_pad = 128 / p.rep;
    // The A stage holds a_rows rows (rep copies, rows_pad rows apart).  The MMA still reads 128 rows from
    // its start: what lies behind the tile (other stages of the ring, always inside it) or between the
    // copies only feeds accumulator lanes nobody reads.
    p.a_bytes = p.rep > 1 ? 128 * 128 : (p.a_rows * 128 + 1023) / 1024 * 1024;
    p.b_bytes = (p.TRN * 128 + 1023) / 1024 * 1024;
    // (the draft step's epilogue keeps its candidate queues in the last bytes of the ring)
    const int ring_bytes = kUmmaRingBytes - ((DRAFT && !STATS) ? kUmmaQueueBytes : 0);
    p.stages = std::max(2, std::min(kUmmaMaxStages, ring_bytes / (p.a_bytes + p.b_bytes)));
    p.status = c->status;
    p.keys = c->keys;
    p.part_rec = reinterpret_cast<float4*>(c->stamped_rec);
    p.probs = probs;
    if (DRAFT && ((size_t)R * p.CN > (size_t)128 * c->sm_count || R > c->part_rows)) return DISCO_ERR_WORKSPACE;
    CUtensorMap tmap_W, tmap_H;
    if (!encode_bf16_2d(c, &tmap_W, W, c->V, d, p.TRN) || !encode_bf16_2d(c, &tmap_H, H, R, d, p.a_rows))
        return DISCO_ERR_CUDA;
    auto kern = umma_tail_kernel<DRAFT, STATS>;
    static KernelSetup setup;
    if (!raise_smem_limit(c, setup, kern, (size_t)kUmmaSmemBytes + umma_clf_bytes(DISCO_MAX_CLF_HIDDEN), nullptr))
        return DISCO_ERR_CUDA;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(dev_R ? c->sm_count : p.MT * p.CN));
    cfg.blockDim = dim3(kUmmaThreads);
    cfg.dynamicSmemBytes = kUmmaSmemBytes + (draft_final ? umma_clf_bytes(draft_final->clf_H) : 0);
    cfg.stream = st;
    // The draft step's second phase waits for every CTA of the grid: a cooperative launch makes the
    // driver refuse the launch unless all of them can be resident at once.
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (DRAFT) {
        attr[na].id = cudaLaunchAttributeCooperative;
        attr[na].val.cooperative = 1;
        ++na;
    }
    if (c->pdl) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    const DraftFinalParams f = draft_final ? *draft_final : DraftFinalParams{};
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tmap_W, tmap_H, p, f);
    c->launches += 1;
    return cuda_ok(e, "umma_tail_kernel launch") ? DISCO_OK : DISCO_ERR_CUDA;
}


// Launch the tensor-core GEMV-shaped draft step (1..16 sequences).
template <int RK>
int launch_gemv_rk(disco_ctx* c, GemvParams& g, const CUtensorMap& mW, const CUtensorMap& mH, cudaStream_t st) {
    auto kern = umma_gemv_draft_kernel<RK>;
    static KernelSetup setup;
    size_t dyn_limit = 0;
    if (!raise_smem_limit(c, setup, kern, 0, &dyn_limit)) return DISCO_ERR_CUDA;
    // the ring takes what the fixed part leaves; it must hold at least two stages and the 16 KB that the
    // MMA reads behind the last box of hidden rows
    const size_t fixed = gemv_fixed_smem_bytes(RK, g.t.clf_H, g.t.d, g.h_rows);
    if (dyn_limit < fixed + 2 * (size_t)g.b_bytes) return DISCO_ERR_UNSUPPORTED_SHAPE;
    g.stages = (int)std::min<size_t>(kGemvMaxStages, (dyn_limit - fixed) / g.b_bytes);
    if ((size_t)g.stages * g.b_bytes < 16384) return DISCO_ERR_UNSUPPORTED_SHAPE;
    const size_t smem = gemv_smem_bytes(RK, g.t.clf_H, g.t.d, g.h_rows, g.stages, g.b_bytes);
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)c->sm_count);
    cfg.blockDim = dim3(kGemvThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = c->pdl ? 1 : 0;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, mW, mH, g);
    c->launches += 1;
    return cuda_ok(e, "umma_gemv_draft_kernel launch") ? DISCO_OK : DISCO_ERR_CUDA;
}

int launch_gemv(disco_ctx* c, const TailParams& t, cudaStream_t st) {
    GemvParams g{};
    g.t = t;
    const int grid = c->sm_count;
    if (grid > c->part_slots || t.R > c->part_rows) return DISCO_ERR_WORKSPACE;
    g.TR = (t.V + grid - 1) / grid;
    g.t.slab_rows = g.TR;
    g.tiles = (g.TR + 255) / 256;
    g.TRt = (g.TR + g.tiles - 1) / g.tiles;
    g.TRN = (g.TRt + 15) / 16 * 16;
    g.b_bytes = (g.TRN * 128 + 1023) / 1024 * 1024;
    g.h_rows = t.R <= 8 ? 8 : 16;
    CUtensorMap mW, mH;
    if (!encode_bf16_2d(c, &mW, t.W, t.V, t.d, g.TRN) || !encode_bf16_2d(c, &mH, t.H, t.R, t.d, g.h_rows))
        return DISCO_ERR_CUDA;
    if (t.R == 1) return launch_gemv_rk<1>(c, g, mW, mH, st);
    if (t.R == 2) return launch_gemv_rk<2>(c, g, mW, mH, st);
    if (t.R <= 4) return launch_gemv_rk<4>(c, g, mW, mH, st);
    if (t.R <= 8) return launch_gemv_rk<8>(c, g, mW, mH, st);
    return launch_gemv_rk<16>(c, g, mW, mH, st);
}

// The draft phase as one persistent kernel (1..4 sequences): see umma_gemv_loop.cuh.
template <int RK>
int launch_gemv_loop_rk(disco_ctx* c, GemvLoopParams& lp, const CUtensorMap& mW, const CUtensorMap& mH, cudaStream_t st) {
    auto kern = umma_gemv_loop_kernel<RK>;
    static KernelSetup setup;
    size_t dyn_limit = 0;
    if (!raise_smem_limit(c, setup, kern, 0, &dyn_limit)) return DISCO_ERR_CUDA;
    GemvParams& g = lp.g;
    const size_t fixed = gemv_loop_fixed_smem_bytes(RK, g.t.clf_H, g.t.d, g.h_rows);
    if (dyn_limit < fixed + 2 * (size_t)g.b_bytes) return DISCO_ERR_UNSUPPORTED_SHAPE;
    g.stages = (int)std::min<size_t>(kGemvMaxStages, (dyn_limit - fixed) / g.b_bytes);
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)c->sm_count);
    cfg.blockDim = dim3(kGemvThreads);
    cfg.dynamicSmemBytes = fixed + (size_t)g.stages * g.b_bytes;
    cfg.stream = st;
    // the steps hand over through global memory: every CTA has to be running, which a cooperative launch checks
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = c->pdl ? 2 : 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, mW, mH, lp);
    c->launches += 1;
    return cuda_ok(e, "umma_gemv_loop_kernel launch") ? DISCO_OK : DISCO_ERR_CUDA;
}

bool gemv_loop_possible(const disco_ctx* c, int B, int sl_max, size_t w_step_stride) {
    if (!c->encode_tiled || B > 4 || sl_max > kLoopMaxSteps) return false;
    if (c->path != 0 && c->path != 3) return false;
    if (w_step_stride != 0 && w_step_stride != (size_t)c->V * c->d_draft * 2) return false;   // one tensor map over all copies
    if ((long long)c->V * sl_max > 0x7fffffffll) return false;
    return (size_t)((c->d_draft + kUmmaBK - 1) / kUmmaBK) * 8 * 128 <= 48 * 1024;
}

int launch_gemv_loop(disco_ctx* c, const TailParams& t, int steps, size_t w_step_stride, cudaStream_t st) {
    GemvLoopParams lp{};
    GemvParams& g = lp.g;
    g.t = t;
    const int grid = c->sm_count;
    if (grid > kGroupMaxRecords) return DISCO_ERR_UNSUPPORTED_SHAPE;
    g.TR = (t.V + grid - 1) / grid;
    g.t.slab_rows = g.TR;
    g.tiles = (g.TR + 255) / 256;
    g.TRt = (g.TR + g.tiles - 1) / g.tiles;
    g.TRN = (g.TRt + 15) / 16 * 16;
    g.b_bytes = (g.TRN * 128 + 1023) / 1024 * 1024;
    g.h_rows = 8;
    lp.steps = steps;
    lp.w_rows_per_step = w_step_stride ? t.V : 0;
    lp.flags = c->ticket + 64;
    lp.epoch = c->ticket + 128;
    lp.records = reinterpret_cast<float4*>(c->loop_rec);
    CUtensorMap mW, mH;
    if (!encode_bf16_2d(c, &mW, t.W, t.V * (w_step_stride ? steps : 1), t.d, g.TRN) ||
        !encode_bf16_2d(c, &mH, t.H, t.R * steps, t.d, g.h_rows))
        return DISCO_ERR_CUDA;
    if (t.R == 1) return launch_gemv_loop_rk<1>(c, lp, mW, mH, st);
    if (t.R == 2) return launch_gemv_loop_rk<2>(c, lp, mW, mH, st);
    return launch_gemv_loop_rk<4>(c, lp, mW, mH, st);
}

void fill_scratch(const disco_ctx* c, TailParams& p) {
    p.part_rec = reinterpret_cast<float4*>(c->part_rec);
    p.keys = c->keys;
    p.ticket = c->ticket;
    p.status = c->status;
    p.final_stats = c->final_stats;
}

int check_clf(const disco_ctx* c, const disco_clf* clf) {
    if (!clf || !clf->W1 || !clf->b1 || !clf->w2 || !clf->b2) return DISCO_ERR_INVALID_ARG;
    if (clf->H < 1 || clf->H > DISCO_MAX_CLF_HIDDEN) return DISCO_ERR_INVALID_ARG;
    if (clf->H > c->clf_hidden) return DISCO_ERR_WORKSPACE;
    return DISCO_OK;
}

}  // namespace

extern "C" {

const char* disco_strerror(int code) {
    switch (code) {
        case DISCO_OK: return "ok";
        case DISCO_ERR_INVALID_ARG: return "invalid argument (null or misaligned pointer, size out of range)";
        case DISCO_ERR_UNSUPPORTED_SHAPE: return "shape not supported by the kernels";
        case DISCO_ERR_WORKSPACE: return "batch, rows or classifier width beyond what the context was created for";
        case DISCO_ERR_CUDA: return "a CUDA runtime call failed";
        case DISCO_ERR_TIMEOUT: return "a bounded device-side wait ran out";
        case DISCO_ERR_STATIC_LIMIT: return "size beyond the fixed scratch of the allocation-free entry point";
        default: return "unknown disco status";
    }
}

int disco_create(disco_ctx** out, int V, int d_draft, int d_target, int max_batch, int max_rows, int k,
                 int clf_hidden) {
    if (!out) return DISCO_ERR_INVALID_ARG;
    if (V < 1 || d_draft < 8 || d_target < 8 || (d_draft % 8) || (d_target % 8)) return DISCO_ERR_INVALID_ARG;
    if (max_batch < 1 || max_rows < 1 || k != DISCO_TOPK) return DISCO_ERR_INVALID_ARG;
    if (clf_hidden < 1 || clf_hidden > DISCO_MAX_CLF_HIDDEN) return DISCO_ERR_INVALID_ARG;
    if (d_draft > kMaxHidden || d_target > kMaxHidden) return DISCO_ERR_UNSUPPORTED_SHAPE;

    disco_ctx* c = new (std::nothrow) disco_ctx();
    if (!c) return DISCO_ERR_CUDA;
    std::memset(c, 0, sizeof(*c));
    cudaDeviceProp prop;
    if (cudaGetDevice(&c->device) != cudaSuccess || cudaGetDeviceProperties(&prop, c->device) != cudaSuccess) {
        delete c;
        return DISCO_ERR_CUDA;
    }
    c->V = V;
    c->d_draft = d_draft;
    c->d_target = d_target;
    c->max_batch = max_batch;
    c->max_rows = max_rows;
    c->clf_hidden = clf_hidden;
    {
        const char* e = std::getenv("DISCO_PDL");
        c->pdl = !(e && e[0] == '0');
    }
    c->sm_count = prop.multiProcessorCount;
    c->smem_optin = prop.sharedMemPerBlockOptin;

    const int rpc = std::max(1, std::min((V + c->sm_count - 1) / c->sm_count, 2048));
    c->max_grid = (V + rpc - 1) / rpc;
    c->part_rows = std::max(max_batch, max_rows);  // the target rows of a verification with sampling go the same way
    c->part_slots = std::max(c->max_grid, 2 * c->sm_count);
    const size_t slots = (size_t)c->part_rows * c->part_slots;
    {
        cudaDriverEntryPointQueryResult qres;
        void* fn = nullptr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            c->encode_tiled = fn;
    }
    // the largest layout is disco_iteration_host's: 6 arrays of max_batch words and 2 of max_rows
    const size_t n_int = (size_t)8 * max_batch + (size_t)3 * max_rows + 64;
    const size_t hid = std::max((size_t)max_batch * d_draft, (size_t)max_rows * d_target) * 2;
    bool ok = true;
    ok = ok && cudaMalloc(&c->keys, (size_t)max_rows * sizeof(unsigned long long)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->part_rec, slots * 64) == cudaSuccess;
    ok = ok && cudaMalloc(&c->ticket, 1024) == cudaSuccess;
    ok = ok && cudaMalloc(&c->status, 256) == cudaSuccess;
    ok = ok && cudaMalloc(&c->final_stats, (size_t)c->part_rows * 2 * sizeof(float)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->chain_alive, (size_t)max_batch + 64) == cudaSuccess;
    ok = ok && cudaMalloc(&c->sample_seg_tot, (size_t)max_batch * kSampleMaxSegments * 2 * sizeof(double)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->sample_seg_last, (size_t)max_batch * kSampleMaxSegments * 2 * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->sample_tickets, (size_t)max_batch * sizeof(unsigned int)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->pack_rows, (size_t)max_rows * d_target * 2) == cudaSuccess;
    ok = ok && cudaMalloc(&c->pack_off, ((size_t)max_batch + 2) * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&c->loop_rec, (size_t)4 * c->sm_count * 80) == cudaSuccess;
    ok = ok && cudaMemset(c->loop_rec, 0, (size_t)4 * c->sm_count * 80) == cudaSuccess;   // no stamp yet
    ok = ok && cudaMalloc(&c->stage_hidden, hid) == cudaSuccess;
    ok = ok && cudaMalloc(&c->stage_hidden_draft, (size_t)max_rows * d_draft * 2) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&c->copy_done, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaHostAlloc(&c->stage_int_h, n_int * sizeof(int32_t), cudaHostAllocMapped) == cudaSuccess;
    ok = ok && cudaHostAlloc(&c->stage_float_h, ((size_t)max_batch * (1 + kNFeat) + max_rows) * sizeof(float), cudaHostAllocMapped) == cudaSuccess;
    ok = ok && cudaHostAlloc(&c->stage_byte_h, (size_t)max_batch * 2 + max_rows + 64, cudaHostAllocMapped) == cudaSuccess;
    ok = ok && cudaHostGetDevicePointer(&c->stage_int_d, c->stage_int_h, 0) == cudaSuccess;
    ok = ok && cudaHostGetDevicePointer(&c->stage_float_d, c->stage_float_h, 0) == cudaSuccess;
    ok = ok && cudaHostGetDevicePointer(&c->stage_byte_d, c->stage_byte_h, 0) == cudaSuccess;
    ok = ok && cudaMemset(c->keys, 0, (size_t)max_rows * sizeof(unsigned long long)) == cudaSuccess;
    ok = ok && cudaMemset(c->ticket, 0, 1024) == cudaSuccess;
    // R rows take R * (sm_count / ceil(R / 128)) <= 128 * sm_count records
    ok = ok && cudaMalloc(&c->stamped_rec, (size_t)128 * c->sm_count * 80) == cudaSuccess;
    ok = ok && cudaMemset(c->stamped_rec, 0, (size_t)128 * c->sm_count * 80) == cudaSuccess;  // no stamp yet
    ok = ok && cudaMemset(c->status, 0, 256) == cudaSuccess;
    ok = ok && cudaDeviceSynchronize() == cudaSuccess;
    if (!ok) {
        disco_destroy(c);
        return DISCO_ERR_CUDA;
    }
    *out = c;
    return DISCO_OK;
}

int disco_destroy(disco_ctx* c) {
    if (!c) return DISCO_ERR_INVALID_ARG;
    cudaFree(c->keys);
    cudaFree(c->part_rec);
    cudaFree(c->stamped_rec);
    cudaFree(c->ticket);
    cudaFree(c->status);
    cudaFree(c->final_stats);
    cudaFree(c->chain_alive);
    cudaFree(c->sample_seg_tot);
    cudaFree(c->sample_seg_last);
    cudaFree(c->sample_tickets);
    cudaFree(c->loop_rec);
    cudaFree(c->pack_rows);
    cudaFree(c->pack_off);
    cudaFree(c->stage_hidden);
    cudaFree(c->stage_hidden_draft);
    if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
    if (c->copy_done) cudaEventDestroy(c->copy_done);
    cudaFreeHost(c->stage_int_h);
    cudaFreeHost(c->stage_float_h);
    cudaFreeHost(c->stage_byte_h);
    delete c;
    return DISCO_OK;
}

int disco_last_device_status(disco_ctx* c, int* out) {
    if (!c || !out) return DISCO_ERR_INVALID_ARG;
    // read and clear on the stream the context was last used on: nothing else on the device is waited for
    int v = 0;
    if (cudaMemcpyAsync(&v, c->status, sizeof(int), cudaMemcpyDeviceToHost, c->last_stream) != cudaSuccess ||
        cudaMemsetAsync(c->status, 0, sizeof(int), c->last_stream) != cudaSuccess ||
        cudaStreamSynchronize(c->last_stream) != cudaSuccess)
        return DISCO_ERR_CUDA;
    *out = v;
    return DISCO_OK;
}

int disco_launch_count(disco_ctx* c, long long* out) {
    if (!c || !out) return DISCO_ERR_INVALID_ARG;
    *out = c->launches;
    return DISCO_OK;
}

int disco_test_hooks(disco_ctx* c, long long wait_budget_clocks, int withhold_records) {
    if (!c || wait_budget_clocks < 0) return DISCO_ERR_INVALID_ARG;
    const long long budget = wait_budget_clocks ? wait_budget_clocks : kDefaultWaitBudgetClocks;
    if (cudaMemcpyToSymbol(g_wait_budget_clocks, &budget, sizeof(budget)) != cudaSuccess) return DISCO_ERR_CUDA;
    c->test_stamp_skew = withhold_records ? 0x40000000u : 0u;
    return DISCO_OK;
}

int disco_set_kernel_path(disco_ctx* c, int which) {
    if (!c || which < 0 || which > 3) return DISCO_ERR_INVALID_ARG;
    c->path = which;
    return DISCO_OK;
}

}  // extern "C"

namespace {
// Launch a small follow-up kernel with programmatic stream serialization (it waits with griddepcontrol.wait
// before it reads anything), so that its launch latency hides behind the kernel before it.
template <typename... KArgs, typename... Args>
cudaError_t launch_after(const disco_ctx* c, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                         Args... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = c->pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// The sampling kernels stage one row of V floats in dynamic shared memory: raise their limit once per device.
bool configure_sampling(disco_ctx* c) {
    static KernelSetup rows_setup;
    const size_t bytes = (size_t)kSampleSmemFloats * sizeof(float);
    return raise_smem_limit(c, rows_setup, sample_rows_kernel, bytes, nullptr);
}

// Shared body of the LM-head + soft-max passes: B rows of hidden size d against the head W.
//   * nll_sum != null selects the perplexity rule (no classifier; tau is the perplexity bound);
//   * stats_only = 1: arg-max (token, optional) and soft-max statistics only, no classifier: the target
//     rows of a verification with sampling (pos, n_drafted, conf, halt unused);
//   * stats_only = 2: token and features, no classifier: bulk feature extraction (n_drafted, conf, halt unused).
int draft_step_common(disco_ctx* c, const void* W_D, const void* h_D, int d, int B, int max_rows, const int32_t* pos,
                      const int32_t* n_drafted, const uint8_t* active, const disco_clf* clf, float tau,
                      int sl_max, int32_t* token, float* conf, uint8_t* halt, float* feats, float* probs,
                      float* nll_sum, int stats_only, void* stream, bool normalize = true,
                      const float* u_draw = nullptr, float* p_token = nullptr, bool* drew = nullptr,
                      const ChainLink* chain = nullptr, unsigned int* clear_words = nullptr, int clear_n = 0) {
    if (!c || !W_D || !h_D) return DISCO_ERR_INVALID_ARG;
    if (!stats_only && !chain && (!pos || !n_drafted)) return DISCO_ERR_INVALID_ARG;
    if (!stats_only && (!token || !conf || !halt)) return DISCO_ERR_INVALID_ARG;
    if (stats_only == 2 && (!pos || !feats)) return DISCO_ERR_INVALID_ARG;
    if (!aligned16(W_D) || !aligned16(h_D)) return DISCO_ERR_INVALID_ARG;
    if (B < 1 || sl_max < 1) return DISCO_ERR_INVALID_ARG;
    if (B > max_rows) return DISCO_ERR_WORKSPACE;
    static const disco_clf no_clf = {nullptr, nullptr, nullptr, nullptr, 0};
    int rc = DISCO_OK;
    if (nll_sum || stats_only) {
        clf = &no_clf;
    } else {
        rc = check_clf(c, clf);
        if (rc) return rc;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    c->last_stream = st;

    TailParams p{};
    p.W = static_cast<const uint16_t*>(W_D);
    p.H = static_cast<const uint16_t*>(h_D);
    p.V = c->V;
    p.d = d;
    p.R = B;
    p.B = B;
    fill_scratch(c, p);
    p.stats_only = stats_only;
    p.pos = pos;
    p.n_drafted = n_drafted;
    p.active = active;
    if (chain) p.chain = *chain;
    p.clear_words = clear_words;
    p.clear_n = clear_n;
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
    p.probs = probs;
    p.nll_sum = nll_sum;
    // Measured on B200 (Vicuna head, us per step for 1 / 2 / 3 / 4 / 6 / 8 sequences): the tensor-core kernel
    // that folds the logits a block at a time 14.8 / 17.0 / 19.4 / 21.3 / 24.8 / 26.8, the one with a thread
    // per hidden row 22.9 / 23.3 / 23.4 / 23.0 / 23.3 / 23.5: the first up to 4 sequences, the second beyond.
    // The CUDA-core streaming kernel is within 5 % for one sequence and serves as the path without tensor maps.
    // (its hidden rows stay in shared memory: up to 48 KB of them, so that the ring keeps at least 8 stages)
    const bool gemv_ok = c->encode_tiled != nullptr && B <= kGemvMaxRows && !stats_only &&
                         (size_t)((d + kUmmaBK - 1) / kUmmaBK) * (B <= 8 ? 8 : 16) * 128 <= 48 * 1024;
    const bool use_gemv = gemv_ok && (c->path == 3 || (c->path == 0 && B <= 4));
    const bool use_umma = !use_gemv && umma_possible(c, B) && (c->path == 2 || c->path == 3 || (c->path == 0 && B >= 2));
    // Sampled step: the kernels that end in a last-CTA second phase draw the token there (their records are
    // at most 160 and in vocabulary order); the batched kernel leaves the draw to a follow-up kernel.
    const bool fused_draw = u_draw && probs && !use_umma && (use_gemv || c->max_grid <= 160);
    if (fused_draw) {
        p.u_draw = u_draw;
        p.p_token = p_token;
        normalize = true;
    }
    if (drew) *drew = fused_draw;
    if (use_gemv) {
        rc = launch_gemv(c, p, st);
        if (rc) return rc;
    } else if (use_umma) {
        DraftFinalParams f{};
        f.B = B;
        f.pos = pos;
        f.n_drafted = n_drafted;
        f.active = active;
        f.clf_W1 = clf->W1;
        f.clf_b1 = clf->b1;
        f.clf_w2 = clf->w2;
        f.clf_b2 = clf->b2;
        f.clf_H = clf->H;
        f.tau = tau;
        f.sl_max = sl_max;
        f.token = token;
        f.conf = conf;
        f.halt = halt;
        f.feats = feats;
        f.final_stats = c->final_stats;
        f.nll_sum = nll_sum;
        f.stats_only = stats_only;
        f.epoch = c->ticket + 48;
        f.test_stamp_skew = c->test_stamp_skew;
        f.clear_words = clear_words;
        f.clear_n = clear_n;
        if (chain) f.chain = *chain;
        rc = stats_only == 1 ? launch_umma<true, true>(c, W_D, h_D, d, B, probs, &f, nullptr, st)
                        : launch_umma<true>(c, W_D, h_D, d, B, probs, &f, nullptr, st);
        if (rc) return rc;
    } else {
        rc = run_stream<true>(c, p, clf->H, st);
        if (rc) return rc;
    }
    if (probs && normalize) {
        dim3 grid((unsigned)std::min(64, (c->V + 255) / 256), (unsigned)B);
        const cudaError_t e = launch_after(c, normalize_probs_kernel, grid, dim3(256), 0, st, probs,
                                           (const float*)c->final_stats, active, c->V);
        c->launches += 1;
        if (!cuda_ok(e, "normalize_probs_kernel launch")) return DISCO_ERR_CUDA;
    }
    return DISCO_OK;
}

// Verification of R rows for B sequences.  pad == null: packed rows (row_off, or a uniform look-ahead SL);
// pad != null: the fixed-shape layout, R = B * (SL + 1) rows of which the first sl[b] + 1 of each sequence
// count (sl is device memory).
int verify_common(disco_ctx* c, const void* W_T, const void* H_T, const int32_t* draft_ids, const int32_t* row_off,
                  int B, int R, int SL, int32_t* n_accept, int32_t* bonus, int32_t* target_ids,
                  const VerifyPadded* pad, void* stream) {
    if (!aligned16(W_T) || !aligned16(H_T)) return DISCO_ERR_INVALID_ARG;
    if (R > c->max_rows) return DISCO_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    c->last_stream = st;

    TailParams p{};
    p.W = static_cast<const uint16_t*>(W_T);
    p.H = static_cast<const uint16_t*>(H_T);
    p.V = c->V;
    p.d = c->d_target;
    p.R = R;
    p.B = B;
    p.SL = SL;
    fill_scratch(c, p);
    p.draft_ids = draft_ids;
    p.row_off = row_off;
    p.n_accept = n_accept;
    p.bonus = bonus;
    p.target_ids = target_ids;
    if (pad) p.padded = *pad;
    const bool use_umma = umma_possible(c, R) && (c->path == 2 || (c->path == 0 && R >= 2));
    if (!use_umma) return run_stream<false>(c, p, 0, st);
    // Fixed-shape rows beyond one tile of 128: the projection is no longer free of charge for the rows that do not
    // count, so they are packed first and the tensor-core kernel tiles for the row count it finds on the device.
    const int32_t* dev_R = nullptr;
    if (pad && R > 128) {
        PackParams pk{};
        pk.H = static_cast<const uint16_t*>(H_T);
        pk.packed = static_cast<uint16_t*>(c->pack_rows);
        pk.sl = pad->sl;
        pk.off = c->pack_off;
        pk.off_user = pad->row_off_out;
        pk.B = B;
        pk.SL = SL;
        pk.d = c->d_target;
        const cudaError_t e = launch_after(c, pack_rows_kernel, dim3((unsigned)(SL + 1), (unsigned)B), dim3(128), 0, st, pk);
        c->launches += 1;
        if (!cuda_ok(e, "pack_rows_kernel launch")) return DISCO_ERR_CUDA;
        H_T = c->pack_rows;
        p.padded.packed_off = c->pack_off;
        p.padded.row_off_out = nullptr;
        dev_R = c->pack_off + B;
    }
    if (B <= 16) {  // few sequences: the last CTA of the main kernel finishes the job, no second launch
        UmmaParams fp{};
        fp.fuse_final = 1;
        fp.ticket = c->ticket + 32;
        fp.draft_ids = draft_ids;
        fp.row_off = row_off;
        fp.B = B;
        fp.SL = p.SL;
        fp.n_accept = n_accept;
        fp.bonus = bonus;
        fp.target_ids = target_ids;
        fp.padded = p.padded;
        return launch_umma<false>(c, W_T, H_T, c->d_target, R, nullptr, nullptr, &fp, st, dev_R);
    }
    int rc = launch_umma<false>(c, W_T, H_T, c->d_target, R, nullptr, nullptr, nullptr, st, dev_R);
    if (rc) return rc;
    VerifyFinalParams f{};
    f.keys = c->keys;
    f.draft_ids = draft_ids;
    f.row_off = row_off;
    f.B = B;
    f.SL = p.SL;
    f.R = R;
    f.n_accept = n_accept;
    f.bonus = bonus;
    f.target_ids = target_ids;
    f.status = c->status;
    f.ticket = c->ticket + 16;
    f.padded = p.padded;
    f.dev_R = dev_R;
    verify_finalize_kernel<<<(B + 3) / 4, 128, 0, st>>>(f);
    c->launches += 1;
    return cuda_ok(cudaGetLastError(), "verify_finalize_kernel launch") ? DISCO_OK : DISCO_ERR_CUDA;
}

}  // namespace

extern "C" {

int disco_draft_step(disco_ctx* c, const void* W_D, const void* h_D, int B, const int32_t* pos,
                     const int32_t* n_drafted, const uint8_t* active, const disco_clf* clf, float tau,
                     int sl_max, int32_t* token, float* conf, uint8_t* halt, float* feats, float* probs,
                     void* stream) {
    if (!c) return DISCO_ERR_INVALID_ARG;
    return draft_step_common(c, W_D, h_D, c->d_draft, B, c->max_batch, pos, n_drafted, active, clf, tau, sl_max, token,
                             conf, halt, feats, probs, nullptr, 0, stream);
}

int disco_draft_step_ppl(disco_ctx* c, const void* W_D, const void* h_D, int B, const int32_t* n_drafted,
                         const uint8_t* active, float* nll_sum, float ppl_max, int sl_max, int32_t* token,
                         float* ppl, uint8_t* halt, void* stream) {
    if (!nll_sum) return DISCO_ERR_INVALID_ARG;
    if (!c) return DISCO_ERR_INVALID_ARG;
    return draft_step_common(c, W_D, h_D, c->d_draft, B, c->max_batch, n_drafted, n_drafted, active, nullptr, ppl_max,
                             sl_max, token, ppl, halt, nullptr, nullptr, nll_sum, 0, stream);
}

int disco_draft_step_sample(disco_ctx* c, const void* W_D, const void* h_D, int B, const int32_t* pos,
                            const int32_t* n_drafted, const uint8_t* active, const disco_clf* clf, float tau,
                            int sl_max, const float* u, int32_t* token, float* p_token, float* conf, uint8_t* halt,
                            float* feats, float* probs, void* stream) {
    if (!c || !u || !probs) return DISCO_ERR_INVALID_ARG;
    bool drew = false;
    int rc = draft_step_common(c, W_D, h_D, c->d_draft, B, c->max_batch, pos, n_drafted, active, clf, tau, sl_max,
                               token, conf, halt, feats, probs, nullptr, 0, stream, false, u, p_token, &drew);
    if (rc) return rc;
    if (drew) return DISCO_OK;   // token drawn by the LM-head kernel's second phase, probs normalised
    // probs holds the logits: the kernel turns them into y^D and replaces the greedy token by the draw
    const size_t smem = sample_smem_bytes(c->V);
    if (!configure_sampling(c)) return DISCO_ERR_CUDA;
    const cudaError_t e = launch_after(c, sample_rows_kernel, dim3(B), dim3(kSampleThreads), smem,
                                       static_cast<cudaStream_t>(stream), probs, (const float*)c->final_stats, u, active,
                                       c->V, smem ? 1 : 0, token, p_token);
    c->launches += 1;
    return cuda_ok(e, "sample_rows_kernel launch") ? DISCO_OK : DISCO_ERR_CUDA;
}

int disco_verify_sample_ragged(disco_ctx* c, const void* W_T, const void* H_T, const int32_t* draft_ids,
                               const float* draft_probs, const int32_t* row_off, int B, int R,
                               const float* u_accept, const float* u_sample, int32_t* n_accept,
                               int32_t* next_token, float* y_T, int32_t* target_ids, void* stream) {
    if (!c || !W_T || !H_T || !u_sample || !n_accept || !next_token || !y_T) return DISCO_ERR_INVALID_ARG;
    if (B < 1 || R < B) return DISCO_ERR_INVALID_ARG;
    if (R > B && (!draft_ids || !draft_probs || !u_accept)) return DISCO_ERR_INVALID_ARG;
    if (B > c->max_batch || R > c->max_rows) return DISCO_ERR_WORKSPACE;
    if (!row_off && R % B != 0) return DISCO_ERR_INVALID_ARG;
    if (!aligned16(W_T) || !aligned16(H_T)) return DISCO_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // logits and soft-max statistics of all rows by the LM-head pass (which also clears the tickets); one more
    // launch normalises the rows, counts the accepted tokens and draws the next one
    int rc = draft_step_common(c, W_T, H_T, c->d_target, R, c->max_rows, nullptr, nullptr, nullptr, nullptr, 0.f, 1,
                               target_ids, nullptr, nullptr, nullptr, y_T, nullptr, 1, stream, false, nullptr, nullptr,
                               nullptr, nullptr, c->sample_tickets, B);
    if (rc) return rc;
    SampleRowsParams sp{};
    sp.y_T = y_T;
    sp.stats = c->final_stats;
    sp.draft_probs = draft_probs;
    sp.draft_ids = draft_ids;
    sp.row_off = row_off;
    sp.u_accept = u_accept;
    sp.u_sample = u_sample;
    sp.B = B;
    sp.SL = row_off ? 0 : (R / B - 1);
    sp.R = R;
    sp.V = c->V;
    // about two CTAs per SM; a row is cut into at most kSampleMaxSegments segments
    sp.SEG = std::max(1, std::min(kSampleMaxSegments, (2 * c->sm_count + R - 1) / R));
    sp.seg_len = ((c->V + sp.SEG - 1) / sp.SEG + 3) & ~3;
    sp.n_accept = n_accept;
    sp.next_token = next_token;
    sp.seg_tot = c->sample_seg_tot;
    sp.seg_last = c->sample_seg_last;
    sp.tickets = c->sample_tickets;
    sp.status = c->status;
    const cudaError_t e = launch_after(c, sample_rows_fused_kernel, dim3((unsigned)R * sp.SEG), dim3(kSampleThreads), 0, st, sp);
    c->launches += 1;
    return cuda_ok(e, "sample_rows_fused_kernel launch") ? DISCO_OK : DISCO_ERR_CUDA;
}

int disco_extract_features(disco_ctx* c, const void* W_D, const void* H_D, const void* W_T, const void* H_T,
                           const int32_t* pos, int N, float* feats_D, float* feats_T, float* tv, uint8_t* label,
                           int32_t* token_D, int32_t* token_T, float* y_D, float* y_T, void* stream) {
    if (!c || !pos || !feats_D || !feats_T || !tv || !label || !token_D || !token_T || !y_D || !y_T)
        return DISCO_ERR_INVALID_ARG;
    if (N < 1) return DISCO_ERR_INVALID_ARG;
    if (N > c->max_rows) return DISCO_ERR_WORKSPACE;
    // everything both passes will check, before the first of them is enqueued
    if (!W_D || !H_D || !W_T || !H_T) return DISCO_ERR_INVALID_ARG;
    if (!aligned16(W_D) || !aligned16(H_D) || !aligned16(W_T) || !aligned16(H_T)) return DISCO_ERR_INVALID_ARG;
    // the same LM-head pass as a draft step, once per model, without the classifier
    int rc = draft_step_common(c, W_D, H_D, c->d_draft, N, c->max_rows, pos, nullptr, nullptr, nullptr, 0.f, 1, token_D,
                               nullptr, nullptr, feats_D, y_D, nullptr, 2, stream);
    if (rc) return rc;
    rc = draft_step_common(c, W_T, H_T, c->d_target, N, c->max_rows, pos, nullptr, nullptr, nullptr, 0.f, 1, token_T,
                           nullptr, nullptr, feats_T, y_T, nullptr, 2, stream);
    if (rc) return rc;
    tv_label_kernel<<<N, 256, 0, static_cast<cudaStream_t>(stream)>>>(y_D, y_T, token_D, token_T, c->V, tv, label);
    c->launches += 1;
    return cuda_ok(cudaGetLastError(), "tv_label_kernel launch") ? DISCO_OK : DISCO_ERR_CUDA;
}

int disco_verify_ragged(disco_ctx* c, const void* W_T, const void* H_T, const int32_t* draft_ids,
                        const int32_t* row_off, int B, int R, int32_t* n_accept, int32_t* bonus,
                        int32_t* target_ids, void* stream) {
    if (!c || !W_T || !H_T || !n_accept || !bonus) return DISCO_ERR_INVALID_ARG;
    if (B < 1 || R < B) return DISCO_ERR_INVALID_ARG;
    if (R > B && !draft_ids) return DISCO_ERR_INVALID_ARG;
    return verify_common(c, W_T, H_T, draft_ids, row_off, B, R, row_off ? 0 : (R / B - 1), n_accept, bonus, target_ids,
                         nullptr, stream);
}

int disco_verify(disco_ctx* c, const void* W_T, const void* H_T, const int32_t* draft_ids, int B, int SL,
                 int32_t* n_accept, int32_t* bonus, int32_t* target_ids, void* stream) {
    if (B < 1 || SL < 0) return DISCO_ERR_INVALID_ARG;
    const long long R = (long long)B * (SL + 1);
    if (c && R > c->max_rows) return DISCO_ERR_WORKSPACE;
    return disco_verify_ragged(c, W_T, H_T, draft_ids, nullptr, B, (int)R, n_accept, bonus, target_ids, stream);
}

int disco_draft_loop(disco_ctx* c, const void* W_D, size_t w_step_stride, const void* h_D, int B, const int32_t* pos0,
                     const disco_clf* clf, float tau, int sl_max, const int32_t* sl_forced, int32_t* token,
                     float* conf, uint8_t* halt, float* feats, int32_t* sl, void* stream) {
    if (!c || !W_D || !h_D || !pos0 || !token || !conf || !halt || !sl) return DISCO_ERR_INVALID_ARG;
    if (B < 1 || sl_max < 1) return DISCO_ERR_INVALID_ARG;
    if (!aligned16(W_D) || !aligned16(h_D) || (w_step_stride & 15u)) return DISCO_ERR_INVALID_ARG;
    if (B > c->max_batch) return DISCO_ERR_WORKSPACE;
    int rc = check_clf(c, clf);
    if (rc) return rc;
    const size_t h_step = (size_t)B * c->d_draft * 2;   // bytes of one step's hidden states
    if (h_step & 15u) return DISCO_ERR_INVALID_ARG;
    if (gemv_loop_possible(c, B, sl_max, w_step_stride)) {
        // a handful of sequences: all steps in one persistent kernel
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        c->last_stream = st;
        TailParams p{};
        p.W = static_cast<const uint16_t*>(W_D);
        p.H = static_cast<const uint16_t*>(h_D);
        p.V = c->V;
        p.d = c->d_draft;
        p.R = B;
        p.B = B;
        fill_scratch(c, p);
        p.chain = ChainLink{c->chain_alive, sl, pos0, sl_forced, 1};
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
        return launch_gemv_loop(c, p, sl_max, w_step_stride, st);
    }
    for (int step = 1; step <= sl_max; ++step) {
        const size_t k = (size_t)(step - 1);
        const ChainLink link{c->chain_alive, sl, pos0, sl_forced, step};
        rc = draft_step_common(c, static_cast<const char*>(W_D) + k * w_step_stride,
                               static_cast<const char*>(h_D) + k * h_step, c->d_draft, B, c->max_batch, nullptr,
                               nullptr, nullptr, clf, tau, sl_max, token + k * B, conf + k * B, halt + k * B,
                               feats ? feats + k * B * kNFeat : nullptr, nullptr, nullptr, 0, stream, true, nullptr,
                               nullptr, nullptr, &link);
        if (rc) return rc;
    }
    return DISCO_OK;
}

int disco_verify_sl(disco_ctx* c, const void* W_T, const void* H_T, const int32_t* draft_ids, long long ids_stride_b,
                    long long ids_stride_j, const int32_t* sl, int B, int sl_max, int32_t* n_accept, int32_t* bonus,
                    int32_t* target_ids, int32_t* row_off, const int32_t* pos0, int32_t* pos_next, void* stream) {
    if (!c || !W_T || !H_T || !sl || !n_accept || !bonus) return DISCO_ERR_INVALID_ARG;
    if (B < 1 || sl_max < 0) return DISCO_ERR_INVALID_ARG;
    if (sl_max > 0 && !draft_ids) return DISCO_ERR_INVALID_ARG;
    if (pos_next && !pos0) return DISCO_ERR_INVALID_ARG;
    const long long R = (long long)B * (sl_max + 1);
    if (R > c->max_rows) return DISCO_ERR_WORKSPACE;
    const VerifyPadded pad{sl, ids_stride_b, ids_stride_j, row_off, pos0, pos_next};
    return verify_common(c, W_T, H_T, draft_ids, nullptr, B, (int)R, sl_max, n_accept, bonus, target_ids, &pad, stream);
}

// late_src (optional): host memory to copy to H_T (late_bytes bytes) on the context's copy stream once the draft
// phase has been enqueued; the verification waits for it.
static int iteration_impl(disco_ctx* c, const void* W_D, size_t w_step_stride, const void* h_D, const void* W_T,
                          const void* H_T, int B, const int32_t* pos0, const disco_clf* clf, float tau, int sl_max,
                          const int32_t* sl_forced, const int32_t* draft_ids, int32_t* token, float* conf, uint8_t* halt,
                          float* feats, int32_t* sl, int32_t* n_accept, int32_t* bonus, int32_t* target_ids,
                          int32_t* row_off, int32_t* pos_next, void* stream, const void* late_src, size_t late_bytes) {
    // everything the second half will check, before the first half is enqueued
    if (!c || !W_T || !H_T || !n_accept || !bonus || !sl) return DISCO_ERR_INVALID_ARG;
    if (!aligned16(W_T) || !aligned16(H_T)) return DISCO_ERR_INVALID_ARG;
    if (B < 1 || sl_max < 1 || (long long)B * (sl_max + 1) > c->max_rows) return B < 1 || sl_max < 1 ? DISCO_ERR_INVALID_ARG : DISCO_ERR_WORKSPACE;
    int rc = disco_draft_loop(c, W_D, w_step_stride, h_D, B, pos0, clf, tau, sl_max, sl_forced, token, conf, halt, feats,
                              sl, stream);
    if (rc) return rc;
    if (late_src &&
        (!cuda_ok(cudaMemcpyAsync(const_cast<void*>(H_T), late_src, late_bytes, cudaMemcpyHostToDevice, c->copy_stream),
                  "cudaMemcpyAsync") ||
         !cuda_ok(cudaEventRecord(c->copy_done, c->copy_stream), "cudaEventRecord") ||
         !cuda_ok(cudaStreamWaitEvent(static_cast<cudaStream_t>(stream), c->copy_done, 0), "cudaStreamWaitEvent")))
        return DISCO_ERR_CUDA;
    if (draft_ids)
        return disco_verify_sl(c, W_T, H_T, draft_ids, sl_max, 1, sl, B, sl_max, n_accept, bonus, target_ids, row_off,
                               pos0, pos_next, stream);
    return disco_verify_sl(c, W_T, H_T, token, 1, B, sl, B, sl_max, n_accept, bonus, target_ids, row_off, pos0,
                           pos_next, stream);
}

int disco_iteration(disco_ctx* c, const void* W_D, size_t w_step_stride, const void* h_D, const void* W_T,
                    const void* H_T, int B, const int32_t* pos0, const disco_clf* clf, float tau, int sl_max,
                    const int32_t* sl_forced, const int32_t* draft_ids, int32_t* token, float* conf, uint8_t* halt,
                    float* feats, int32_t* sl, int32_t* n_accept, int32_t* bonus, int32_t* target_ids,
                    int32_t* row_off, int32_t* pos_next, void* stream) {
    return iteration_impl(c, W_D, w_step_stride, h_D, W_T, H_T, B, pos0, clf, tau, sl_max, sl_forced, draft_ids, token, conf,
                          halt, feats, sl, n_accept, bonus, target_ids, row_off, pos_next, stream, nullptr, 0);
}

int disco_draft_step_host(disco_ctx* c, const void* W_D, const void* h_D_host, int B, const int32_t* pos_host,
                          const int32_t* n_drafted_host, const uint8_t* active_host, const disco_clf* clf,
                          float tau, int sl_max, int32_t* token_host, float* conf_host, uint8_t* halt_host,
                          float* feats_host, void* stream) {
    if (!c || !h_D_host || !pos_host || !n_drafted_host || !token_host || !conf_host || !halt_host)
        return DISCO_ERR_INVALID_ARG;
    if (B < 1) return DISCO_ERR_INVALID_ARG;
    if (B > c->max_batch) return DISCO_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int mb = c->max_batch;
    int32_t* h_pos = c->stage_int_h;
    int32_t* h_nd = h_pos + mb;
    int32_t* h_tok = h_nd + mb;
    float* h_conf = c->stage_float_h;
    float* h_feats = h_conf + mb;
    uint8_t* h_act = c->stage_byte_h;
    uint8_t* h_halt = h_act + mb;
    // host -> device view of the same words
    auto dev_i = [c](int32_t* h) { return c->stage_int_d + (h - c->stage_int_h); };
    auto dev_f = [c](float* h) { return c->stage_float_d + (h - c->stage_float_h); };
    auto dev_b = [c](uint8_t* h) { return c->stage_byte_d + (h - c->stage_byte_h); };
    std::memcpy(h_pos, pos_host, (size_t)B * 4);
    std::memcpy(h_nd, n_drafted_host, (size_t)B * 4);
    if (active_host) std::memcpy(h_act, active_host, (size_t)B);
    if (cudaMemcpyAsync(c->stage_hidden, h_D_host, (size_t)B * c->d_draft * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return DISCO_ERR_CUDA;
    int rc = disco_draft_step(c, W_D, c->stage_hidden, B, dev_i(h_pos), dev_i(h_nd), active_host ? dev_b(h_act) : nullptr,
                              clf, tau, sl_max, dev_i(h_tok), dev_f(h_conf), dev_b(h_halt),
                              feats_host ? dev_f(h_feats) : nullptr, nullptr, stream);
    if (rc) return rc;
    if (cudaStreamSynchronize(st) != cudaSuccess) return DISCO_ERR_CUDA;
    // inactive sequences keep the caller's values: hand back only what the kernel wrote
    for (int b = 0; b < B; ++b) {
        if (active_host && !active_host[b]) continue;
        token_host[b] = h_tok[b];
        conf_host[b] = h_conf[b];
        halt_host[b] = h_halt[b];
        if (feats_host) std::memcpy(feats_host + (size_t)b * kNFeat, h_feats + (size_t)b * kNFeat, kNFeat * 4);
    }
    return DISCO_OK;
}

int disco_verify_ragged_host(disco_ctx* c, const void* W_T, const void* H_T_host, const int32_t* draft_ids_host,
                             const int32_t* row_off_host, int B, int R, int32_t* n_accept_host,
                             int32_t* bonus_host, int32_t* target_ids_host, void* stream) {
    if (!c || !H_T_host || !row_off_host || !n_accept_host || !bonus_host) return DISCO_ERR_INVALID_ARG;
    if (B < 1 || R < B) return DISCO_ERR_INVALID_ARG;
    if (R > B && !draft_ids_host) return DISCO_ERR_INVALID_ARG;
    if (B > c->max_batch || R > c->max_rows) return DISCO_ERR_WORKSPACE;
    // the host can see row_off here, so check it before anything is enqueued
    if (row_off_host[0] != 0 || row_off_host[B] != R) return DISCO_ERR_INVALID_ARG;
    for (int b = 0; b < B; ++b)
        if (row_off_host[b + 1] <= row_off_host[b]) return DISCO_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int mb = c->max_batch, mr = c->max_rows;
    int32_t* h_ids = c->stage_int_h + 3 * (size_t)mb;
    int32_t* h_off = h_ids + mr;
    int32_t* h_nacc = h_off + mb + 1;
    int32_t* h_bonus = h_nacc + mb;
    int32_t* h_tids = h_bonus + mb;
    auto dev_i = [c](int32_t* h) { return c->stage_int_d + (h - c->stage_int_h); };   // device view of the same words
    if (R > B) std::memcpy(h_ids, draft_ids_host, (size_t)(R - B) * 4);
    std::memcpy(h_off, row_off_host, (size_t)(B + 1) * 4);
    if (cudaMemcpyAsync(c->stage_hidden, H_T_host, (size_t)R * c->d_target * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return DISCO_ERR_CUDA;
    int rc = disco_verify_ragged(c, W_T, c->stage_hidden, dev_i(h_ids), dev_i(h_off), B, R, dev_i(h_nacc), dev_i(h_bonus),
                                 target_ids_host ? dev_i(h_tids) : nullptr, stream);
    if (rc) return rc;
    if (cudaStreamSynchronize(st) != cudaSuccess) return DISCO_ERR_CUDA;
    std::memcpy(n_accept_host, h_nacc, (size_t)B * 4);
    std::memcpy(bonus_host, h_bonus, (size_t)B * 4);
    if (target_ids_host) std::memcpy(target_ids_host, h_tids, (size_t)R * 4);
    return DISCO_OK;
}

int disco_iteration_host(disco_ctx* c, const void* W_D, size_t w_step_stride, const void* h_D_host, const void* W_T,
                         const void* H_T_host, int B, const int32_t* pos0_host, const disco_clf* clf, float tau,
                         int sl_max, const int32_t* sl_forced_host, const int32_t* draft_ids_host,
                         int32_t* token_host, float* conf_host, uint8_t* halt_host, int32_t* sl_host,
                         int32_t* n_accept_host, int32_t* bonus_host, int32_t* pos_next_host, void* stream) {
    if (!c || !h_D_host || !H_T_host || !pos0_host || !token_host || !conf_host || !halt_host || !sl_host ||
        !n_accept_host || !bonus_host)
        return DISCO_ERR_INVALID_ARG;
    if (B < 1 || sl_max < 1) return DISCO_ERR_INVALID_ARG;
    const size_t SB = (size_t)sl_max * B, R = (size_t)B * (sl_max + 1);
    if (B > c->max_batch || R > (size_t)c->max_rows) return DISCO_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t mb = (size_t)c->max_batch, mr = (size_t)c->max_rows;
    // pinned, device-mapped staging: pos0 | forced | sl | n_accept | bonus | pos_next (max_batch each), ids | token
    // (max_rows each); conf; halt
    int32_t* h_pos = c->stage_int_h;
    int32_t* h_forced = h_pos + mb;
    int32_t* h_sl = h_forced + mb;
    int32_t* h_nacc = h_sl + mb;
    int32_t* h_bonus = h_nacc + mb;
    int32_t* h_next = h_bonus + mb;
    int32_t* h_ids = h_next + mb;
    int32_t* h_tok = h_ids + mr;
    float* h_conf = c->stage_float_h;
    uint8_t* h_halt = c->stage_byte_h;
    auto dev_i = [c](int32_t* h) { return c->stage_int_d + (h - c->stage_int_h); };
    std::memcpy(h_pos, pos0_host, (size_t)B * 4);
    if (sl_forced_host) std::memcpy(h_forced, sl_forced_host, (size_t)B * 4);
    if (draft_ids_host) std::memcpy(h_ids, draft_ids_host, SB * 4);
    // entries of steps a sequence does not take are not written by the kernels: hand the caller's values back
    std::memcpy(h_tok, token_host, SB * 4);
    std::memcpy(h_conf, conf_host, SB * 4);
    std::memcpy(h_halt, halt_host, SB);
    // The draft phase needs the draft hidden states only: the (larger) target hidden states are sent once it is
    // enqueued, on a stream of their own, and the verification waits for them.  (Every host entry point returns with its
    // work done, so nothing earlier still reads the staging buffers.)
    if (cudaMemcpyAsync(c->stage_hidden_draft, h_D_host, SB * c->d_draft * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return DISCO_ERR_CUDA;
    int rc = iteration_impl(c, W_D, w_step_stride, c->stage_hidden_draft, W_T, c->stage_hidden, B, dev_i(h_pos), clf, tau,
                            sl_max, sl_forced_host ? dev_i(h_forced) : nullptr, draft_ids_host ? dev_i(h_ids) : nullptr,
                            dev_i(h_tok), c->stage_float_d, c->stage_byte_d, nullptr, dev_i(h_sl), dev_i(h_nacc),
                            dev_i(h_bonus), nullptr, nullptr, pos_next_host ? dev_i(h_next) : nullptr, stream, H_T_host,
                            R * c->d_target * 2);
    if (rc) {
        cudaStreamSynchronize(c->copy_stream);   // the copy must not outlive the call
        return rc;
    }
    if (cudaStreamSynchronize(st) != cudaSuccess) return DISCO_ERR_CUDA;
    std::memcpy(token_host, h_tok, SB * 4);
    std::memcpy(conf_host, h_conf, SB * 4);
    std::memcpy(halt_host, h_halt, SB);
    std::memcpy(sl_host, h_sl, (size_t)B * 4);
    std::memcpy(n_accept_host, h_nacc, (size_t)B * 4);
    std::memcpy(bonus_host, h_bonus, (size_t)B * 4);
    if (pos_next_host) std::memcpy(pos_next_host, h_next, (size_t)B * 4);
    return DISCO_OK;
}

}  // extern "C"
