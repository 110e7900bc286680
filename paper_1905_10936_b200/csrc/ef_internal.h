// Internal to libef: workspace layout, the host context and small helpers shared by the
// translation units of the library.  Not part of the interface (that is include/ef.h).
#pragma once

#include "../../include/ef.h"
#include "ef_kernels.cuh"

#include <cstddef>
#include <cstdint>
#include <utility>
#include <vector>

#include <nvtx3/nvToolsExt.h>

namespace efh {

using efk::Block;
using efk::Tile;

constexpr size_t kAlign = 256;
inline size_t align_up(size_t v, size_t a = kAlign) { return (v + a - 1) / a * a; }

// Rows of four elements per thread and chunk: a chunk is 1024*U elements (one CTA of the worker
// and apply kernels), a tile is kTileChunks chunks (one CTA of the server kernel).
constexpr int kU = 4;
constexpr int kChunkLen = 1024 * kU;
// ef_server_step on large layouts: blocks of up to this many tiles get their scale from the
// update kernel itself (every CTA adds the block's <= 4 * 256 partial sums, 8 KB from L2),
// larger ones from ef_scale_kernel.
constexpr int kSelfScaleTiles = 256;
// Grids up to this many chunks (about two waves of CTAs) finalise block scales in-kernel.
constexpr int64_t kFusedMaxChunks = 1024;

struct Layout {
    int64_t d = 0, W = 0;
    int32_t B = 0, M = 0;
    int32_t Ml = 0;                                   // worker state slots held here: M, or 1 with
                                                      // EF_FLAG_ONE_LOCAL_WORKER; the server's buffers sit in slot Ml
    int64_t num_tiles = 0;
    int32_t tile_chunks = 0;                          // chunks per tile: 1 for launch-bound layouts, else kTileChunks
    size_t dpad = 0, wpad = 0, bpad = 0, tpad = 0;    // padded element counts per sub-buffer
    size_t off_x = 0, off_m = 0, off_pb = 0, off_spb = 0, off_words = 0, off_scales = 0,
           off_rscale = 0, off_partials = 0, off_tickets = 0, off_tiles = 0, off_blocks = 0,
           off_multi = 0, off_multi_big = 0, off_ctiles = 0, off_stage = 0, off_mt = 0, off_dpartials = 0,
           off_diag = 0, off_status = 0, total = 0;
    int32_t num_multi = 0;                            // blocks that span more than one chunk
    int32_t num_multi_big = 0;                        // ... and more than kSelfScaleTiles tiles
    int32_t num_ctiles = 0;                           // work items of the one-launch server call (0: not used)
};

}  // namespace efh

struct ef_ctx {
    efh::Layout L;
    float mu = 0.f, eta = 0.f;
    float eta_prev = 0.f;                  // stepsize of the last completed iteration
    float lambda = 0.f;                    // weight decay (needs EF_FLAG_WEIGHT_DECAY)
    uint32_t flags = 0;
    char* ws = nullptr;
    cudaStream_t stream = nullptr;
    int64_t t = 0;
    int64_t launches = 0;
    int last_cuda = 0;
    int pending = 0;                       // workers stepped in the current iteration
    int mode = 0;                          // method of the current iteration (efh::kMode*)
    std::vector<uint8_t> stepped;
    // block-range calls (ef_server_step_range / ef_apply_update): what has been done in this iteration
    std::vector<uint8_t> served, applied;
    int32_t n_served = 0, n_applied = 0;
    std::vector<efk::Tile> h_tiles;             // kept alive: source of an asynchronous upload
    std::vector<efk::Block> h_blocks;
    std::vector<int32_t> h_multi, h_multi_big;
    std::vector<efk::Tile> h_ctiles;            // cluster work items of the one-launch server call
    int fused = 0;                         // block scales finalised inside the main kernels
    // blocks cut across devices (ef_set_block_divisors): slot k's scales of the pieces are still
    // to be completed from the sum over all pieces (ef_complete_scales)
    bool has_partial = false;
    std::vector<uint8_t> scales_open;
    // worker i's last step stored its packed words at the caller's destinations, not in words(i)
    std::vector<uint8_t> pushed;
    bool use_bulk = false;                 // the server kernel stages its inputs with cp.async.bulk
    bool pdl = false;                      // kernels are launched with programmatic stream serialization
    bool one_launch_server = false;        // ef_server_step is the cluster-launched server + update kernel
    // host-staging path
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ev_copied[2] = {nullptr, nullptr};
    cudaEvent_t ev_free[2] = {nullptr, nullptr};
    int64_t host_calls = 0;

    float* x() const { return (float*)(ws + L.off_x); }
    float* m(int i) const { return (float*)(ws + L.off_m) + (size_t)i * L.dpad; }
    int srv() const { return L.Ml; }            // slot of the server's buffers
    float* pb(int i) const {   // i == srv(): server
        return i < L.Ml ? (float*)(ws + L.off_pb) + (size_t)i * L.dpad : (float*)(ws + L.off_spb);
    }
    uint32_t* words(int i) const { return (uint32_t*)(ws + L.off_words) + (size_t)i * L.wpad; }
    float* scales(int i) const { return (float*)(ws + L.off_scales) + (size_t)i * L.bpad; }
    float* rscale(int i) const { return (float*)(ws + L.off_rscale) + (size_t)i * L.bpad; }
    double* partials(int i) const { return (double*)(ws + L.off_partials) + (size_t)i * L.tpad; }
    unsigned* tickets(int i) const { return (unsigned*)(ws + L.off_tickets) + (size_t)i * L.bpad; }
    const efk::Tile* tiles() const { return (const efk::Tile*)(ws + L.off_tiles); }
    const efk::Block* blocks() const { return (const efk::Block*)(ws + L.off_blocks); }
    const int* multi() const { return (const int*)(ws + L.off_multi); }
    const int* multi_big() const { return (const int*)(ws + L.off_multi_big); }
    const efk::Tile* ctiles() const { return (const efk::Tile*)(ws + L.off_ctiles); }
    float* mt() const { return (float*)(ws + L.off_mt); }
    double* dpartials(int i) const { return (double*)(ws + L.off_dpartials) + (size_t)i * 3 * L.tpad; }
    double* diag(int i) const { return (double*)(ws + L.off_diag) + (size_t)i * 4 * L.bpad; }
    float* stage(int s) const { return (float*)(ws + L.off_stage) + (size_t)s * L.dpad; }
    unsigned* status() const { return (unsigned*)(ws + L.off_status); }
    efk::DebugLimits limits() const { return efk::DebugLimits{L.d, L.W, L.B, L.tile_chunks, status()}; }
};

namespace efh {

// NVTX range around one call of the interface, named after the call: a profiler that is
// attached can group or filter the kernels by call (e.g. ncu --nvtx --nvtx-include
// "ef_server_step/"); without one the two calls cost a pointer test each.
struct ApiRange {
    explicit ApiRange(const char* name) { nvtxRangePushA(name); }
    ~ApiRange() { nvtxRangePop(); }
    ApiRange(const ApiRange&) = delete;
    ApiRange& operator=(const ApiRange&) = delete;
};
#define EF_API_RANGE() efh::ApiRange ef_api_range_(__func__)

// Which method the worker calls of the current iteration belong to: the two methods share the
// context's momentum, parameter and packed-word buffers and must not be mixed inside one
// iteration.
enum { kModeNone = 0, kModeEF = 1, kModeVote = 2 };

inline int cuda_fail(ef_ctx* c, cudaError_t e) {
    if (c) c->last_cuda = (int)e;
    return EF_ERR_CUDA;
}
#define EF_CUDA(c, call)                                         \
    do {                                                         \
        cudaError_t e_ = (call);                                 \
        if (e_ != cudaSuccess) return efh::cuda_fail((c), e_);        \
    } while (0)

inline bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

// Launches one of the library's kernels (all take their arguments by value and run kThreads
// threads per CTA) on the context's stream.  With programmatic stream serialization the kernel
// may be scheduled while its predecessor on the stream drains; every kernel begins with
// efk::pdl_enter(), which holds it back until the predecessor's results are complete.
template <typename... KArgs, typename... Args>
inline void launch_kernel(ef_ctx* c, void (*kernel)(KArgs...), dim3 grid, size_t smem, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(efk::kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = c->stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = c->pdl ? 1 : 0;
    cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// Common checks of a per-worker call of method `mode`.
inline int check_worker_call(ef_ctx* c, int32_t i, const float* grad, int mode) {
    if (!c || !grad || i < 0 || i >= c->L.Ml) return EF_ERR_INVALID_ARG;
    if (c->stepped[i]) return EF_ERR_BAD_STATE;
    if (c->pending > 0 && c->mode != mode) return EF_ERR_BAD_STATE;
    return EF_OK;
}
inline void mark_stepped(ef_ctx* c, int32_t i, int mode) {
    c->stepped[i] = 1; c->pending += 1; c->mode = mode;
}
inline void mark_all_stepped(ef_ctx* c, int mode) {
    for (auto& v : c->stepped) v = 1;
    c->pending = c->L.Ml; c->mode = mode;
}
// Host gradients (EF_FLAG_HOST_STAGING): the copy into one of the two staging buffers runs on
// the copy stream, the step kernel on the context's stream waits for it, and a buffer is reused
// only after the kernel that last read it.  stage_host_gradient enqueues copy and wait and
// returns the buffer; host_gradient_consumed is called after the kernel has been enqueued.
inline int stage_host_gradient(ef_ctx* c, const float* grad, float** staged) {
    const int s = (int)(c->host_calls & 1);
    if (c->host_calls >= 2) EF_CUDA(c, cudaStreamWaitEvent(c->copy_stream, c->ev_free[s], 0));
    EF_CUDA(c, cudaMemcpyAsync(c->stage(s), grad, (size_t)c->L.d * 4, cudaMemcpyHostToDevice,
                               c->copy_stream));
    EF_CUDA(c, cudaEventRecord(c->ev_copied[s], c->copy_stream));
    EF_CUDA(c, cudaStreamWaitEvent(c->stream, c->ev_copied[s], 0));
    *staged = c->stage(s);
    return EF_OK;
}
inline int host_gradient_consumed(ef_ctx* c) {
    const int s = (int)(c->host_calls & 1);
    EF_CUDA(c, cudaEventRecord(c->ev_free[s], c->stream));
    c->host_calls += 1;
    return EF_OK;
}

inline void end_iteration(ef_ctx* c) {
    for (auto& v : c->stepped) v = 0;
    for (auto& v : c->served) v = 0;
    for (auto& v : c->applied) v = 0;
    c->n_served = c->n_applied = 0;
    c->pending = 0; c->mode = kModeNone;
    c->t += 1;
}

}  // namespace efh
