// Host side of libef: argument checking, workspace layout, tile table, kernel launches.
// The interface is documented in include/ef.h.
#include "ef_internal.h"

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

namespace {

using efk::Block;
using efk::Tile;
using namespace efh;

int check_problem(int64_t d, int32_t B, const int64_t* offsets, int32_t M) {
    if (!offsets || d < 1 || B < 1 || M < 1 || M > EF_MAX_WORKERS) return EF_ERR_INVALID_ARG;
    if (offsets[0] != 0 || offsets[B] != d) return EF_ERR_INVALID_ARG;
    for (int32_t b = 0; b < B; ++b)
        if (offsets[b + 1] <= offsets[b]) return EF_ERR_INVALID_ARG;
    return EF_OK;
}

int make_layout(int64_t d, int32_t B, const int64_t* offsets, int32_t M, uint32_t flags,
                Layout* L) {
    int rc = check_problem(d, B, offsets, M);
    if (rc != EF_OK) return rc;
    if (flags & ~(EF_FLAG_HOST_STAGING | EF_FLAG_FUSED_SCALE | EF_FLAG_SPLIT_SCALE |
                  EF_FLAG_WEIGHT_DECAY | EF_FLAG_DIAGNOSTICS | EF_FLAG_ONE_LOCAL_WORKER |
                  EF_FLAG_SERVER_NO_BULK | EF_FLAG_PROGRAMMATIC_LAUNCH | EF_FLAG_SEPARATE_UPDATE))
        return EF_ERR_INVALID_ARG;
    if ((flags & EF_FLAG_FUSED_SCALE) && (flags & (EF_FLAG_SPLIT_SCALE | EF_FLAG_DIAGNOSTICS)))
        return EF_ERR_INVALID_ARG;
    L->d = d; L->B = B; L->M = M;
    L->Ml = (flags & EF_FLAG_ONE_LOCAL_WORKER) ? 1 : M;
    int64_t W = 0, chunks = 0;
    for (int32_t b = 0; b < B; ++b) {
        const int64_t db = offsets[b + 1] - offsets[b];
        W += (db + 31) / 32;
        chunks += (db + kChunkLen - 1) / kChunkLen;
        if (db > kChunkLen) L->num_multi += 1;
    }
    // Small layouts are launch-bound: one chunk per tile gives the server and update kernels
    // four times as many (and shorter) CTAs.  Large ones amortise the per-tile set-up over
    // kTileChunks chunks.
    L->tile_chunks = (chunks <= kFusedMaxChunks) ? 1 : efk::kTileChunks;
    const int64_t tile_len = (int64_t)kChunkLen * L->tile_chunks;
    int64_t T = 0, most = 0, single = 0;
    for (int32_t b = 0; b < B; ++b) {
        const int64_t tiles_b = (offsets[b + 1] - offsets[b] + tile_len - 1) / tile_len;
        T += tiles_b;
        most = std::max(most, tiles_b);
        single += tiles_b == 1;
        if (tiles_b > kSelfScaleTiles) L->num_multi_big += 1;
    }
    // One-launch server call (clusters): few chunks, all workers local, no block beyond one cluster.
    // A cluster per multi-chunk block, single-chunk blocks share clusters.
    if (L->tile_chunks == 1 && L->Ml == M && most <= efk::kClusterCtas &&
        !(flags & (EF_FLAG_SEPARATE_UPDATE | EF_FLAG_SPLIT_SCALE | EF_FLAG_DIAGNOSTICS))) {
        const int64_t ctas = efk::kClusterCtas *
                             ((B - single) + (single + efk::kClusterCtas - 1) / efk::kClusterCtas);
        if (ctas <= std::max<int64_t>(4 * T, 512)) L->num_ctiles = (int32_t)ctas;   // not where thousands of CTAs would idle
    }
    if (T * L->tile_chunks > 0x7fffffffLL) return EF_ERR_INVALID_ARG;
    L->W = W; L->num_tiles = T;
    L->dpad = align_up((size_t)d * 4) / 4;
    L->wpad = align_up((size_t)W * 4) / 4;
    L->bpad = align_up((size_t)B * 4) / 4;
    L->tpad = align_up((size_t)T * L->tile_chunks * 8) / 8;     // partial-sum slots
    const size_t Ml = (size_t)L->Ml, M1 = Ml + 1;
    size_t o = 0;
    L->off_x = o;        o += L->dpad * 4;
    L->off_m = o;        o += Ml * L->dpad * 4;
    L->off_pb = o;       o += Ml * L->dpad * 4;
    L->off_spb = o;      o += L->dpad * 4;
    L->off_mt = o;       if (flags & EF_FLAG_WEIGHT_DECAY) o += L->dpad * 4;
    L->off_words = o;    o += M1 * L->wpad * 4;
    L->off_scales = o;   o += M1 * L->bpad * 4;
    L->off_rscale = o;   o += M1 * L->bpad * 4;
    L->off_partials = o; o += M1 * L->tpad * 8;
    L->off_tickets = o;  o += M1 * L->bpad * 4;
    L->off_dpartials = o; if (flags & EF_FLAG_DIAGNOSTICS) o += Ml * 3 * L->tpad * 8;
    L->off_diag = o;      if (flags & EF_FLAG_DIAGNOSTICS) o += Ml * 4 * L->bpad * 8;
    L->off_tiles = o;    o += align_up((size_t)T * sizeof(Tile));
    L->off_blocks = o;   o += align_up((size_t)B * sizeof(Block));
    L->off_multi = o;    o += align_up((size_t)L->num_multi * sizeof(int32_t) + 4);
    L->off_multi_big = o; o += align_up((size_t)L->num_multi_big * sizeof(int32_t) + 4);
    L->off_ctiles = o;   o += align_up((size_t)L->num_ctiles * sizeof(Tile));
    L->off_status = o;   o += kAlign;
    L->off_stage = o;
    if (flags & EF_FLAG_HOST_STAGING) o += 2 * L->dpad * 4;
    L->total = o;
    return EF_OK;
}

}  // namespace

namespace {

// Non-fused mode: adds the partial sums of every block larger than one chunk of buffer set k
// (worker k, or the server for k == M) after the kernel that produced them.
int launch_scale(ef_ctx* c, int k, int count = 1, efk::PushTable push = nullptr) {
    if (c->fused || c->L.num_multi == 0) return EF_OK;
    efk::ScaleArgs a;
    a.push = push;
    a.partials = c->partials(k); a.blocks = c->blocks(); a.multi = c->multi();
    a.scale_out = c->scales(k); a.rscale = c->rscale(k);
    a.partial_stride = (long long)c->L.tpad; a.scale_stride = (int)c->L.bpad;
    a.tc = c->L.tile_chunks;
    const bool diag = (c->flags & EF_FLAG_DIAGNOSTICS) && k < c->L.Ml;
    a.dpartials = diag ? c->dpartials(k) : nullptr;
    a.diag = diag ? c->diag(k) : nullptr;
    const dim3 grid((unsigned)c->L.num_multi, (unsigned)count);
    if (diag) launch_kernel(c, efk::ef_scale_kernel<true>, grid, 0, a);
    else launch_kernel(c, efk::ef_scale_kernel<false>, grid, 0, a);
    EF_CUDA(c, cudaGetLastError());
    c->launches += 1;
    return EF_OK;
}

// Steps workers i .. i+count-1; worker i+k reads its gradient at grad + k*g_stride.
// With a push table (single worker only) the packed words and a copy of the scales go there.
int launch_worker(ef_ctx* c, int i, const float* grad, int count = 1, long long g_stride = 0,
                  efk::PushTable push = nullptr) {
    efk::WorkerArgs a;
    a.push = push;
    a.g = grad; a.m = c->m(i); a.pb = c->pb(i); a.words = c->words(i);
    a.scale_out = c->scales(i); a.rscale = c->rscale(i);
    a.partials = c->partials(i); a.tickets = c->tickets(i);
    a.tiles = c->tiles(); a.blocks = c->blocks(); a.mu = c->mu; a.fused = c->fused;
    a.ratio = c->eta_prev / c->eta;
    a.g_stride = g_stride; a.state_stride = (long long)c->L.dpad;
    a.word_stride = (long long)c->L.wpad; a.partial_stride = (long long)c->L.tpad;
    a.scale_stride = (int)c->L.bpad;
    const bool diag = (c->flags & EF_FLAG_DIAGNOSTICS) != 0;
    a.dpartials = diag ? c->dpartials(i) : nullptr;
    a.diag = diag ? c->diag(i) : nullptr;
    a.lim = c->limits();
    const dim3 grid((unsigned)(c->L.num_tiles * c->L.tile_chunks), (unsigned)count);
    if (diag) launch_kernel(c, efk::ef_worker_kernel<kU, true>, grid, 0, a);
    else launch_kernel(c, efk::ef_worker_kernel<kU, false>, grid, 0, a);
    EF_CUDA(c, cudaGetLastError());
    c->launches += 1;
    for (int k = i; k < i + count; ++k) c->pushed[k] = push != nullptr;
    return launch_scale(c, i, count, push);
}

template <int MT>
size_t server_smem_bytes(int M, bool bulk) {
    return (MT > 0 ? efk::server_ring_bytes<kU>(MT, bulk) : 0) + (size_t)M * sizeof(float);
}

// Raises the dynamic shared-memory limit of the server kernel this context will use.  Done once
// in ef_init so that the step calls themselves only enqueue work.
template <int MT>
cudaError_t prepare_server_t(int M) {
    const size_t smem = server_smem_bytes<MT>(M, false);
    if (smem <= 16 * 1024) return cudaSuccess;    // static + dynamic stays far below the 48 KB default
    cudaError_t e = cudaFuncSetAttribute(efk::ef_server_kernel<kU, MT, false>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess || MT == 0) return e;
    return cudaFuncSetAttribute(efk::ef_server_kernel<kU, (MT > 0 ? MT : 1), true>,
                                cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)server_smem_bytes<MT>(M, true));
}

// Runs CALL(MT) with the template argument that serves M workers: M itself up to 16 (table path), else 0.
#define EF_FOR_WORKER_COUNT(M, CALL)                                                           \
    switch (M) {                                                                               \
        case 1: CALL(1); break;   case 2: CALL(2); break;   case 3: CALL(3); break;            \
        case 4: CALL(4); break;   case 5: CALL(5); break;   case 6: CALL(6); break;            \
        case 7: CALL(7); break;   case 8: CALL(8); break;   case 9: CALL(9); break;            \
        case 10: CALL(10); break; case 11: CALL(11); break; case 12: CALL(12); break;          \
        case 13: CALL(13); break; case 14: CALL(14); break; case 15: CALL(15); break;          \
        case 16: CALL(16); break; default: CALL(0); break;                                     \
    }

cudaError_t prepare_server(int M) {
    cudaError_t e = cudaSuccess;
#define EF_CALL(MT) e = prepare_server_t<MT>(M)
    EF_FOR_WORKER_COUNT(M, EF_CALL)
#undef EF_CALL
    return e;
}

// The one-launch server call: clusters of kClusterCtas CTAs need the kernel's opt-in (above 8),
// and its staging ring may need a raised dynamic shared-memory limit.
template <int MT>
cudaError_t prepare_server_update_t(int M) {
    auto kernel = efk::ef_server_update_kernel<kU, MT>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
    const size_t smem = server_smem_bytes<MT>(M, false);
    if (smem <= 16 * 1024) return cudaSuccess;
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}

// Launch configuration of the one-launch server call; attr must have room for two entries.
template <int MT>
void server_update_config(const ef_ctx* c, cudaLaunchConfig_t* cfg, cudaLaunchAttribute* attr) {
    *cfg = cudaLaunchConfig_t{};
    cfg->gridDim = dim3((unsigned)c->L.num_ctiles);
    cfg->blockDim = dim3(efk::kThreads);
    cfg->dynamicSmemBytes = server_smem_bytes<MT>(c->L.M, false);
    cfg->stream = c->stream;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = efk::kClusterCtas;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg->attrs = attr;
    cfg->numAttrs = c->pdl ? 2 : 1;
}

// Can the device hold at least one cluster of this kernel at a time?  (If not, the call keeps
// its two kernels.)
template <int MT>
cudaError_t server_update_fits_t(const ef_ctx* c, bool* fits) {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    server_update_config<MT>(c, &cfg, attr);
    cfg.numAttrs = 1;
    int clusters = 0;
    const cudaError_t e = cudaOccupancyMaxActiveClusters(&clusters, efk::ef_server_update_kernel<kU, MT>, &cfg);
    *fits = e == cudaSuccess && clusters >= 1;
    return e;
}

template <int MT>
cudaError_t launch_server_update_t(ef_ctx* c, const efk::ServerUpdateArgs& aa) {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    server_update_config<MT>(c, &cfg, attr);
    return cudaLaunchKernelEx(&cfg, efk::ef_server_update_kernel<kU, MT>, aa);
}

cudaError_t prepare_server_update(int M) {
    cudaError_t e = cudaSuccess;
#define EF_CALL(MT) e = prepare_server_update_t<MT>(M)
    EF_FOR_WORKER_COUNT(M, EF_CALL)
#undef EF_CALL
    return e;
}

// Range of tiles that covers the blocks [b0, b1).
struct TileRange { int tile0; unsigned count; };
TileRange tiles_of(const ef_ctx* c, int b0, int b1) {
    const int t0 = c->h_blocks[b0].tile_begin;
    const int t1 = c->h_blocks[b1 - 1].tile_begin + c->h_blocks[b1 - 1].tile_count;
    return {t0, (unsigned)(t1 - t0)};
}

template <int MT>
cudaError_t launch_server_t(ef_ctx* c, const efk::ServerArgs& a, unsigned grid, bool bulk) {
    constexpr int MS = MT > 0 ? MT : 1;
    if (MT > 0 && bulk)
        launch_kernel(c, efk::ef_server_kernel<kU, MS, true>, dim3(grid), server_smem_bytes<MT>(c->L.M, true), a);
    else
        launch_kernel(c, efk::ef_server_kernel<kU, MT, false>, dim3(grid), server_smem_bytes<MT>(c->L.M, false), a);
    return cudaGetLastError();
}

// Server lines of Algorithm 4 on the blocks [b0, b1).  msgs == nullptr: the workers' words and
// scales are the context's own; otherwise worker i's fused message for exactly this block range
// starts at msgs + i * msg_stride.
// defer_scales: the caller applies the update right away with launch_apply_range(.., self_scale):
// only the blocks too large for that get their scale from ef_scale_kernel here.
efk::ServerArgs server_args(ef_ctx* c, int b0, int tile0, const uint32_t* msgs, long long msg_stride) {
    const int M = c->L.M, S = c->srv();
    efk::ServerArgs a;
    a.wwords = msgs ? msgs : c->words(0);
    a.wstride = msgs ? msg_stride : (long long)c->L.wpad;
    a.wscales = c->scales(0); a.sstride = (int)c->L.bpad; a.M = M;
    a.pb = c->pb(S); a.words = c->words(S); a.scale_out = c->scales(S); a.rscale = c->rscale(S);
    a.partials = c->partials(S); a.tickets = c->tickets(S);
    a.tiles = c->tiles(); a.blocks = c->blocks(); a.fused = c->fused;
    a.ratio = c->eta_prev / c->eta;
    a.tile0 = tile0;
    a.fused_in = msgs ? 1 : 0;
    a.msg_base = efk::message_unit(c->h_blocks[b0].word, b0);
    a.status = c->status();
    a.lim = c->limits();
    return a;
}

int launch_server_range(ef_ctx* c, int b0, int b1, const uint32_t* msgs, long long msg_stride,
                        bool defer_scales = false) {
    const int M = c->L.M, S = c->srv();
    const TileRange tr = tiles_of(c, b0, b1);
    const efk::ServerArgs a = server_args(c, b0, tr.tile0, msgs, msg_stride);
    // bulk staging needs every chunk's packed words on a 16-byte boundary: plain layout only
    const bool bulk = c->use_bulk && !msgs;
    cudaError_t le = cudaSuccess;
#define EF_CALL(MT) le = launch_server_t<MT>(c, a, tr.count, bulk)
    EF_FOR_WORKER_COUNT(M, EF_CALL)
#undef EF_CALL
    EF_CUDA(c, le);
    c->launches += 1;
    const std::vector<int32_t>& list = defer_scales ? c->h_multi_big : c->h_multi;
    if (!c->fused && !list.empty()) {
        // follow-up sums for the blocks of the range that span more than one chunk
        const auto lo = std::lower_bound(list.begin(), list.end(), b0) - list.begin();
        const auto hi = std::lower_bound(list.begin(), list.end(), b1) - list.begin();
        if (hi > lo) {
            efk::ScaleArgs sa;
            sa.partials = c->partials(S); sa.blocks = c->blocks();
            sa.multi = (defer_scales ? c->multi_big() : c->multi()) + lo;
            sa.scale_out = c->scales(S); sa.rscale = c->rscale(S);
            sa.partial_stride = (long long)c->L.tpad; sa.scale_stride = (int)c->L.bpad;
            sa.dpartials = nullptr; sa.diag = nullptr; sa.tc = c->L.tile_chunks;
            launch_kernel(c, efk::ef_scale_kernel<false>, dim3((unsigned)(hi - lo), 1), 0, sa);
            EF_CUDA(c, cudaGetLastError());
            c->launches += 1;
        }
    }
    return EF_OK;
}

// x_{t+1} = x_t - eta Deltatilde_t on the blocks [b0, b1); the update is the context's own
// server message (update == nullptr) or a fused message for exactly this block range.
int launch_apply_range(ef_ctx* c, int b0, int b1, const uint32_t* update, bool self_scale = false) {
    const int S = c->srv();
    const TileRange tr = tiles_of(c, b0, b1);
    efk::ApplyArgs p;
    p.x = c->x(); p.words = update ? update : c->words(S); p.scales = c->scales(S);
    p.tiles = c->tiles(); p.blocks = c->blocks(); p.tile0 = tr.tile0;
    p.fused_in = update ? 1 : 0;
    p.msg_base = efk::message_unit(c->h_blocks[b0].word, b0);
    p.eta = c->eta; p.mu = c->mu; p.lambda = c->lambda; p.mt = c->mt();
    p.lim = c->limits();
    p.partials = c->partials(S); p.scale_out = c->scales(S); p.rscale = c->rscale(S);
    p.self_scale_tiles = self_scale ? kSelfScaleTiles : 0;
    if (c->lambda > 0.f)
        launch_kernel(c, efk::ef_apply_kernel<kU, true>, dim3(tr.count), 0, p);
    else
        launch_kernel(c, efk::ef_apply_kernel<kU, false>, dim3(tr.count), 0, p);
    EF_CUDA(c, cudaGetLastError());
    c->launches += 1;
    return EF_OK;
}

// Few chunks, no block beyond one cluster: server lines and update in one launch.
int launch_server_update(ef_ctx* c) {
    efk::ServerUpdateArgs aa;
    aa.s = server_args(c, 0, 0, nullptr, 0);
    aa.ctiles = c->ctiles();
    aa.x = c->x();
    aa.eta = c->eta;
    cudaError_t e = cudaSuccess;
#define EF_CALL(MT) e = launch_server_update_t<MT>(c, aa)
    EF_FOR_WORKER_COUNT(c->L.M, EF_CALL)
#undef EF_CALL
    EF_CUDA(c, e);
    c->launches += 1;
    return EF_OK;
}

int launch_server(ef_ctx* c) {
    if (c->one_launch_server && c->lambda == 0.f) return launch_server_update(c);
    // Large layouts: the update kernel completes the scales of all but the largest blocks itself.
    const bool self_scale = !c->fused;
    const int rc = launch_server_range(c, 0, c->L.B, nullptr, 0, self_scale);
    if (rc != EF_OK) return rc;
    return launch_apply_range(c, 0, c->L.B, nullptr, self_scale);
}

int check_block_range(const ef_ctx* c, int32_t b0, int32_t b1) {
    return (c && b0 >= 0 && b0 < b1 && b1 <= c->L.B) ? EF_OK : EF_ERR_INVALID_ARG;
}

}  // namespace

extern "C" {

int ef_workspace_bytes(int64_t d, int32_t B, const int64_t* offsets, int32_t M, uint32_t flags,
                       size_t* bytes) {
    if (!bytes) return EF_ERR_INVALID_ARG;
    Layout L;
    const int rc = make_layout(d, B, offsets, M, flags, &L);
    if (rc != EF_OK) return rc;
    *bytes = L.total;
    return EF_OK;
}

int ef_init(ef_ctx** out, int64_t d, int32_t B, const int64_t* offsets, int32_t M, float mu,
            float eta, uint32_t flags, void* workspace, size_t workspace_bytes,
            void* cuda_stream) {
    EF_API_RANGE();
    if (!out) return EF_ERR_INVALID_ARG;
    *out = nullptr;
    Layout L;
    int rc = make_layout(d, B, offsets, M, flags, &L);
    if (rc != EF_OK) return rc;
    if (!(mu >= 0.f && mu < 1.f)) return EF_ERR_INVALID_ARG;
    if (!(eta > 0.f) || !std::isfinite(eta)) return EF_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < L.total) return EF_ERR_WORKSPACE;
    if (((uintptr_t)workspace & (kAlign - 1)) != 0) return EF_ERR_ALIGNMENT;

    int dev = -1;
    cudaError_t ce = cudaGetDevice(&dev);
    if (ce != cudaSuccess) return EF_ERR_CUDA;
    int major = 0;
    ce = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (ce != cudaSuccess) return EF_ERR_CUDA;
    if (major != 10) return EF_ERR_UNSUPPORTED_DEVICE;

    ef_ctx* c = new (std::nothrow) ef_ctx();
    if (!c) return EF_ERR_NO_MEMORY;
    c->L = L; c->mu = mu; c->eta = eta; c->eta_prev = eta; c->flags = flags;
    c->ws = (char*)workspace;
    c->stream = (cudaStream_t)cuda_stream;
    c->pdl = (flags & EF_FLAG_PROGRAMMATIC_LAUNCH) != 0;
    try {
    c->stepped.assign(L.Ml, 0);
    c->served.assign(B, 0);
    c->applied.assign(B, 0);
    c->scales_open.assign(L.Ml + 1, 0);
    c->pushed.assign(L.Ml + 1, 0);

    // tile and block tables
    c->h_tiles.reserve((size_t)L.num_tiles);
    c->h_blocks.resize((size_t)B);
    int64_t word = 0;
    for (int32_t b = 0; b < B; ++b) {
        const int64_t start = offsets[b], len = offsets[b + 1] - offsets[b];
        Block& blk = c->h_blocks[b];
        blk.start = start; blk.len = len; blk.word = word;
        blk.div = len; blk.partial = 0; blk.pad = 0;
        blk.tile_begin = (int)c->h_tiles.size();
        const int64_t tile_len = (int64_t)kChunkLen * L.tile_chunks;
        for (int64_t o = 0; o < len; o += tile_len) {
            Tile t;
            t.start = start + o; t.word = word + o / 32;
            t.len = (int)((len - o < tile_len) ? (len - o) : tile_len);
            t.block = b; t.pad0 = 0; t.pad1 = 0;
            c->h_tiles.push_back(t);
        }
        blk.tile_count = (int)c->h_tiles.size() - blk.tile_begin;
        if (len > kChunkLen) c->h_multi.push_back(b);
        if (blk.tile_count > kSelfScaleTiles) c->h_multi_big.push_back(b);
        word += (len + 31) / 32;
    }
    if (L.num_ctiles > 0) {
        // cluster work items: a cluster per multi-chunk block (CTA r takes its r-th chunk and the
        // cluster meets at its barrier), then the single-chunk blocks, kClusterCtas to a cluster
        const Tile idle = {0, 0, 0, 0, 0, 0};
        for (int32_t b = 0; b < B; ++b) {
            const Block& blk = c->h_blocks[b];
            if (blk.tile_count == 1) continue;
            for (int r = 0; r < efk::kClusterCtas; ++r) {
                Tile t = idle;
                if (r < blk.tile_count) { t = c->h_tiles[blk.tile_begin + r]; t.pad1 = blk.tile_begin + r; }
                t.block = b;
                t.pad0 = efk::kClusterTileSync;
                c->h_ctiles.push_back(t);
            }
        }
        for (int32_t b = 0; b < B; ++b) {
            const Block& blk = c->h_blocks[b];
            if (blk.tile_count != 1) continue;
            Tile t = c->h_tiles[blk.tile_begin];
            t.pad1 = blk.tile_begin;
            c->h_ctiles.push_back(t);
        }
        while (c->h_ctiles.size() % efk::kClusterCtas != 0) c->h_ctiles.push_back(idle);
        if ((int64_t)c->h_ctiles.size() != L.num_ctiles) { delete c; return EF_ERR_INVALID_ARG; }
    }
    } catch (const std::bad_alloc&) {
        delete c;
        return EF_ERR_NO_MEMORY;
    }
    // Small grids are launch-bound: finish block scales inside the main kernels.  Large grids
    // are bandwidth-bound: the per-CTA fence of the fused form costs more than a tiny launch.
    if (flags & EF_FLAG_FUSED_SCALE) c->fused = 1;
    else if (flags & (EF_FLAG_SPLIT_SCALE | EF_FLAG_DIAGNOSTICS)) c->fused = 0;
    else c->fused = (L.tile_chunks == 1) ? 1 : 0;

    auto fail = [&](cudaError_t e) { delete c; (void)e; return EF_ERR_CUDA; };
    // Algorithm 4 "Initialize": x_0, m, e, etilde = 0; also words, scales, tickets, partials.
    if ((ce = cudaMemsetAsync(c->ws, 0, L.off_tiles, c->stream)) != cudaSuccess) return fail(ce);
    if ((ce = cudaMemsetAsync(c->status(), 0, kAlign, c->stream)) != cudaSuccess) return fail(ce);
    if ((ce = cudaMemcpyAsync(c->ws + L.off_tiles, c->h_tiles.data(),
                              c->h_tiles.size() * sizeof(Tile), cudaMemcpyHostToDevice,
                              c->stream)) != cudaSuccess) return fail(ce);
    if ((ce = cudaMemcpyAsync(c->ws + L.off_blocks, c->h_blocks.data(),
                              c->h_blocks.size() * sizeof(Block), cudaMemcpyHostToDevice,
                              c->stream)) != cudaSuccess) return fail(ce);
    if (!c->h_multi.empty() &&
        (ce = cudaMemcpyAsync(c->ws + L.off_multi, c->h_multi.data(),
                              c->h_multi.size() * sizeof(int32_t), cudaMemcpyHostToDevice,
                              c->stream)) != cudaSuccess) return fail(ce);
    if (!c->h_multi_big.empty() &&
        (ce = cudaMemcpyAsync(c->ws + L.off_multi_big, c->h_multi_big.data(),
                              c->h_multi_big.size() * sizeof(int32_t), cudaMemcpyHostToDevice,
                              c->stream)) != cudaSuccess) return fail(ce);
    if (!c->h_ctiles.empty() &&
        (ce = cudaMemcpyAsync(c->ws + L.off_ctiles, c->h_ctiles.data(), c->h_ctiles.size() * sizeof(Tile),
                              cudaMemcpyHostToDevice, c->stream)) != cudaSuccess) return fail(ce);
    if ((ce = prepare_server(M)) != cudaSuccess) return fail(ce);
    if (L.num_ctiles > 0) {
        if ((ce = prepare_server_update(M)) != cudaSuccess) return fail(ce);
        bool fits = false;
#define EF_CALL(MT) ce = server_update_fits_t<MT>(c, &fits)
        EF_FOR_WORKER_COUNT(M, EF_CALL)
#undef EF_CALL
        (void)cudaGetLastError();          // a device without room for such a cluster keeps the two kernels
        c->one_launch_server = fits;
        // Programmatic launches pay off exactly where the whole step is two single-wave kernels (the
        // next kernel finds free SMs while its predecessor drains): switched on by default there.
        int per_sm = 0, sms = 0;
        if (fits && cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, efk::ef_worker_kernel<kU, false>,
                                                                  efk::kThreads, 0) == cudaSuccess &&
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess &&
            L.num_tiles * L.tile_chunks * (int64_t)L.Ml <= (int64_t)per_sm * sms)
            c->pdl = true;
    }
    {
        // bulk staging: every block but the last must hold a multiple of 128 elements (so that
        // every chunk's 128 packed words start on a 16-byte boundary) and start 16-byte aligned
        bool aligned = (L.wpad % 4) == 0;
        for (int32_t b = 0; b < B && aligned; ++b)
            aligned = (c->h_blocks[b].word % 4) == 0 && (c->h_blocks[b].start % 4) == 0;
        c->use_bulk = aligned && M <= 16 && !(flags & EF_FLAG_SERVER_NO_BULK);
    }
    if (flags & EF_FLAG_HOST_STAGING) {
        if ((ce = cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking)) != cudaSuccess)
            return fail(ce);
        for (int s = 0; s < 2; ++s) {
            if ((ce = cudaEventCreateWithFlags(&c->ev_copied[s], cudaEventDisableTiming)) != cudaSuccess ||
                (ce = cudaEventCreateWithFlags(&c->ev_free[s], cudaEventDisableTiming)) != cudaSuccess) {
                ef_destroy(c);
                return EF_ERR_CUDA;
            }
        }
    }
    *out = c;
    return EF_OK;
}

int ef_worker_step(ef_ctx* c, int32_t i, const float* grad) {
    EF_API_RANGE();
    int rc = check_worker_call(c, i, grad, kModeEF);
    if (rc != EF_OK) return rc;
    if (!aligned16(grad)) return EF_ERR_ALIGNMENT;
    if (c->scales_open[i]) return EF_ERR_BAD_STATE;      // the last step's cut-block scales are not complete
    rc = launch_worker(c, i, grad);
    if (rc != EF_OK) return rc;
    mark_stepped(c, i, kModeEF);
    if (c->has_partial) c->scales_open[i] = 1;
    return EF_OK;
}

int ef_worker_step_push(ef_ctx* c, int32_t i, const float* grad, uint32_t* const* block_dst) {
    EF_API_RANGE();
    int rc = check_worker_call(c, i, grad, kModeEF);
    if (rc != EF_OK) return rc;
    if (!block_dst) return EF_ERR_INVALID_ARG;
    if (!aligned16(grad)) return EF_ERR_ALIGNMENT;
    if (c->has_partial) return EF_ERR_BAD_STATE;         // a piece's scale is not known inside the step
    rc = launch_worker(c, i, grad, 1, 0, block_dst);
    if (rc != EF_OK) return rc;
    mark_stepped(c, i, kModeEF);
    return EF_OK;
}

int ef_worker_step_all(ef_ctx* c, const float* grads, int64_t stride) {
    EF_API_RANGE();
    if (!c || !grads || stride < c->L.d) return EF_ERR_INVALID_ARG;
    if (!aligned16(grads) || (stride & 3) != 0) return EF_ERR_ALIGNMENT;
    if (c->pending != 0) return EF_ERR_BAD_STATE;
    for (int i = 0; i < c->L.Ml; ++i)
        if (c->scales_open[i]) return EF_ERR_BAD_STATE;
    const int rc = launch_worker(c, 0, grads, c->L.Ml, (long long)stride);
    if (rc != EF_OK) return rc;
    mark_all_stepped(c, kModeEF);
    if (c->has_partial) std::fill(c->scales_open.begin(), c->scales_open.begin() + c->L.Ml, (uint8_t)1);
    return EF_OK;
}

int ef_worker_step_host(ef_ctx* c, int32_t i, const float* grad) {
    EF_API_RANGE();
    int rc = check_worker_call(c, i, grad, kModeEF);
    if (rc != EF_OK) return rc;
    if (!(c->flags & EF_FLAG_HOST_STAGING) || c->scales_open[i]) return EF_ERR_BAD_STATE;
    float* staged = nullptr;
    rc = stage_host_gradient(c, grad, &staged);
    if (rc != EF_OK) return rc;
    rc = launch_worker(c, i, staged);
    if (rc != EF_OK) return rc;
    rc = host_gradient_consumed(c);
    if (rc != EF_OK) return rc;
    mark_stepped(c, i, kModeEF);
    if (c->has_partial) c->scales_open[i] = 1;
    return EF_OK;
}

int ef_server_step(ef_ctx* c) {
    EF_API_RANGE();
    if (!c) return EF_ERR_INVALID_ARG;
    if (c->pending != c->L.M || c->L.Ml != c->L.M || c->mode != kModeEF) return EF_ERR_BAD_STATE;
    if (c->n_served != 0 || c->n_applied != 0) return EF_ERR_BAD_STATE;   // finish the range calls instead
    if (c->has_partial) return EF_ERR_BAD_STATE;        // cut blocks: range calls with ef_complete_scales between
    for (int i = 0; i < c->L.Ml; ++i)
        if (c->pushed[i]) return EF_ERR_BAD_STATE;      // that worker's words are not in the context
    const int rc = launch_server(c);
    if (rc != EF_OK) return rc;
    c->eta_prev = c->eta;
    end_iteration(c);
    return EF_OK;
}

int64_t ef_message_units(ef_ctx* c, int32_t b0, int32_t b1) {
    if (check_block_range(c, b0, b1) != EF_OK) return -1;
    return efk::message_unit(c->h_blocks[b1 - 1].word + (c->h_blocks[b1 - 1].len + 31) / 32, b1) -
           efk::message_unit(c->h_blocks[b0].word, b0);
}

int ef_pack_message(ef_ctx* c, int32_t who, int32_t b0, int32_t b1, uint32_t* dst) {
    return ef_push_message(c, who, b0, b1, 1, &dst);
}

int ef_push_message(ef_ctx* c, int32_t who, int32_t b0, int32_t b1, int32_t n_dst, uint32_t* const* dst) {
    EF_API_RANGE();
    if (check_block_range(c, b0, b1) != EF_OK || !dst || who < -1 || who >= c->L.Ml ||
        n_dst < 1 || n_dst > efk::kMaxPackTargets)
        return EF_ERR_INVALID_ARG;
    for (int q = 0; q < n_dst; ++q)
        if (!dst[q]) return EF_ERR_INVALID_ARG;
    const int k = who < 0 ? c->srv() : who;
    if (c->scales_open[k] || (who >= 0 && c->pushed[k])) return EF_ERR_BAD_STATE;
    const TileRange tr = tiles_of(c, b0, b1);
    efk::PackArgs a;
    a.words = c->words(k); a.scales = c->scales(k);
    a.n_dst = n_dst;
    for (int q = 0; q < efk::kMaxPackTargets; ++q) a.dst[q] = q < n_dst ? dst[q] : nullptr;
    a.tiles = c->tiles(); a.blocks = c->blocks(); a.tile0 = tr.tile0;
    a.msg_base = efk::message_unit(c->h_blocks[b0].word, b0);
    a.lim = c->limits();
    launch_kernel(c, efk::ef_pack_kernel, dim3(tr.count), 0, a);
    EF_CUDA(c, cudaGetLastError());
    c->launches += 1;
    return EF_OK;
}

int ef_server_step_range(ef_ctx* c, int32_t b0, int32_t b1, const uint32_t* msgs, int64_t msg_stride) {
    EF_API_RANGE();
    if (check_block_range(c, b0, b1) != EF_OK) return EF_ERR_INVALID_ARG;
    if (c->pending != c->L.Ml || c->mode != kModeEF) return EF_ERR_BAD_STATE;
    if (!msgs && c->L.Ml != c->L.M) return EF_ERR_BAD_STATE;     // the other workers' messages are needed
    if (!msgs)
        for (int i = 0; i < c->L.Ml; ++i)      // workers' cut-block scales not complete, or words not here
            if (c->scales_open[i] || c->pushed[i]) return EF_ERR_BAD_STATE;
    if (c->scales_open[c->srv()]) return EF_ERR_BAD_STATE;
    if (msgs && c->L.M > 1 && msg_stride < ef_message_units(c, b0, b1)) return EF_ERR_INVALID_ARG;
    for (int32_t b = b0; b < b1; ++b)
        if (c->served[b]) return EF_ERR_BAD_STATE;
    const int rc = launch_server_range(c, b0, b1, msgs, (long long)msg_stride);
    if (rc != EF_OK) return rc;
    for (int32_t b = b0; b < b1; ++b) c->served[b] = 1;
    c->n_served += b1 - b0;
    if (c->has_partial) c->scales_open[c->srv()] = 1;
    return EF_OK;
}

int ef_apply_update(ef_ctx* c, int32_t b0, int32_t b1, const uint32_t* update) {
    EF_API_RANGE();
    if (check_block_range(c, b0, b1) != EF_OK) return EF_ERR_INVALID_ARG;
    if (c->pending != c->L.Ml || c->mode != kModeEF) return EF_ERR_BAD_STATE;
    for (int32_t b = b0; b < b1; ++b)
        if (c->applied[b] || (!update && !c->served[b])) return EF_ERR_BAD_STATE;
    if (!update && c->scales_open[c->srv()]) return EF_ERR_BAD_STATE;
    const int rc = launch_apply_range(c, b0, b1, update);
    if (rc != EF_OK) return rc;
    for (int32_t b = b0; b < b1; ++b) c->applied[b] = 1;
    c->n_applied += b1 - b0;
    if (c->n_applied == c->L.B) {        // every block has its update: the iteration is complete
        c->eta_prev = c->eta;
        end_iteration(c);
    }
    return EF_OK;
}

int ef_set_block_divisors(ef_ctx* c, const int64_t* full_len) {
    if (!c || !full_len) return EF_ERR_INVALID_ARG;
    if (c->t != 0 || c->pending != 0 || (c->flags & EF_FLAG_DIAGNOSTICS)) return EF_ERR_BAD_STATE;
    for (int32_t b = 0; b < c->L.B; ++b)
        if (full_len[b] < c->h_blocks[b].len) return EF_ERR_INVALID_ARG;
    c->has_partial = false;
    for (int32_t b = 0; b < c->L.B; ++b) {
        c->h_blocks[b].div = full_len[b];
        c->h_blocks[b].partial = full_len[b] > c->h_blocks[b].len ? 1 : 0;
        c->has_partial = c->has_partial || c->h_blocks[b].partial;
    }
    EF_CUDA(c, cudaMemcpyAsync(c->ws + c->L.off_blocks, c->h_blocks.data(),
                               c->h_blocks.size() * sizeof(Block), cudaMemcpyHostToDevice, c->stream));
    return EF_OK;
}

int ef_block_sums(ef_ctx* c, int32_t who, double* dst) {
    EF_API_RANGE();
    if (!c || !dst || who < -1 || who >= c->L.Ml) return EF_ERR_INVALID_ARG;
    const int k = who < 0 ? c->srv() : who;
    launch_kernel(c, efk::ef_block_sums_kernel, dim3((unsigned)((c->L.B + efk::kThreads - 1) / efk::kThreads)), 0,
                  c->blocks(), (const double*)c->partials(k), (int)c->L.tile_chunks, (int)c->L.B, dst);
    EF_CUDA(c, cudaGetLastError());
    c->launches += 1;
    return EF_OK;
}

int ef_complete_scales(ef_ctx* c, int32_t who, const double* totals) {
    EF_API_RANGE();
    if (!c || !totals || who < -1 || who >= c->L.Ml) return EF_ERR_INVALID_ARG;
    const int k = who < 0 ? c->srv() : who;
    if (!c->scales_open[k]) return EF_ERR_BAD_STATE;
    launch_kernel(c, efk::ef_complete_scales_kernel,
                  dim3((unsigned)((c->L.B + efk::kThreads - 1) / efk::kThreads)), 0, c->blocks(), totals,
                  (int)c->L.B, c->scales(k), c->rscale(k));
    EF_CUDA(c, cudaGetLastError());
    c->launches += 1;
    c->scales_open[k] = 0;
    return EF_OK;
}

int ef_set_eta(ef_ctx* c, float eta) {
    if (!c || !(eta > 0.f) || !std::isfinite(eta)) return EF_ERR_INVALID_ARG;
    if (c->pending != 0) return EF_ERR_BAD_STATE;
    c->eta = eta;
    return EF_OK;
}

int ef_set_weight_decay(ef_ctx* c, float lambda) {
    if (!c || !(lambda >= 0.f) || !std::isfinite(lambda)) return EF_ERR_INVALID_ARG;
    if (c->pending != 0 || !(c->flags & EF_FLAG_WEIGHT_DECAY)) return EF_ERR_BAD_STATE;
    c->lambda = lambda;
    return EF_OK;
}

const double* ef_worker_diagnostics(ef_ctx* c, int32_t i) {
    return (c && (c->flags & EF_FLAG_DIAGNOSTICS) && i >= 0 && i < c->L.Ml) ? c->diag(i) : nullptr;
}

float* ef_decay_momentum(ef_ctx* c) {
    return (c && (c->flags & EF_FLAG_WEIGHT_DECAY)) ? c->mt() : nullptr;
}

int ef_read_update_host(ef_ctx* c, uint32_t* words, float* scales) {
    EF_API_RANGE();
    if (!c || !words || !scales) return EF_ERR_INVALID_ARG;
    const int M = c->srv();
    EF_CUDA(c, cudaMemcpyAsync(words, c->words(M), (size_t)c->L.W * 4, cudaMemcpyDeviceToHost,
                               c->stream));
    EF_CUDA(c, cudaMemcpyAsync(scales, c->scales(M), (size_t)c->L.B * 4, cudaMemcpyDeviceToHost,
                               c->stream));
    return EF_OK;
}

const uint32_t* ef_worker_words(ef_ctx* c, int32_t i) {
    return (c && i >= 0 && i < c->L.Ml) ? c->words(i) : nullptr;
}
const float* ef_worker_scales(ef_ctx* c, int32_t i) {
    return (c && i >= 0 && i < c->L.Ml) ? c->scales(i) : nullptr;
}
const uint32_t* ef_server_words(ef_ctx* c) { return c ? c->words(c->srv()) : nullptr; }
const float* ef_server_scales(ef_ctx* c) { return c ? c->scales(c->srv()) : nullptr; }
float* ef_params(ef_ctx* c) { return c ? c->x() : nullptr; }
int64_t ef_num_words(ef_ctx* c) { return c ? c->L.W : -1; }

int ef_get_momentum(ef_ctx* c, int32_t i, float* dst) {
    EF_API_RANGE();
    if (!c || !dst || i < 0 || i >= c->L.Ml) return EF_ERR_INVALID_ARG;
    if (!aligned16(dst)) return EF_ERR_ALIGNMENT;
    EF_CUDA(c, cudaMemcpyAsync(dst, c->m(i), (size_t)c->L.d * 4, cudaMemcpyDeviceToDevice,
                               c->stream));
    return EF_OK;
}

int ef_get_residual(ef_ctx* c, int32_t i, float* dst) {
    EF_API_RANGE();
    if (!c || !dst || i < -1 || i >= c->L.Ml) return EF_ERR_INVALID_ARG;
    if (!aligned16(dst)) return EF_ERR_ALIGNMENT;
    const int k = (i < 0) ? c->srv() : i;
    efk::ResidualArgs a;
    a.pb = c->pb(k); a.rscale = c->rscale(k); a.dst = dst; a.tiles = c->tiles();
    a.lim = c->limits();
    launch_kernel(c, efk::ef_residual_kernel, dim3((unsigned)c->L.num_tiles), 0, a);
    EF_CUDA(c, cudaGetLastError());
    c->launches += 1;
    return EF_OK;
}

int ef_set_state(ef_ctx* c, int32_t i, const float* momentum, const float* residual) {
    EF_API_RANGE();
    if (!c || !residual || i < -1 || i >= c->L.Ml) return EF_ERR_INVALID_ARG;
    if (i >= 0 && !momentum) return EF_ERR_INVALID_ARG;
    if (!aligned16(residual) || (momentum && !aligned16(momentum))) return EF_ERR_ALIGNMENT;
    if (c->pending != 0) return EF_ERR_BAD_STATE;
    const int k = (i < 0) ? c->srv() : i;
    const size_t nbytes = (size_t)c->L.d * 4;
    if (i >= 0)
        EF_CUDA(c, cudaMemcpyAsync(c->m(i), momentum, nbytes, cudaMemcpyDeviceToDevice, c->stream));
    // deferred form with scale 0: p -+ 0 gives back the residual exactly (-0 is stored as +0)
    {
        const long long n = c->L.d;
        const unsigned grid = (unsigned)std::min<long long>((n + efk::kThreads - 1) / efk::kThreads, 148 * 16);
        launch_kernel(c, efk::ef_import_kernel, dim3(grid), 0, residual, c->pb(k), n);
        EF_CUDA(c, cudaGetLastError());
        c->launches += 1;
    }
    EF_CUDA(c, cudaMemsetAsync(c->rscale(k), 0, (size_t)c->L.B * 4, c->stream));
    return EF_OK;
}

int ef_step_count(ef_ctx* c, int64_t* t) {
    if (!c || !t) return EF_ERR_INVALID_ARG;
    *t = c->t;
    return EF_OK;
}

int ef_check_status(ef_ctx* c) {
    if (!c) return EF_ERR_INVALID_ARG;
    unsigned word = 0;
    EF_CUDA(c, cudaMemcpyAsync(&word, c->status(), sizeof(word), cudaMemcpyDeviceToHost, c->stream));
    EF_CUDA(c, cudaStreamSynchronize(c->stream));
    if (word == 0) return EF_OK;
    EF_CUDA(c, cudaMemsetAsync(c->status(), 0, sizeof(word), c->stream));
    if (word & efk::kStatusBounds) return EF_ERR_BOUNDS;
    return (word & efk::kStatusWaitTimeout) ? EF_ERR_TIMEOUT : EF_ERR_CUDA;
}

int ef_debug_build(void) {
#ifdef EF_DEBUG
    return 1;
#else
    return 0;
#endif
}

int ef_debug_shift_tile(ef_ctx* c, int64_t tile, int64_t delta) {
#ifdef EF_DEBUG
    if (c && tile == -1) tile = c->L.num_tiles - 1;          // -1 names the last tile
    if (!c || tile < 0 || tile >= c->L.num_tiles || c->pending != 0) return EF_ERR_INVALID_ARG;
    c->h_tiles[(size_t)tile].start += delta;
    EF_CUDA(c, cudaMemcpyAsync(c->ws + c->L.off_tiles + (size_t)tile * sizeof(Tile), &c->h_tiles[(size_t)tile],
                               sizeof(Tile), cudaMemcpyHostToDevice, c->stream));
    // the same tile among the work items of the one-launch server call
    for (size_t k = 0; k < c->h_ctiles.size(); ++k) {
        Tile& ct = c->h_ctiles[k];
        if (ct.len <= 0 || ct.pad1 != (int)tile) continue;
        ct.start += delta;
        EF_CUDA(c, cudaMemcpyAsync(c->ws + c->L.off_ctiles + k * sizeof(Tile), &ct, sizeof(Tile),
                                   cudaMemcpyHostToDevice, c->stream));
    }
    return EF_OK;
#else
    (void)c; (void)tile; (void)delta;
    return EF_ERR_BAD_STATE;
#endif
}

uint32_t* ef_status_word(ef_ctx* c) { return c ? (uint32_t*)c->status() : nullptr; }

int64_t ef_launch_count(ef_ctx* c) { return c ? c->launches : -1; }

const char* ef_strerror(int status) {
    switch (status) {
        case EF_OK: return "ok";
        case EF_ERR_INVALID_ARG: return "invalid argument";
        case EF_ERR_BAD_STATE: return "call order violated";
        case EF_ERR_WORKSPACE: return "workspace missing or too small";
        case EF_ERR_ALIGNMENT: return "pointer not sufficiently aligned";
        case EF_ERR_CUDA: return "CUDA runtime error";
        case EF_ERR_UNSUPPORTED_DEVICE: return "device is not compute capability 10.x";
        case EF_ERR_TIMEOUT: return "device-side wait timed out";
        case EF_ERR_TOO_LARGE: return "size exceeds the fixed scratch of the no-allocation entry point";
        case EF_ERR_NO_MEMORY: return "host allocation failed";
        case EF_ERR_BOUNDS: return "a work item reached outside its arrays (checked build)";
        default: return "unknown status";
    }
}

int ef_last_cuda_error(ef_ctx* c) { return c ? c->last_cuda : 0; }

int ef_destroy(ef_ctx* c) {
    if (!c) return EF_OK;
    for (int s = 0; s < 2; ++s) {
        if (c->ev_copied[s]) cudaEventDestroy(c->ev_copied[s]);
        if (c->ev_free[s]) cudaEventDestroy(c->ev_free[s]);
    }
    if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
    delete c;
    return EF_OK;
}

}  // extern "C"

// =============================================================================================
// ef_stream_probe: no-compute stream kernels with the access mix of the step kernels, so that a
// measured rate can be set against what the memory system gives a kernel of the same shape
// (one 4096-element chunk per CTA, 128-bit accesses through L2) that does no arithmetic worth
// the name.  A measurement aid; not part of the method.
// =============================================================================================
namespace {

template <int MODE>
__global__ void __launch_bounds__(efk::kThreads) ef_stream_probe_kernel(const float* __restrict__ a,
                                                                        float* __restrict__ b,
                                                                        float* __restrict__ c) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long base = (long long)blockIdx.x * kChunkLen + warp * (128 * kU) + lane * 4;
    float4 A[kU], Bv[kU], C[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) {
        if (MODE != EF_PROBE_1R1W) A[u] = efk::ld_stream(a + base + u * 128);
        if (MODE != EF_PROBE_COPY) Bv[u] = efk::ld_stream(b + base + u * 128);
        if (MODE == EF_PROBE_3R2W) C[u] = efk::ld_stream(c + base + u * 128);
    }
#pragma unroll
    for (int u = 0; u < kU; ++u) {
        if (MODE == EF_PROBE_3R2W) {
            Bv[u].x += A[u].x; Bv[u].y += A[u].y; Bv[u].z += A[u].z; Bv[u].w += A[u].w;
            C[u].x += Bv[u].x; C[u].y += Bv[u].y; C[u].z += Bv[u].z; C[u].w += Bv[u].w;
            efk::st_stream(b + base + u * 128, Bv[u]);
            efk::st_stream(c + base + u * 128, C[u]);
        } else if (MODE == EF_PROBE_1R1W) {
            Bv[u].x += 1.f; Bv[u].y -= 1.f; Bv[u].z += 1.f; Bv[u].w -= 1.f;
            efk::st_stream(b + base + u * 128, Bv[u]);
        } else {
            efk::st_stream(c + base + u * 128, A[u]);
        }
    }
}

}  // namespace

extern "C" int ef_stream_probe(int32_t mode, const float* a, float* b, float* c, int64_t n,
                               void* cuda_stream) {
    if (!a || !b || !c || n < kChunkLen || n % kChunkLen != 0 || n / kChunkLen > 0x7fffffffLL)
        return EF_ERR_INVALID_ARG;
    if (!aligned16(a) || !aligned16(b) || !aligned16(c)) return EF_ERR_ALIGNMENT;
    const unsigned grid = (unsigned)(n / kChunkLen);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    switch (mode) {
        case EF_PROBE_3R2W: ef_stream_probe_kernel<EF_PROBE_3R2W><<<grid, efk::kThreads, 0, st>>>(a, b, c); break;
        case EF_PROBE_1R1W: ef_stream_probe_kernel<EF_PROBE_1R1W><<<grid, efk::kThreads, 0, st>>>(a, b, c); break;
        case EF_PROBE_COPY: ef_stream_probe_kernel<EF_PROBE_COPY><<<grid, efk::kThreads, 0, st>>>(a, b, c); break;
        default: return EF_ERR_INVALID_ARG;
    }
    return cudaGetLastError() == cudaSuccess ? EF_OK : EF_ERR_CUDA;
}

// =============================================================================================
// ef_worker_step_noalloc: the worker step for callers that cannot allocate device memory.
//
// Some hosts of this library are not allowed to call cudaMalloc at the point where they step
// the optimizer: code running while another framework owns the allocator or the stream,
// plugins that were handed a fixed arena and must not grow it, and real-time loops
// where an allocation (which may synchronise the whole device) is not tolerable.  The regular
// entry points avoid allocation by taking a caller-sized workspace; this variant needs not even
// that: its scratch memory (one fp64 partial sum per 4096-element chunk plus one arrival
// counter) lives in a fixed array inside the library image, so the caller passes only the
// inputs and outputs of the step.  The price is a size limit (EF_NOALLOC_MAX_ELEMS) and that all
// calls on a device share the one array.
// =============================================================================================
namespace {

constexpr int kNoAllocMaxChunks = EF_NOALLOC_MAX_ELEMS / kChunkLen;
// Scratch of the no-allocation entry point: [0, kNoAllocMaxChunks) partial sums, then one
// 8-byte cell whose low word is the arrival counter.  Every GPU that loads the library holds
// this array (33 KB) until the process exits.
static __device__ __align__(256) double ef_noalloc_scratch[kNoAllocMaxChunks + 1];

struct NoAllocArgs {
    efk::WorkerArgs w;        // g, m, pb, words, mu (tables unused)
    float* rscale_io;         // scale that belongs to pb: read at entry, replaced at exit
    float* scale_out;         // the message's scale
    double* partials;         // device address of ef_noalloc_scratch
    unsigned* ticket;         // arrival counter inside the scratch array (0 at launch)
    long long n;
    int chunks;
};

// Same element arithmetic, chunking and summation order as ef_worker_kernel on a layout with
// a single block of n elements; chunk geometry is computed instead of read from a table.
template <int U>
__global__ void __launch_bounds__(efk::kThreads) ef_worker_noalloc_kernel(const NoAllocArgs a) {
    __shared__ double s_sum[efk::kWarps];
    __shared__ int s_last;
    Tile t;
    t.start = (long long)blockIdx.x * (1024 * U);
    t.word = (long long)blockIdx.x * (1024 * U / 32);
    const long long rest = a.n - t.start;
    t.len = (int)(rest < 1024 * U ? rest : 1024 * U);
    t.block = 0; t.pad0 = 0; t.pad1 = 0;
    const float sp = *a.rscale_io;
    const double acc = (t.len == 1024 * U) ? efk::worker_rows<U, true>(a.w, t, sp)
                                           : efk::worker_rows<U, false>(a.w, t, sp);
    double S = efk::cta_sum(acc, s_sum);
    if (threadIdx.x == 0) {
        int last = 0;
        if (a.chunks == 1) {
            const float s = (float)(S / (double)a.n);
            *a.scale_out = s;
            *a.rscale_io = s;
        } else {
            a.partials[blockIdx.x] = S;
            __threadfence();
            last = (atomicAdd(a.ticket, 1u) + 1u == (unsigned)a.chunks);
        }
        s_last = last;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    double v = 0.0;
    for (int k = threadIdx.x; k < a.chunks; k += efk::kThreads) v += __ldcg(&a.partials[k]);
    S = efk::cta_sum(v, s_sum);
    if (threadIdx.x == 0) {
        const float s = (float)(S / (double)a.n);
        *a.scale_out = s;
        *a.rscale_io = s;       // every CTA has read the old value before it took its ticket
    }
}

constexpr int kNoAllocMaxDevices = 64;
std::mutex g_noalloc_mutex;
double* g_noalloc_ptr[kNoAllocMaxDevices] = {};   // device address of the scratch, per device

}  // namespace

extern "C" int ef_worker_step_noalloc(const float* grad, float* momentum, float* residual,
                                      float* residual_scale, int64_t n, float mu,
                                      uint32_t* words, float* scale, void* cuda_stream) {
    if (!grad || !momentum || !residual || !residual_scale || !words || !scale || n < 1)
        return EF_ERR_INVALID_ARG;
    if (!(mu >= 0.f && mu < 1.f)) return EF_ERR_INVALID_ARG;
    if (n > (int64_t)EF_NOALLOC_MAX_ELEMS) return EF_ERR_TOO_LARGE;
    if (!aligned16(grad) || !aligned16(momentum) || !aligned16(residual)) return EF_ERR_ALIGNMENT;

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return EF_ERR_CUDA;
    if (dev < 0 || dev >= kNoAllocMaxDevices) return EF_ERR_UNSUPPORTED_DEVICE;
    double* scratch = nullptr;
    {
        // One-time set-up per device, done by the first call on that device (with the device
        // current).  In host code the array's name is only a stand-in for the symbol, not a
        // device address, so the address is looked up once and kept.
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (!g_noalloc_ptr[dev]) {
            int major = 0;
            if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
                return EF_ERR_CUDA;
            if (major != 10) return EF_ERR_UNSUPPORTED_DEVICE;
            double* p = nullptr;
            if (cudaGetSymbolAddress((void**)&p, ef_noalloc_scratch) != cudaSuccess || !p)
                return EF_ERR_CUDA;
            g_noalloc_ptr[dev] = p;
        }
        scratch = g_noalloc_ptr[dev];
    }

    cudaStream_t stream = (cudaStream_t)cuda_stream;
    NoAllocArgs a;
    a.w.g = grad; a.w.m = momentum; a.w.pb = residual; a.w.words = words;
    a.w.scale_out = nullptr; a.w.rscale = nullptr; a.w.partials = nullptr; a.w.tickets = nullptr;
    a.w.tiles = nullptr; a.w.blocks = nullptr; a.w.mu = mu; a.w.ratio = 1.f; a.w.fused = 1;
    a.w.g_stride = 0; a.w.state_stride = 0; a.w.word_stride = 0; a.w.partial_stride = 0;
    a.w.scale_stride = 0; a.w.dpartials = nullptr; a.w.diag = nullptr;
    a.rscale_io = residual_scale; a.scale_out = scale;
    a.partials = scratch;
    a.ticket = reinterpret_cast<unsigned*>(scratch + kNoAllocMaxChunks);
    a.n = n;
    a.chunks = (int)((n + kChunkLen - 1) / kChunkLen);
    // The array keeps whatever the previous call left; only the counter must start at zero.
    if (cudaMemsetAsync(a.ticket, 0, sizeof(double), stream) != cudaSuccess) return EF_ERR_CUDA;
    ef_worker_noalloc_kernel<kU><<<(unsigned)a.chunks, efk::kThreads, 0, stream>>>(a);
    if (cudaGetLastError() != cudaSuccess) return EF_ERR_CUDA;
    return EF_OK;
}
