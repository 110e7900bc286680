// Device code of libef: the fused worker and server kernels of dist-EF-blockSGDM
// (Algorithm 4 of arXiv 1905.10936) for sm_100a.
//
// Design in one paragraph.  The path is a pure HBM stream (about 20 bytes and 15 flops per
// element), so there is no tensor-core work; what matters is touching every byte once, with
// 128-bit coalesced accesses and enough loads in flight.  The only non-elementwise step is the
// per-block L1 norm, and the residual e' = p - scale*sign(p) needs that norm.  Instead of a
// second pass over p, the residual is kept in a *deferred* form: the buffer stores p_t and the
// block's scale s_t, and the next iteration rebuilds e_{t+1,j} = p_{t,j} -+ s_t in registers
// while loading (one fp32 add, the same single rounding as the eager form).  The sign used is
// that of p_{t,j}, which is exactly the bit that was sent.  Each launch is therefore one
// streaming pass: read g, m, p_prev; write m, p; write 1 bit per element; plus one fp64
// partial sum per CTA.  The partial sums of a block are added in a fixed order, either by a
// tiny follow-up kernel (large grids: the kernel boundary orders the partial sums for free,
// whereas a device-wide fence in every CTA costs about 8% of the streaming rate) or, for small
// launch-bound grids, by the last CTA to finish the block (one atomic ticket, no waiting).
//
// Work decomposition.  The flat vector is cut into tiles of at most `tc` chunks (tc = kTileChunks
// for bandwidth-bound layouts, 1 for small launch-bound ones, where more and shorter CTAs win) of
// 1024*U elements; a tile never crosses a block boundary.  The worker kernel runs one CTA per
// chunk (three read and two write streams of 16 KB each per CTA keep enough bytes in flight).
// The server and apply kernels have one read and one write stream only, so one CTA walks all
// chunks of a tile: the server kernel stages them ahead through a two-stage shared-memory ring
// (bulk copies issued by one thread and an mbarrier where the layout is 16-byte aligned per
// chunk, per-thread cp.async otherwise), the apply kernel loads chunk c+1 into a second
// register set while it updates c.  The server kernel is the one kernel bound by latency and
// instruction issue rather than by HBM: it needs four CTAs per SM, which fixes how much shared
// memory its sign-pattern tables may take.
//
// Arithmetic is IEEE binary32 with explicit round-to-nearest intrinsics in a fixed order so
// that results do not depend on compiler contraction; block sums are binary64.
#pragma once

#include <cstdint>
#include <type_traits>
#include <cuda_runtime.h>

namespace efk {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr unsigned kFull = 0xffffffffu;
constexpr int kTileChunks = 4;        // most chunks per tile; partial-sum slots per tile = the layout's tc

// A tile is a run of at most kTileChunks*1024*U consecutive elements inside one block.  Tiles
// of a block start at multiples of the tile length from the block's first element, so tiles
// and chunks always start on a packed-word boundary.
struct __align__(16) Tile {
    long long start;   // flat index of the first element
    long long word;    // index of the first packed word
    int len;           // elements in this tile
    int block;         // block id
    int pad0, pad1;
};
static_assert(sizeof(Tile) == 32, "Tile must be 32 bytes");

struct __align__(16) Block {
    long long start;   // flat index of the first element
    long long len;     // elements of the block held here
    long long word;    // index of the block's first packed word
    int tile_begin;    // first tile of this block
    int tile_count;    // number of tiles
    long long div;     // d_b, the divisor of the scale: len, or the whole block's size when this
                       // context holds only a piece of a block that is cut across devices
    int partial;       // 1: such a piece.  Its scale cannot be formed here: the kernels leave the
                       // piece's fp64 sum of |p| in the block's first partial-sum slot instead, and
                       // ef_complete_scales forms the scale from the sum over all pieces
    int pad;
};
static_assert(sizeof(Block) == 48, "Block must be 48 bytes");

// Push table of a worker launch (null: none).  Entry b is where block b's fused message
// [scale | packed words] is to be written: any memory this device can store to, e.g. the receive
// buffer of the block's server on another device.
using PushTable = uint32_t* const*;

// The scale of block b from its L1 sum S (Section 3.2: ||p_b||_1 / d_b), or, for a piece of a
// cut block, the sum itself for ef_complete_scales.  One thread.
__device__ __forceinline__ void publish_scale(const Block& b, int block_id, double S,
                                              double* __restrict__ partials, int tc,
                                              float* __restrict__ scale_out, float* __restrict__ rscale,
                                              PushTable push = nullptr) {
    if (b.partial) {
        partials[(long long)b.tile_begin * tc] = S;
    } else {
        const float s = (float)(S / (double)b.div);
        scale_out[block_id] = s;
        rscale[block_id] = s;
        if (push) push[block_id][0] = __float_as_uint(s);      // first unit of the block's message
    }
}

// Sizes of the problem, carried by every launch.  A build with -DEF_DEBUG checks each CTA's
// work item (tile or chunk descriptor) against them before touching memory: a descriptor that
// reaches outside its arrays is not used; the CTA records kStatusBounds in the status word and
// ends (no trap, no assert: the context stays usable and ef_check_status reports it).
struct DebugLimits {
    long long d, W;      // elements, packed words
    int B;               // blocks
    int tc;              // chunks per tile of this layout (1 or kTileChunks)
    unsigned* status;
};
constexpr unsigned kStatusBounds = 2u;
__device__ __forceinline__ bool work_item_ok(const Tile& t, const DebugLimits& lim, int max_len) {
#ifdef EF_DEBUG
    const long long len = t.len > 0 ? t.len : 0;      // an empty item touches no element
    const bool ok = t.block >= 0 && t.block < lim.B && t.len <= max_len &&
                    (len == 0 || (t.start >= 0 && t.start + len <= lim.d && t.word >= 0 &&
                                  t.word + (len + 31) / 32 <= lim.W));
    if (!ok && threadIdx.x == 0) atomicOr(lim.status, kStatusBounds);
    return ok;
#else
    return true;
#endif
}

struct WorkerArgs {
    const float* g;        // gradient g_{t,i}
    float* m;              // momentum m_i (in/out)
    float* pb;             // deferred residual: p_{t-1,i} in, p_{t,i} out
    uint32_t* words;       // packed signs of p_{t,i}
    float* scale_out;      // per-block scales of the message
    float* rscale;         // per-block scale that belongs to pb (in: t-1, out: t)
    double* partials;      // kTileChunks fp64 partial L1 sums per tile
    unsigned* tickets;     // one arrival counter per block (0 between launches)
    const Tile* tiles;
    const Block* blocks;
    float mu;
    float ratio;           // eta_{t-1} / eta_t: rescale of the residual (1 for a constant stepsize)
    int fused;             // 1: last CTA of a block finalises its scale; 0: ef_scale_kernel does
    // batched launches: blockIdx.y selects the worker; its buffers lie at these strides
    long long g_stride, state_stride, word_stride, partial_stride;
    int scale_stride;      // also the stride of the ticket arrays
    // diagnostics (DIAG instantiation only): per-CTA partial sums of p^2, |g|, g^2 in three
    // arrays of `partial_stride` slots each, and the per-block results [B][4] (|p|, p^2, |g|, g^2)
    double* dpartials;
    double* diag;
    PushTable push;        // not null: the message goes there instead of to `words` (single-worker launches)
    DebugLimits lim;
};

struct ServerArgs {
    const uint32_t* wwords;  // packed signs of worker 0; worker i at + i*wstride
    long long wstride;
    const float* wscales;    // scales of worker 0; worker i at + i*sstride
    int sstride;
    int M;
    float* pb;               // deferred server residual: ptilde_{t-1} in, ptilde_t out
    uint32_t* words;         // packed signs of ptilde_t
    float* scale_out;
    float* rscale;
    double* partials;
    unsigned* tickets;
    const Tile* tiles;
    const Block* blocks;
    int fused;
    float ratio;             // eta_{t-1} / eta_t
    // block-range launches: the grid covers tiles tile0 .. tile0 + gridDim.x - 1
    int tile0;
    // fused messages: worker i's packed words AND scales come from one buffer per worker,
    // wwords + i*wstride, that holds the blocks from block `first` on as [scale | words] units
    // (message_unit below); wscales is unused then
    int fused_in;
    long long msg_base;      // message_unit of the first block the buffers hold
    unsigned* status;        // the context's status word (bounded waits report here)
    DebugLimits lim;
};

// Fused message layout: the message of a block range [b0, b1) is, block after block, one 32-bit
// unit holding the block's scale (a float) followed by the block's packed words.  The scale of
// block b sits at unit (word_b + b) - (word_b0 + b0) and its words right behind it, where word_b
// is the block's first packed word in the plain layout.
__host__ __device__ __forceinline__ long long message_unit(long long block_word, int block) {
    return block_word + block;
}

struct ScaleArgs {
    double* partials;
    const Block* blocks;
    const int* multi;        // ids of the blocks that span more than one chunk
    float* scale_out;
    float* rscale;
    long long partial_stride;   // blockIdx.y selects the buffer set (worker)
    int scale_stride;
    double* dpartials;          // DIAG instantiation only, as in WorkerArgs
    double* diag;
    int tc;                     // chunks (= partial-sum slots) per tile
    PushTable push;             // as in WorkerArgs
};

struct ApplyArgs {
    float* x;
    const uint32_t* words;   // server packed signs (or a fused message, see ServerArgs)
    const float* scales;     // server scales (unused with fused_in)
    const Tile* tiles;
    const Block* blocks;
    int tile0;
    int fused_in;
    long long msg_base;
    float eta;
    // weight decay kept out of the compressor (Appendix A); used by the DECAY instantiation only
    float* mt;               // decay momentum mtilde
    float mu, lambda;
    DebugLimits lim;
    // Scales completed here (ef_server_step, large layouts): for a block of more than one chunk
    // and at most `self_scale_tiles` tiles (0: never) every CTA adds the block's partial sums
    // itself, in ef_scale_kernel's order, instead of waiting for a launch of that kernel; the
    // CTA of the block's first tile also records the scale.  Saves a launch per server step.
    const double* partials;
    float* scale_out;
    float* rscale;
    int self_scale_tiles;
};

struct ResidualArgs {
    const float* pb;
    const float* rscale;
    float* dst;
    const Tile* tiles;
    DebugLimits lim;
};

// ------------------------------------------------------------------ programmatic dependent launch
// pdl_wait(): until the kernel launched before this one on the stream has completed and its
// writes are visible (a no-op for an ordinary launch).  pdl_trigger(): the kernel launched after
// this one may be scheduled as soon as SM resources free up.  With the launch attribute set on
// the host side (EF_FLAG_PROGRAMMATIC_LAUNCH) this overlaps a kernel's launch latency, its
// descriptor loads and whatever else it may do before its wait with the predecessor's tail.
//
// Most kernels start with pdl_enter() = wait, then trigger: nothing of theirs touches global
// memory before the predecessor is complete.  Two kernels do part of their work BEFORE the wait:
//  * the worker kernel loads its descriptors and the worker's own state (m_i, the deferred
//    residual and its scales) first; the gradient and every store come after the wait;
//  * the one-launch server kernel loads its work item and its x values first.
// That is safe as long as the kernel directly before them does not write what they read early
// while having triggered early itself.  Inside the library the only writers of a worker's state
// that can directly precede that worker's step are the state import and the completion of cut
// blocks' scales: those two wait and never trigger (their dependents start when they are done).
// x is written by the update kernels, and a server call is always preceded by worker kernels.
// Kernels of the caller that write x or worker state through the raw pointers must not signal
// early either when this mode is on.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_enter() {
    pdl_wait();
    pdl_trigger();
}

// ------------------------------------------------------------------ small helpers
// Streaming accesses go through L2 only (.cg): every byte is used once per launch, and on
// B200 this measured about 2% faster than the evict-first (.cs) forms.
__device__ __forceinline__ float4 ld_stream(const float* p) {
    return __ldcg(reinterpret_cast<const float4*>(p));
}
__device__ __forceinline__ void st_stream(float* p, float4 v) {
    __stcg(reinterpret_cast<float4*>(p), v);
}

// Sign convention: sign(+-0) = +1 (Appendix A maps signs to {-1,+1}), i.e. "negative" means
// p < 0.  The kernels test the IEEE sign bit instead, which is the same predicate for every
// value except -0.0, so -0.0 must never be stored in a residual buffer:
//  * constant stepsize (ratio == 1): the scale s is >= +0, so e = p - s*sign(p) is never -0
//    (x - x = +0 in round-to-nearest); p = fl(v + e) with e != -0 is -0 only if the exact sum is
//    zero, which rounds to +0 (a sum of two binary32 numbers never underflows);
//  * rescaled residual (ratio != 1): p = fma(ratio, e, v) CAN underflow to -0 (e.g. ratio = 1/2,
//    e = -2^-149, v = +0), so those paths add +0 afterwards (corrected_vector below), which maps
//    -0 to +0 and changes nothing else;
//  * the buffers start at +0 and ef_set_state adds +0 to what it imports.  (NaN is unspecified.)
//
// e_{t+1,j} = p_{t,j} - s * sign(p_{t,j})   (Algorithm 4): one rounding, as p + s or p - s.
// It enters the next corrected vector as fma(eta_{t-1}/eta_t, e, .), which is fl(. + e) for a
// constant stepsize.
__device__ __forceinline__ float residual_of(float pb, float s) {
    const float signed_s = __uint_as_float((__float_as_uint(pb) & 0x80000000u) | __float_as_uint(s));
    return __fsub_rn(pb, signed_s);
}

// p = v + (eta_{t-1}/eta_t) e (Algorithm 4), never -0 (see above).  `rescale` is ratio != 1,
// uniform over the launch.
__device__ __forceinline__ float corrected_vector(float ratio, bool rescale, float e, float v) {
    const float p = __fmaf_rn(ratio, e, v);
    return rescale ? __fadd_rn(p, 0.0f) : p;
}

// Sign bits of four values as a nibble, element k in bit k.
__device__ __forceinline__ unsigned sign_nibble(const float (&v)[4]) {
    unsigned n = __float_as_uint(v[3]) >> 31;
    n = __funnelshift_l(__float_as_uint(v[2]), n, 1);
    n = __funnelshift_l(__float_as_uint(v[1]), n, 1);
    n = __funnelshift_l(__float_as_uint(v[0]), n, 1);
    return n;
}

__device__ __forceinline__ double abs_sum4(const float (&v)[4]) {
    return ((double)fabsf(v[0]) + (double)fabsf(v[1])) + ((double)fabsf(v[2]) + (double)fabsf(v[3]));
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}

// Sum over the CTA in a fixed order; the result is valid in thread 0 only.
__device__ __forceinline__ double cta_sum(double v, double* s_sum) {
    v = warp_sum(v);
    if ((threadIdx.x & 31) == 0) s_sum[threadIdx.x >> 5] = v;
    __syncthreads();
    double S = 0.0;
    if (threadIdx.x == 0) {
        S = s_sum[0];
#pragma unroll
        for (int w = 1; w < kWarps; ++w) S += s_sum[w];
    }
    return S;
}

// Adds the partial sums of block b in a fixed order (thread k takes slots k, k+256, ...; then
// the CTA tree) and writes the scale s_b = ||p_b||_1 / d_b (Section 3.2).  Called by a whole CTA.
// Sum of the block's partial-sum slots in a fixed order; valid in thread 0.
__device__ __forceinline__ double sum_slots(const Block& b, const double* __restrict__ partials,
                                            double* s_sum, int tc) {
    const double* src = partials + (long long)b.tile_begin * tc;
    const int n = b.tile_count * tc;
    double v = 0.0;
    for (int k = threadIdx.x; k < n; k += kThreads) v += __ldcg(&src[k]);
    return cta_sum(v, s_sum);
}

__device__ __forceinline__ double sum_partials_and_write(const Block& b, int block_id,
                                                         double* __restrict__ partials,
                                                         float* __restrict__ scale_out,
                                                         float* __restrict__ rscale,
                                                         double* s_sum, int tc, PushTable push = nullptr) {
    const double S = sum_slots(b, partials, s_sum, tc);
    if (threadIdx.x == 0) publish_scale(b, block_id, S, partials, tc, scale_out, rscale, push);
    return S;
}

// End of a CTA's work: turns its |p| sum into the block scale or a published partial sum.
//   slot      partial-sum slot of this CTA; `zero_slots` further slots are set to 0
//   alone     this CTA covered the whole block: write the scale directly
//   expected  number of CTAs that arrive at the block's ticket in fused mode
// For blocks covered by several CTAs the partial sum is stored; if `fused`, the CTA that
// arrives last at the block's ticket also adds all partial sums (no CTA ever waits for another
// one), otherwise ef_scale_kernel does that after this launch.
__device__ __forceinline__ void finish_block(double acc, long long slot, int zero_slots, bool alone,
                                             unsigned expected, int block_id,
                                             const Block* __restrict__ blocks,
                                             double* __restrict__ partials,
                                             unsigned* __restrict__ tickets,
                                             float* __restrict__ scale_out,
                                             float* __restrict__ rscale, int fused, int tc,
                                             PushTable push = nullptr) {
    __shared__ double s_sum[kWarps];
    __shared__ int s_last;
    const double S = cta_sum(acc, s_sum);
    if (threadIdx.x == 0) {
        int last = 0;
        if (alone) {
            publish_scale(blocks[block_id], block_id, S, partials, tc, scale_out, rscale, push);
        } else {
            partials[slot] = S;
            for (int z = 1; z <= zero_slots; ++z) partials[slot + z] = 0.0;
            if (fused) {
                __threadfence();
                const unsigned old = atomicAdd(&tickets[block_id], 1u);
                last = (old + 1u == expected);
            }
        }
        s_last = last;
    }
    if (!fused) return;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const Block b = blocks[block_id];
    sum_partials_and_write(b, block_id, partials, scale_out, rscale, s_sum, tc, push);
    if (threadIdx.x == 0) tickets[block_id] = 0u;      // ready for the next launch
}

// Follow-up kernel of the non-fused mode: one CTA per block that spans more than one chunk.
// DIAG also completes the three diagnostic sums and records all four per block.
template <bool DIAG>
__global__ void __launch_bounds__(kThreads) ef_scale_kernel(const ScaleArgs a) {
    __shared__ double s_sum[kWarps];
    pdl_enter();
    const int block_id = a.multi[blockIdx.x];
    const Block b = a.blocks[block_id];
    const long long so = (long long)blockIdx.y * a.scale_stride;
    const double S = sum_partials_and_write(b, block_id, a.partials + blockIdx.y * a.partial_stride,
                                            a.scale_out + so, a.rscale + so, s_sum, a.tc, a.push);
    if (DIAG) {
        double* dg = a.diag + (so + block_id) * 4;
        if (threadIdx.x == 0) dg[0] = S;
        const double* dp = a.dpartials + blockIdx.y * (3 * a.partial_stride);
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            __syncthreads();
            const double v = sum_slots(b, dp + k * a.partial_stride, s_sum, a.tc);
            if (threadIdx.x == 0) dg[1 + k] = v;
        }
    }
}

// Diagnostic sums of one thread: p^2, |g|, g^2 (|p| is the compressor's own sum).
struct DiagAcc {
    double p2 = 0.0, g1 = 0.0, g2 = 0.0;
};

// End of a CTA's work in the DIAG instantiation (always the non-fused mode): publishes the four
// sums as partial sums, or as final per-block values when the CTA covered the whole block.
__device__ __forceinline__ void finish_block_diag(double acc, const DiagAcc& d, long long slot,
                                                  bool alone, int block_id, long long block_len,
                                                  double* __restrict__ partials,
                                                  double* __restrict__ dpartials,
                                                  long long partial_stride,
                                                  double* __restrict__ diag,
                                                  float* __restrict__ scale_out,
                                                  float* __restrict__ rscale, PushTable push) {
    __shared__ double s_sum[kWarps];
    const double in[4] = {acc, d.p2, d.g1, d.g2};
    double r[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        r[k] = cta_sum(in[k], s_sum);
        __syncthreads();
    }
    if (threadIdx.x != 0) return;
    if (alone) {
        const float s = (float)(r[0] / (double)block_len);
        scale_out[block_id] = s;
        rscale[block_id] = s;
        if (push) push[block_id][0] = __float_as_uint(s);
#pragma unroll
        for (int k = 0; k < 4; ++k) diag[(long long)block_id * 4 + k] = r[k];
    } else {
        partials[slot] = r[0];
#pragma unroll
        for (int k = 0; k < 3; ++k) dpartials[k * partial_stride + slot] = r[1 + k];
    }
}

// Packs the four sign bits each lane holds (nibble, element k in bit k) into 32-bit words:
// lanes 8q..8q+7 together hold 32 consecutive elements.  Returns the word in every lane of
// the group.
__device__ __forceinline__ unsigned pack_nibbles(unsigned nib, int lane) {
    // three xor-shuffles; a single __reduce_or_sync over the 8-lane group measured slower
    unsigned v = nib << ((lane & 7) * 4);
    v |= __shfl_xor_sync(kFull, v, 1);
    v |= __shfl_xor_sync(kFull, v, 2);
    v |= __shfl_xor_sync(kFull, v, 4);
    return v;
}

__device__ __forceinline__ void load4(const float* p, int o, int len, bool full, float (&v)[4]) {
    if (full || o + 4 <= len) {
        const float4 q = ld_stream(p);
        v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
    } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) v[k] = (o + k < len) ? p[k] : 0.f;
    }
}
__device__ __forceinline__ void store4(float* p, int o, int len, bool full, const float (&v)[4]) {
    if (full || o + 4 <= len) {
        st_stream(p, make_float4(v[0], v[1], v[2], v[3]));
    } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) if (o + k < len) p[k] = v[k];
    }
}

// Chunk `sub` of tile t as a tile of its own (len <= 0 if the tile has no such chunk).
template <int U>
__device__ __forceinline__ Tile chunk_of(const Tile& t, int sub) {
    Tile c = t;
    c.start += (long long)sub * (1024 * U);
    c.word += sub * (1024 * U / 32);
    const int rest = t.len - sub * (1024 * U);
    c.len = rest < 1024 * U ? rest : 1024 * U;
    return c;
}

// ------------------------------------------------------------------ worker kernel
// One chunk per CTA.  Warp w owns the 128*U consecutive elements starting at w*128*U; in row u
// lane l holds elements u*128 + 4l .. +3 (a 128-bit access, 512 contiguous bytes per warp).
template <int U, bool FULL, bool DIAG = false>
__device__ __forceinline__ double worker_rows(const WorkerArgs& a, const Tile& t, float sp,
                                              DiagAcc* dacc = nullptr) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int o0 = warp * (128 * U) + lane * 4;
    const float* gp = a.g + t.start + o0;
    float* mp = a.m + t.start + o0;
    float* pp = a.pb + t.start + o0;
    float g[U][4], m[U][4], p[U][4];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        load4(mp + u * 128, o0 + u * 128, t.len, FULL, m[u]);
        load4(pp + u * 128, o0 + u * 128, t.len, FULL, p[u]);
    }
    // the worker's own state is in flight; the gradient (the caller's) and all stores follow the wait
    pdl_wait();
#pragma unroll
    for (int u = 0; u < U; ++u) load4(gp + u * 128, o0 + u * 128, t.len, FULL, g[u]);
    double acc = 0.0;
    const bool rescale = a.ratio != 1.0f;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int o = o0 + u * 128;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float e = residual_of(p[u][k], sp);                // e_{t,i}
            m[u][k] = __fmaf_rn(a.mu, m[u][k], g[u][k]);             // m_t = mu m_{t-1} + g
            const float v = __fmaf_rn(a.mu, m[u][k], g[u][k]);       // mu m_t + g
            float pv = corrected_vector(a.ratio, rescale, e, v);     // p_t = v + (eta_{t-1}/eta_t) e
            if (!FULL && o + k >= t.len) pv = 0.f;
            p[u][k] = pv;
        }
        const unsigned nib = sign_nibble(p[u]);
        acc += abs_sum4(p[u]);
        if (DIAG) {
            // The four elements of a lane are combined in fp32 (all terms are >= 0, so the
            // relative error stays below 4 * 2^-24) and added to the fp64 sums once per row:
            // diagnostics need 1e-6, not the 1e-13 of the scale.  g is 0 beyond the chunk's end.
            float p2 = __fmul_rn(p[u][0], p[u][0]), g2 = __fmul_rn(g[u][0], g[u][0]);
#pragma unroll
            for (int k = 1; k < 4; ++k) {
                p2 = __fmaf_rn(p[u][k], p[u][k], p2);
                g2 = __fmaf_rn(g[u][k], g[u][k], g2);
            }
            const float g1 = __fadd_rn(__fadd_rn(fabsf(g[u][0]), fabsf(g[u][1])),
                                       __fadd_rn(fabsf(g[u][2]), fabsf(g[u][3])));
            dacc->p2 += (double)p2;
            dacc->g1 += (double)g1;
            dacc->g2 += (double)g2;
        }
        const unsigned w = pack_nibbles(nib, lane);
        store4(mp + u * 128, o, t.len, FULL, m[u]);
        store4(pp + u * 128, o, t.len, FULL, p[u]);
        if ((lane & 7) == 0 && (FULL || o < t.len)) a.words[t.word + (o >> 5)] = w;
    }
    return acc;
}

// Fallback for chunks that do not start on a 16-byte boundary: 32-bit accesses, one ballot per
// 32 elements.
template <bool DIAG = false>
__device__ __forceinline__ double worker_rows_scalar(const WorkerArgs& a, const Tile& t, float sp,
                                                     DiagAcc* dacc = nullptr) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rows = (t.len + 31) >> 5;
    double acc = 0.0;
    pdl_wait();
    for (int r = warp; r < rows; r += kWarps) {
        const int o = r * 32 + lane;
        const bool valid = o < t.len;
        float pv = 0.f;
        if (valid) {
            const long long j = t.start + o;
            const float g = a.g[j];
            const float e = residual_of(a.pb[j], sp);
            const float m = __fmaf_rn(a.mu, a.m[j], g);
            pv = corrected_vector(a.ratio, a.ratio != 1.0f, e, __fmaf_rn(a.mu, m, g));
            a.m[j] = m;
            a.pb[j] = pv;
            if (DIAG) {
                const double pd = (double)pv, gd = (double)g;
                dacc->p2 = fma(pd, pd, dacc->p2);
                dacc->g1 += fabs(gd);
                dacc->g2 = fma(gd, gd, dacc->g2);
            }
        }
        acc += (double)fabsf(pv);
        const unsigned w = __ballot_sync(kFull, valid && pv < 0.f);
        if (lane == 0) a.words[t.word + r] = w;
    }
    return acc;
}

// grid.x = chunks, grid.y = workers stepped by this launch (1 for ef_worker_step).
// Four CTAs per SM (64 registers) for the plain form: the launch-bound layouts need all CTAs of
// the M workers resident at once (flat 2^20, M = 2: 512 CTAs on 148 SMs).
template <int U, bool DIAG>
__global__ void __launch_bounds__(kThreads, DIAG ? 3 : 4) ef_worker_kernel(const WorkerArgs a0) {
    pdl_trigger();
    WorkerArgs a = a0;
    {
        const long long wi = blockIdx.y;
        if (DIAG) {
            a.dpartials += wi * (3 * a.partial_stride);
            a.diag += wi * (4LL * a.scale_stride);
        }
        a.g += wi * a.g_stride;
        a.m += wi * a.state_stride;
        a.pb += wi * a.state_stride;
        a.words += wi * a.word_stride;
        a.partials += wi * a.partial_stride;
        a.scale_out += wi * a.scale_stride;
        a.rscale += wi * a.scale_stride;
        a.tickets += wi * a.scale_stride;
    }
    const Tile t = chunk_of<U>(a.tiles[blockIdx.x / a.lim.tc], blockIdx.x % a.lim.tc);
    if (!work_item_ok(t, a.lim, 1024 * U)) return;
    const Block b = a.blocks[t.block];
    const bool alone = b.len <= 1024 * U;              // the block is this single chunk
    if (t.len <= 0 && alone) return;
    // word w of the layout is word w - b.word of its block: unit 1 + w - b.word of the block's message
    if (a.push) a.words = a.push[t.block] + 1 - b.word;
    double acc = 0.0;
    DiagAcc dacc;
    if (t.len <= 0) pdl_wait();
    if (t.len > 0) {
        const float sp = a.rscale[t.block];
        if ((t.start & 3) != 0)
            acc = worker_rows_scalar<DIAG>(a, t, sp, &dacc);
        else if (t.len == 1024 * U)
            acc = worker_rows<U, true, DIAG>(a, t, sp, &dacc);
        else
            acc = worker_rows<U, false, DIAG>(a, t, sp, &dacc);
    }
    if (DIAG)
        finish_block_diag(acc, dacc, blockIdx.x, alone, t.block, b.len, a.partials, a.dpartials,
                          a.partial_stride, a.diag, a.scale_out, a.rscale, a.push);
    else
        finish_block(acc, blockIdx.x, 0, alone, (unsigned)(b.tile_count * a.lim.tc), t.block,
                     a.blocks, a.partials, a.tickets, a.scale_out, a.rscale, a.fused, a.lim.tc, a.push);
}

// ------------------------------------------------------------------ server kernel
// a_j = sum over ascending i of (bit_i ? -c_i : +c_i), c_i = fl(scale_{i,b} / M), the first
// term taken as is (Algorithm 4, server line: (1/M) sum_i Delta_{t,i}).
//
// For M <= 16 the sum over the first min(M, 6) workers is tabulated once per CTA in shared
// memory (each entry is the same chain of fp32 additions, so the table is exact) and the
// remaining workers are added to the looked-up value directly, in order.  An element then costs one
// lookup plus at most two additions instead of M dependent additions with 2 bit operations
// each.  The table has at most 64 entries and is stored 32 times, entry e of copy l at word
// 32*e + l, so that lane l always reads bank l: the lookups are free of bank conflicts.
//
// Building the table index without per-worker work in every lane: the 8 lanes that share a
// packed word each load the word of ONE worker per group of 8 workers (lane q -> worker
// kLaneWorker(q) of the group; M > 8 uses two groups, i.e. two words and two transposes).  Seen as an
// 8x8 matrix of nibbles (row = lane that loaded it, column = lane whose 4 elements the nibble
// belongs to), a three-stage butterfly over the lanes (xor 4: half-words, xor 2: bytes, xor 1:
// nibbles) transposes it, so lane r ends with N = the 8 nibbles for its own 4 elements.  Two
// delta swaps of the bit-index (4 <-> 1, 3 <-> 0) then turn N into R, whose byte k holds the 8
// sign bits of element k; the data loaded by lane q lands at bit kLaneWorker(q), i.e. worker w
// sits at bit w.
constexpr int kMaxLutWorkers = 16;      // workers the table path handles (two lane groups)
constexpr int kLutWorkers = 6;        // workers covered by the replicated table (7 would cost a CTA per SM)
constexpr int kLutCopies = 32;        // one copy per lane

__host__ __device__ constexpr int kLaneWorker(int q) {
    return 4 * (q & 1) + 2 * ((q >> 2) & 1) + ((q >> 1) & 1);
}
__host__ __device__ constexpr int kLutEntries(int M) { return 1 << (M < kLutWorkers ? M : kLutWorkers); }
// M > 8 (two lane groups): ONE table, not replicated, over the first min(M, 10 or 11) workers, indexed by
// the element's sign byte of workers 0-7 and the low bits of its sign byte of workers 8-15.  Its
// lookups do collide in the banks (about 3.4 lanes per bank on random indices), which is still
// far cheaper than three instructions per element for each worker added outside a table.
// The table size is set by occupancy: the kernel is latency-bound and loses a third of its rate
// at three CTAs per SM instead of four, so ring + table must stay within a quarter of the SM's
// shared memory: 11 workers (8 KB) next to the bulk-staged ring for M <= 15, 10 (4 KB) next to
// the slightly larger per-thread ring and for M = 16.
__host__ __device__ constexpr int kWideLutWorkers(int M, bool bulk) { return (bulk && M <= 15) ? 11 : 10; }
__host__ __device__ constexpr int kWideLutBits(int M, bool bulk) {
    return M < kWideLutWorkers(M, bulk) ? M : kWideLutWorkers(M, bulk);
}
__host__ __device__ constexpr bool kUseWideLut(int M) { return M > 8; }
// floats of static shared memory the table path needs
__host__ __device__ constexpr int kLutFloats(int M, bool bulk) {
    return kUseWideLut(M) ? (1 << kWideLutBits(M, bulk)) : kLutEntries(M) * kLutCopies;
}

__device__ __forceinline__ void build_scaled(const ServerArgs& a, const Tile& t, int M, float* s_c) {
    if (a.fused_in) {
        const long long unit = message_unit(a.blocks[t.block].word, t.block) - a.msg_base;
        for (int i = threadIdx.x; i < M; i += kThreads)
            s_c[i] = __fdiv_rn(__uint_as_float(__ldg(a.wwords + (long long)i * a.wstride + unit)), (float)M);
    } else {
        for (int i = threadIdx.x; i < M; i += kThreads)
            s_c[i] = __fdiv_rn(a.wscales[(long long)i * a.sstride + t.block], (float)M);
    }
}

// Where the packed words of tile t start in worker 0's buffer (plain layout, or a fused message).
__device__ __forceinline__ const uint32_t* tile_words(const ServerArgs& a, const Tile& t) {
    return a.wwords + (a.fused_in ? message_unit(t.word, t.block) + 1 - a.msg_base : t.word);
}

// s_base[idx] = (+-c_0) +- c_1 ... +- c_{T-1}, bit i of idx set = worker i negative, T = min(M, 6);
// then every entry is written once per copy.  Ends with a barrier.
template <int MT>
__device__ __forceinline__ void build_lut(const float* s_c, float* s_base, float* s_lut) {
    constexpr int T = MT < kLutWorkers ? MT : kLutWorkers;
    if (threadIdx.x < (1 << T)) {
        const int idx = threadIdx.x;
        float v = (idx & 1) ? -s_c[0] : s_c[0];
#pragma unroll
        for (int i = 1; i < T; ++i) v = __fadd_rn(v, ((idx >> i) & 1) ? -s_c[i] : s_c[i]);
        s_base[idx] = v;
    }
    __syncthreads();
    for (int e = threadIdx.x; e < (1 << T) * kLutCopies; e += kThreads)
        s_lut[e] = s_base[e / kLutCopies];
    __syncthreads();
}

// Wide table (M > 8): entry idx = (+-c_0) +- c_1 ... +- c_{T-1}, T = kWideLutBits, bit i of idx set =
// worker i negative; every entry is the same chain of fp32 additions as the direct evaluation.
// Built by doubling: thread k first forms entry k over the workers 0..7 (256 entries), then
// worker i = 8, 9, ... turns every entry e < 2^i (a sum over workers 0..i-1) into the two entries
// e (+c_i) and e + 2^i (-c_i): one addition per entry instead of T.  Ends with a barrier.
template <int MT, bool BULK>
__device__ __forceinline__ void build_wide_lut(const float* s_c, float* s_lut) {
    constexpr int T = kWideLutBits(MT, BULK);
    static_assert(T >= 8 && kThreads == 256, "the first level fills 256 entries, one per thread");
    {
        const int idx = threadIdx.x;
        float v = (idx & 1) ? -s_c[0] : s_c[0];
#pragma unroll
        for (int i = 1; i < 8; ++i) v = __fadd_rn(v, ((idx >> i) & 1) ? -s_c[i] : s_c[i]);
        s_lut[idx] = v;
    }
    __syncthreads();
#pragma unroll
    for (int i = 8; i < T; ++i) {
        const float ci = s_c[i];
        for (int e = threadIdx.x; e < (1 << i); e += kThreads) {
            const float v = s_lut[e];
            s_lut[e] = __fadd_rn(v, ci);
            s_lut[e + (1 << i)] = __fadd_rn(v, -ci);
        }
        __syncthreads();
    }
}

__device__ __forceinline__ unsigned delta_swap(unsigned x, int d, unsigned mask) {
    const unsigned t = ((x >> d) ^ x) & mask;
    return x ^ t ^ (t << d);
}

// Lane-dependent constants of the butterfly (q = lane & 7).
struct Butterfly {
    unsigned sel1, sel2, keep3;
    int rot3;
    __device__ __forceinline__ explicit Butterfly(int q)
        : sel1((q & 4) ? 0x3276u : 0x5410u), sel2((q & 2) ? 0x3715u : 0x6240u),
          keep3((q & 1) ? 0xF0F0F0F0u : 0x0F0F0F0Fu), rot3((q & 1) ? 28 : 4) {}
    // w: the packed word this lane loaded (worker kLaneWorker(q), or 0 if there is no such worker).
    // Returns R: bit 8k + i = sign bit of worker i for the lane's element k.
    __device__ __forceinline__ unsigned indices(unsigned w) const {
        unsigned x = w;
        x = __byte_perm(x, __shfl_xor_sync(kFull, x, 4), sel1);
        x = __byte_perm(x, __shfl_xor_sync(kFull, x, 2), sel2);
        const unsigned y = __shfl_xor_sync(kFull, x, 1);
        x = (x & keep3) | (__funnelshift_l(y, y, rot3) & ~keep3);
        x = delta_swap(x, 14, 0x0000CCCCu);
        return delta_swap(x, 7, 0x00AA00AAu);
    }
};

// Asynchronous global->shared copies (LDGSTS).  Every thread copies exactly the bytes it will
// read back itself, so completion is tracked per thread with wait_group and no barrier or
// flag wait is involved.
__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(
                     (unsigned)__cvta_generic_to_shared(smem)), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async4(void* smem, const void* gmem) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(
                     (unsigned)__cvta_generic_to_shared(smem)), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

constexpr int kServerStages = 2;

// ---- bulk staging (TMA, 1-D): one elected thread copies a whole chunk of ptilde (16 KB) and
// each worker's 128 packed words (512 B) into a shared-memory stage with cp.async.bulk and an
// mbarrier that counts the bytes; the other threads only wait.  Each copy has this CTA as its
// only destination, and only this GPU's own memory is read.  Every wait is bounded: when the limit runs out the kernel records
// kStatusWaitTimeout in the context's status word, waits (bounded again) for the copies it
// still has in flight, and ends.
constexpr unsigned kStatusWaitTimeout = 1u;
constexpr int kMbarWaitLimit = 1 << 22;          // try_wait attempts (each blocks for a while itself)
constexpr int kBulkWordStride = 1024 * 4 / 32 + 4;   // words per worker and stage: +4 keeps the
                                                     // eight workers a warp reads in different banks
__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, unsigned parity) {
    unsigned ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
                 " selp.u32 %0, 1, 0, p;\n}" : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0u;
}
__device__ __forceinline__ bool mbar_wait_bounded(unsigned long long* bar, unsigned parity) {
    for (int it = 0; it < kMbarWaitLimit; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, unsigned bytes,
                                          unsigned long long* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// Dynamic shared memory of the server kernel: staging ring, then M scaled scales.  A stage holds
// either, per thread, U float4 of ptilde and U words for each group of 8 workers (per-thread
// cp.async), or one chunk of ptilde in memory order and kBulkWordStride words per worker (bulk).
template <int U>
__host__ __device__ constexpr size_t server_stage_bytes(int M, bool bulk) {
    const size_t per_thread = (size_t)U * kThreads * (sizeof(float4) + ((M + 7) / 8) * sizeof(unsigned));
    const size_t bulk_bytes = (size_t)1024 * U * sizeof(float) + (size_t)M * kBulkWordStride * sizeof(unsigned);
    return ((bulk ? bulk_bytes : per_thread) + 127) / 128 * 128;
}
template <int U>
__host__ __device__ constexpr size_t server_ring_bytes(int M, bool bulk) {
    return (size_t)kServerStages * server_stage_bytes<U>(M, bulk);
}

// Table path: one CTA walks the chunks of its tile.  Full chunks are staged through a ring of
// kServerStages shared-memory slots filled two chunks ahead with cp.async, so loads stay in
// flight during the lookups without costing registers; a ragged last chunk is loaded directly.
//
// BULK: the stages are filled by thread 0 with cp.async.bulk instead (see above); `full` are the
// stages' mbarriers, `phase` their parities (bit s).
// Returns the thread's sum of |ptilde|; sets *failed when a bounded wait ran out.
template <int U, int MT, bool BULK>
__device__ __forceinline__ double server_tile_lut(const ServerArgs& a, const Tile& t, float sp,
                                                  unsigned char* ring, float* s_c, float* s_base,
                                                  float* s_lut, unsigned long long* full,
                                                  unsigned& phase, bool* failed, unsigned* signs = nullptr) {
    constexpr int kChunk = 1024 * U;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q = lane & 7;
    const int o0 = warp * (128 * U) + lane * 4;
    constexpr int G = (MT + 7) / 8;                // groups of 8 workers (lane q loads one of each)
    const int wq = kLaneWorker(q);                 // the worker (of every group) this lane loads
    const Butterfly bf(q);
    float* const pbase = a.pb + t.start + o0;
    bool has_w[G];
    const uint32_t* wbase[G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        has_w[g] = wq + 8 * g < MT;
        wbase[g] = tile_words(a, t) + (long long)(has_w[g] ? wq + 8 * g : 0) * a.wstride + (o0 >> 5);
    }
    const int nfull = t.len / kChunk;              // chunks staged through shared memory
    const int tail = t.len - nfull * kChunk;       // ragged rest (only at the end of a block)
    const char* lut = reinterpret_cast<const char*>(s_lut + lane);   // this lane's copy
    constexpr size_t kStage = server_stage_bytes<U>(MT, BULK);
    // per-thread staging: slot (stage s, row u) of this thread, consecutive threads 16 (4) bytes apart
    float4* const ring_p = reinterpret_cast<float4*>(ring) + threadIdx.x;
    unsigned* const ring_w =
        reinterpret_cast<unsigned*>(ring + (size_t)U * kThreads * sizeof(float4)) + threadIdx.x;
    constexpr int kStageP4 = (int)(kStage / sizeof(float4)), kStageW = (int)(kStage / sizeof(unsigned));
    double acc = 0.0;
    const bool rescale = a.ratio != 1.0f;
    // bit patterns of the scaled scales of the workers the table does not cover
    unsigned cdir[kMaxLutWorkers - kLutWorkers + 1] = {};

    auto issue_chunk = [&](int c) {
        if (c < nfull) {
            const int s = c % kServerStages;
            const float* pp = pbase + (long long)c * kChunk;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                cp_async16(ring_p + s * kStageP4 + u * kThreads, pp + u * 128);
#pragma unroll
                for (int g = 0; g < G; ++g)
                    if (has_w[g])
                        cp_async4(ring_w + s * kStageW + (u * G + g) * kThreads,
                                  wbase[g] + c * (kChunk / 32) + u * 4);
            }
        }
        cp_async_commit();                 // one (possibly empty) group per chunk index
    };
    // bulk staging, thread 0 only: chunk c of ptilde in memory order, then 128 words per worker
    auto issue_chunk_bulk = [&](int c) {
        const int s = c % kServerStages;
        unsigned char* stage = ring + s * kStage;
        mbar_expect_tx(&full[s], (unsigned)(kChunk * sizeof(float) + MT * (kChunk / 32) * sizeof(unsigned)));
        bulk_load(stage, a.pb + t.start + (long long)c * kChunk, kChunk * sizeof(float), &full[s]);
        const uint32_t* wsrc = tile_words(a, t) + c * (kChunk / 32);
        unsigned* wdst = reinterpret_cast<unsigned*>(stage + kChunk * sizeof(float));
#pragma unroll
        for (int i = 0; i < MT; ++i)
            bulk_load(wdst + i * kBulkWordStride, wsrc + (long long)i * a.wstride,
                      (kChunk / 32) * sizeof(unsigned), &full[s]);
    };
    // full_c: std::true_type for a whole chunk (no bounds checks), std::false_type for the tail
    auto compute_chunk = [&](auto full_c, int c, int clen, float (&p)[U][4], unsigned (&w)[U][G]) {
        constexpr bool full = decltype(full_c)::value;
        float* pp = pbase + (long long)c * kChunk;
        uint32_t* words = a.words + t.word + c * (kChunk / 32);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int o = o0 + u * 128;
            unsigned Rg[G];                 // Rg[g]: bit 8k + i = sign of worker 8g + i, element k
#pragma unroll
            for (int g = 0; g < G; ++g) Rg[g] = bf.indices(w[u][g]);
            const unsigned R = Rg[0];
            float avg[4];
            if constexpr (kUseWideLut(MT)) {
                // byte offset 4 * (byte k of R | low bits of byte k of Rg[1] << 8) in the one table
                constexpr int kT = kWideLutBits(MT, BULK);
                constexpr unsigned kHiMask = ((1u << (kT > 8 ? kT - 8 : 0)) - 1u) << 10;
                const unsigned R1 = Rg[G - 1];
                const char* wl = reinterpret_cast<const char*>(s_lut);
                avg[0] = *reinterpret_cast<const float*>(wl + (((R << 2) & 0x3FCu) | ((R1 << 10) & kHiMask)));
                avg[1] = *reinterpret_cast<const float*>(wl + (((R >> 6) & 0x3FCu) | ((R1 << 2) & kHiMask)));
                avg[2] = *reinterpret_cast<const float*>(wl + (((R >> 14) & 0x3FCu) | ((R1 >> 6) & kHiMask)));
                avg[3] = *reinterpret_cast<const float*>(wl + (((R >> 22) & 0x3FCu) | ((R1 >> 14) & kHiMask)));
            } else {
                // byte offset of entry (R_k & (entries-1)) in this lane's copy: 128 * index
                constexpr unsigned kIdxMask = (unsigned)(kLutEntries(MT) - 1) << 7;
                avg[0] = *reinterpret_cast<const float*>(lut + ((R << 7) & kIdxMask));
                avg[1] = *reinterpret_cast<const float*>(lut + ((R >> 1) & kIdxMask));
                avg[2] = *reinterpret_cast<const float*>(lut + ((R >> 9) & kIdxMask));
                avg[3] = *reinterpret_cast<const float*>(lut + ((R >> 17) & kIdxMask));
            }
            constexpr int kFirstDirect = kUseWideLut(MT) ? kWideLutBits(MT, BULK) : kLutWorkers;
#pragma unroll
            for (int wk = kFirstDirect; wk < MT; ++wk) {    // remaining workers follow in order
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    avg[k] = __fadd_rn(avg[k], __uint_as_float(
                        cdir[wk - kLutWorkers] ^
                        ((Rg[wk / 8] << (31 - (wk % 8) - 8 * k)) & 0x80000000u)));
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                float pv = corrected_vector(a.ratio, rescale, residual_of(p[u][k], sp), avg[k]);   // ptilde_t
                if (!full && o + k >= clen) pv = 0.f;
                p[u][k] = pv;
            }
            const unsigned nib = sign_nibble(p[u]);
            if (signs) *signs |= nib << (4 * u);         // one-chunk tiles only: the caller keeps the signs
            acc += abs_sum4(p[u]);
            const unsigned word = pack_nibbles(nib, lane);
            store4(pp + u * 128, o, clen, full, p[u]);
            if (q == 0 && (full || o < clen)) words[o >> 5] = word;
        }
    };

    float p[U][4];
    unsigned w[U][G];
    if (BULK) {
        if (threadIdx.x == 0) {
            fence_proxy_async();                 // the stages were last read through ordinary loads
            for (int c = 0; c < kServerStages && c < nfull; ++c) issue_chunk_bulk(c);
        }
    } else {
#pragma unroll
        for (int c = 0; c < kServerStages - 1; ++c) issue_chunk(c);   // in flight while the table is built
    }
    build_scaled(a, t, MT, s_c);
    __syncthreads();
    if constexpr (kUseWideLut(MT)) build_wide_lut<MT, BULK>(s_c, s_lut);
    else build_lut<MT>(s_c, s_base, s_lut);
#pragma unroll
    for (int wk = kLutWorkers; wk < MT; ++wk) cdir[wk - kLutWorkers] = __float_as_uint(s_c[wk]);
    for (int c = 0; c < nfull; ++c) {
        const int s = c % kServerStages;
        if (BULK) {
            const bool ok = mbar_wait_bounded(&full[s], (phase >> s) & 1u);
            phase ^= 1u << s;
            const float4* sp4 = reinterpret_cast<const float4*>(ring + s * kStage) + warp * (32 * U) + lane;
            const unsigned* sw = reinterpret_cast<const unsigned*>(ring + s * kStage + kChunk * sizeof(float)) +
                                 warp * (4 * U) + (lane >> 3);
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const float4 v = sp4[u * 32];
                p[u][0] = v.x; p[u][1] = v.y; p[u][2] = v.z; p[u][3] = v.w;
#pragma unroll
                for (int g = 0; g < G; ++g)
                    w[u][g] = has_w[g] ? sw[(wq + 8 * g) * kBulkWordStride + u * 4] : 0u;
            }
            // everyone has read stage s (it may be refilled) -- and did every wait succeed?
            if (__syncthreads_or(!ok)) {
                if (threadIdx.x == 0) atomicOr(a.status, kStatusWaitTimeout);
                // chunks c+1 .. are still in flight into the other stages: let them land
                for (int c2 = c + 1; c2 < nfull && c2 < c + kServerStages; ++c2) {
                    const int s2 = c2 % kServerStages;
                    mbar_wait_bounded(&full[s2], (phase >> s2) & 1u);
                    phase ^= 1u << s2;
                }
                *failed = true;
                return acc;
            }
            if (threadIdx.x == 0 && c + kServerStages < nfull) {
                fence_proxy_async();
                issue_chunk_bulk(c + kServerStages);
            }
        } else {
            issue_chunk(c + kServerStages - 1);      // reuses the slot this thread consumed at c - 1
            cp_async_wait<kServerStages - 1>();      // only the groups after chunk c may be in flight
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const float4 v = ring_p[s * kStageP4 + u * kThreads];
                p[u][0] = v.x; p[u][1] = v.y; p[u][2] = v.z; p[u][3] = v.w;
#pragma unroll
                for (int g = 0; g < G; ++g)
                    w[u][g] = has_w[g] ? ring_w[s * kStageW + (u * G + g) * kThreads] : 0u;
            }
        }
        compute_chunk(std::true_type{}, c, kChunk, p, w);
    }
    if (tail > 0) {
        const float* pp = pbase + (long long)nfull * kChunk;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int o = o0 + u * 128;
            load4(pp + u * 128, o, tail, false, p[u]);
#pragma unroll
            for (int g = 0; g < G; ++g)
                w[u][g] = (has_w[g] && (o & ~31) < tail)
                              ? __ldg(wbase[g] + nfull * (kChunk / 32) + u * 4) : 0u;
        }
        compute_chunk(std::false_type{}, nfull, tail, p, w);
    }
    if (!BULK) cp_async_wait<0>();
    return acc;
}

// Direct evaluation for any M.
__device__ __forceinline__ void average4(const ServerArgs& a, const float* s_c, const uint32_t* wp,
                                         int sh, float (&avg)[4]) {
#pragma unroll 4
    for (int i = 0; i < a.M; ++i) {
        const unsigned nib = __ldg(wp + (long long)i * a.wstride) >> sh;
        const unsigned cb = __float_as_uint(s_c[i]);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float v = __uint_as_float(cb ^ ((nib << (31 - k)) & 0x80000000u));
            avg[k] = (i == 0) ? v : __fadd_rn(avg[k], v);
        }
    }
}

// signs (optional): bit 4u + k = sign bit of this thread's element k of row u.
template <int U>
__device__ __forceinline__ double server_rows(const ServerArgs& a, const Tile& t, float sp,
                                              const float* s_c, unsigned* signs = nullptr) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int o0 = warp * (128 * U) + lane * 4;
    const int sh = (lane & 7) * 4;
    const bool full = t.len == 1024 * U;
    float* pp = a.pb + t.start + o0;
    float p[U][4];
#pragma unroll
    for (int u = 0; u < U; ++u) load4(pp + u * 128, o0 + u * 128, t.len, full, p[u]);
    double acc = 0.0;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int o = o0 + u * 128;
        float avg[4] = {0.f, 0.f, 0.f, 0.f};
        if (full || o < t.len) average4(a, s_c, tile_words(a, t) + (o >> 5), sh, avg);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            float pv = corrected_vector(a.ratio, a.ratio != 1.0f, residual_of(p[u][k], sp), avg[k]);   // ptilde_t
            if (!full && o + k >= t.len) pv = 0.f;
            p[u][k] = pv;
        }
        const unsigned nib = sign_nibble(p[u]);
        if (signs) *signs |= nib << (4 * u);
        acc += abs_sum4(p[u]);
        const unsigned w = pack_nibbles(nib, lane);
        store4(pp + u * 128, o, t.len, full, p[u]);
        if ((lane & 7) == 0 && (full || o < t.len)) a.words[t.word + (o >> 5)] = w;
    }
    return acc;
}

// Any alignment, any M, any tile length.  signs (optional): bit n = sign bit of the element this
// thread handled in its n-th row (row warp + n * kWarps).
__device__ __forceinline__ double server_rows_scalar(const ServerArgs& a, const Tile& t, float sp,
                                                     const float* s_c, unsigned* signs = nullptr) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rows = (t.len + 31) >> 5;
    double acc = 0.0;
    for (int r = warp; r < rows; r += kWarps) {
        const int o = r * 32 + lane;
        const bool valid = o < t.len;
        float pv = 0.f;
        if (valid) {
            float avg = 0.f;
            for (int i = 0; i < a.M; ++i) {
                const unsigned w = __ldg(tile_words(a, t) + (long long)i * a.wstride + r);
                const float v = ((w >> lane) & 1u) ? -s_c[i] : s_c[i];
                avg = (i == 0) ? v : __fadd_rn(avg, v);
            }
            const long long j = t.start + o;
            pv = corrected_vector(a.ratio, a.ratio != 1.0f, residual_of(a.pb[j], sp), avg);
            a.pb[j] = pv;
        }
        acc += (double)fabsf(pv);
        const unsigned w = __ballot_sync(kFull, valid && pv < 0.f);
        if (signs) *signs |= ((w >> lane) & 1u) << ((r - warp) / kWarps);
        if (lane == 0) a.words[t.word + r] = w;
    }
    return acc;
}

// One tile per CTA.  MT = number of workers when 1 <= M <= 16 (table path), 0 for any other M.
// BULK (table path, layouts whose packed words are 16-byte aligned per chunk only): stages are
// filled with cp.async.bulk.
template <int U, int MT, bool BULK>
__global__ void __launch_bounds__(kThreads) ef_server_kernel(const ServerArgs a) {
    // dynamic shared memory: [staging ring (table path only)] [M scaled worker scales]
    extern __shared__ __align__(128) unsigned char s_dyn[];
    float* s_c = reinterpret_cast<float*>(s_dyn + (MT > 0 ? server_ring_bytes<U>(MT, BULK) : 0));
    __shared__ float s_base[(MT > 0 && !kUseWideLut(MT)) ? kLutEntries(MT) : 1];
    __shared__ float s_lut[MT > 0 ? kLutFloats(MT, BULK) : 1];
    __shared__ unsigned long long s_full[kServerStages];
    unsigned phase = 0u;
    bool failed = false;
    if (BULK) {
        if (threadIdx.x == 0) {
            for (int s = 0; s < kServerStages; ++s) mbar_init(&s_full[s], 1u);
            mbar_fence_init();
        }
        __syncthreads();
    }
    pdl_enter();                       // the barrier set-up above overlaps the previous kernel's tail
    const Tile t = a.tiles[blockIdx.x + a.tile0];
    if (!work_item_ok(t, a.lim, a.lim.tc * 1024 * U)) return;
    const float sp = a.rscale[t.block];
    double acc = 0.0;
    if (MT > 0 && (t.start & 3) == 0) {
        acc = server_tile_lut<U, (MT > 0 ? MT : 1), BULK>(a, t, sp, s_dyn, s_c, s_base, s_lut, s_full,
                                                          phase, &failed);
        if (BULK && failed) return;
    } else {
        build_scaled(a, t, a.M, s_c);
        __syncthreads();
        if ((t.start & 3) != 0) {
            acc = server_rows_scalar(a, t, sp, s_c);
        } else {
            for (int c = 0; c * (1024 * U) < t.len; ++c)
                acc += server_rows<U>(a, chunk_of<U>(t, c), sp, s_c);
        }
    }
    const Block b = a.blocks[t.block];
    finish_block(acc, (long long)(blockIdx.x + a.tile0) * a.lim.tc, a.lim.tc - 1, b.len <= 1024 * U,
                 (unsigned)b.tile_count, t.block, a.blocks, a.partials, a.tickets, a.scale_out,
                 a.rscale, a.fused, a.lim.tc);
}

// ------------------------------------------------------------------ server lines + update, one launch
// Layouts of few chunks are bound by the latency of their short kernels, not by memory.  When no
// block spans more than kClusterCtas chunks, ef_server_step runs as ONE kernel launched in
// thread-block clusters: a cluster owns one block (CTA r takes chunk r; the rest of the cluster
// idles) or up to kClusterCtas single-chunk blocks.  A CTA keeps its chunk's sign bits and x values
// in registers; the CTAs of a block publish their partial L1 sums, meet at the cluster barrier
// (hardware, all CTAs of a cluster are co-scheduled: nothing polls memory), add the partial sums
// in the usual fixed order -- every CTA for itself, so the scale has the same bits everywhere and
// the same bits as in the two-kernel path -- and apply  x <- x - eta * stilde_b * sign(ptilde).
constexpr int kClusterCtas = 16;
constexpr int kClusterTileSync = 1;     // Tile::pad0 of a cluster work item: the cluster meets at its barrier

struct ServerUpdateArgs {
    ServerArgs s;          // plain inputs (the context's own worker words and scales), whole layout
    const Tile* ctiles;    // one work item per CTA in cluster order: len 0 = idle, pad0 = flags,
                           // pad1 = index of the tile in the ordinary tile table (its partial-sum slot)
    float* x;
    float eta;
};

__device__ __forceinline__ void cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

template <int U, int MT>
__global__ void __launch_bounds__(kThreads) ef_server_update_kernel(const ServerUpdateArgs aa) {
    extern __shared__ __align__(128) unsigned char s_dyn[];
    float* s_c = reinterpret_cast<float*>(s_dyn + (MT > 0 ? server_ring_bytes<U>(MT, false) : 0));
    __shared__ float s_base[(MT > 0 && !kUseWideLut(MT)) ? kLutEntries(MT) : 1];
    __shared__ float s_lut[MT > 0 ? kLutFloats(MT, false) : 1];
    __shared__ unsigned long long s_full[kServerStages];      // unused: the stages are filled per thread
    __shared__ double s_sum[kWarps];
    __shared__ float s_scale;
    const ServerArgs& a = aa.s;
    pdl_trigger();
    const Tile t = aa.ctiles[blockIdx.x];
    const bool meet = (t.pad0 & kClusterTileSync) != 0;
    // An idle CTA, or (checked build) one whose work item is refused, only keeps its appointment.
    if (t.len <= 0 || !work_item_ok(t, a.lim, 1024 * U)) {
        pdl_wait();
        if (meet) cluster_barrier();
        return;
    }
    const float sp = a.rscale[t.block];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool vec = (t.start & 3) == 0;
    const bool full = t.len == 1024 * U;
    const int o0 = warp * (128 * U) + lane * 4;
    float x[U][4];
    if (vec) {                                 // needed at the very end only: the loads overlap everything
#pragma unroll
        for (int u = 0; u < U; ++u) load4(aa.x + t.start + o0 + u * 128, o0 + u * 128, t.len, full, x[u]);
    }
    pdl_wait();
    unsigned signs = 0u;
    double acc;
    if (MT > 0 && vec) {
        unsigned phase = 0u;
        bool failed = false;
        acc = server_tile_lut<U, (MT > 0 ? MT : 1), false>(a, t, sp, s_dyn, s_c, s_base, s_lut, s_full, phase,
                                                            &failed, &signs);
    } else {
        build_scaled(a, t, a.M, s_c);
        __syncthreads();
        acc = vec ? server_rows<U>(a, t, sp, s_c, &signs) : server_rows_scalar(a, t, sp, s_c, &signs);
    }
    const Block b = a.blocks[t.block];
    double S = cta_sum(acc, s_sum);            // valid in thread 0
    if (meet) {
        if (threadIdx.x == 0) a.partials[t.pad1] = S;
        cluster_barrier();                     // every CTA of the block has published its sum
        S = sum_slots(b, a.partials, s_sum, 1);
    }
    if (threadIdx.x == 0) {
        const float s = (float)(S / (double)b.div);
        s_scale = s;
        if (t.start == b.start) {              // the block's first chunk records the scale
            a.scale_out[t.block] = s;
            a.rscale[t.block] = s;             // every CTA of the block read the old one before the barrier
        }
    }
    __syncthreads();
    const float step = __fmul_rn(aa.eta, s_scale);
    if (vec) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
#pragma unroll
            for (int k = 0; k < 4; ++k)
                x[u][k] = __fsub_rn(x[u][k], __uint_as_float(__float_as_uint(step) ^
                                                             ((signs << (31 - 4 * u - k)) & 0x80000000u)));
            store4(aa.x + t.start + o0 + u * 128, o0 + u * 128, t.len, full, x[u]);
        }
    } else {
        const int rows = (t.len + 31) >> 5;
        for (int r = warp, n = 0; r < rows; r += kWarps, ++n) {
            const int o = r * 32 + lane;
            if (o < t.len) {
                const long long j = t.start + o;
                aa.x[j] = __fsub_rn(aa.x[j], ((signs >> n) & 1u) ? -step : step);
            }
        }
    }
}

// ------------------------------------------------------------------ parameter update
// x_{t+1,j} = x_{t,j} - eta * stilde_b * sign(ptilde_j)  (Algorithm 4, worker line after the pull)
// One tile per CTA; chunk c+1 is loaded into a second register set while chunk c is updated, so
// the tile descriptor's latency is paid once per tile and loads stay in flight.
//
// DECAY adds the weight-decay side path of Appendix A, which is not compressed:
//   mtilde_t = mu mtilde_{t-1} + lambda x_t;  x_{t+1} = x_t - eta (Deltatilde_t + mu mtilde_t + lambda x_t),
// evaluated as wd = fl(lambda x); mtilde = fma(mu, mtilde, wd); v = fma(mu, mtilde, wd);
// x = fl(fl(x -+ eta s_b) - fl(eta v)).
template <bool DECAY>
__device__ __forceinline__ float apply_one(const ApplyArgs& a, float x, float signed_step, float* mt) {
    const float xs = __fsub_rn(x, signed_step);
    if (!DECAY) return xs;
    const float wd = __fmul_rn(a.lambda, x);
    *mt = __fmaf_rn(a.mu, *mt, wd);
    const float v = __fmaf_rn(a.mu, *mt, wd);
    return __fsub_rn(xs, __fmul_rn(a.eta, v));
}

template <int U, bool DECAY>
__global__ void __launch_bounds__(kThreads) ef_apply_kernel(const ApplyArgs a) {
    constexpr int kChunk = 1024 * U;
    pdl_enter();
    const Tile t = a.tiles[blockIdx.x + a.tile0];
    if (!work_item_ok(t, a.lim, a.lim.tc * kChunk)) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // packed words of this tile and the block's scale: plain layout or a fused message
    const uint32_t* const twords =
        a.words + (a.fused_in ? message_unit(t.word, t.block) + 1 - a.msg_base : t.word);
    const float* const scale_ptr =
        a.fused_in ? reinterpret_cast<const float*>(a.words) +
                         (message_unit(a.blocks[t.block].word, t.block) - a.msg_base)
                   : a.scales + t.block;
    // The block's scale: read, or formed here from the block's partial sums (uniform per CTA).
    auto block_scale = [&]() -> float {
        if (a.self_scale_tiles > 0) {
            const Block b = a.blocks[t.block];
            if (b.len > kChunk && b.tile_count <= a.self_scale_tiles) {
                __shared__ double s_sum[kWarps];
                __shared__ float s_scale;
                const double S = sum_slots(b, a.partials, s_sum, a.lim.tc);     // valid in thread 0
                if (threadIdx.x == 0) {
                    const float s = (float)(S / (double)b.div);
                    s_scale = s;
                    if (t.start == b.start) {
                        a.scale_out[t.block] = s;
                        a.rscale[t.block] = s;
                    }
                }
                __syncthreads();
                return s_scale;
            }
        }
        return *scale_ptr;
    };
    if ((t.start & 3) != 0) {
        const float step = __fmul_rn(a.eta, block_scale());
        const int rows = (t.len + 31) >> 5;
        for (int r = warp; r < rows; r += kWarps) {
            const int o = r * 32 + lane;
            if (o < t.len) {
                const unsigned w = __ldg(twords + r);
                const long long j = t.start + o;
                float mt = DECAY ? a.mt[j] : 0.f;
                a.x[j] = apply_one<DECAY>(a, a.x[j], ((w >> lane) & 1u) ? -step : step, &mt);
                if (DECAY) a.mt[j] = mt;
            }
        }
        return;
    }
    const int o0 = warp * (128 * U) + lane * 4;
    const int sh = (lane & 7) * 4;
    float* const xbase = a.x + t.start + o0;
    float* const mbase = DECAY ? a.mt + t.start + o0 : nullptr;
    const uint32_t* const wbase = twords + (o0 >> 5);
    const int nchunks = (t.len + kChunk - 1) / kChunk;
    constexpr int UM = DECAY ? U : 1;      // the decay momentum is only held when it is used

    auto load_chunk = [&](int c, float (&x)[U][4], float (&mt)[UM][4], unsigned (&nib)[U]) {
        const int clen = min(kChunk, t.len - c * kChunk);
        const bool full = clen == kChunk;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int o = o0 + u * 128;
            load4(xbase + (long long)c * kChunk + u * 128, o, clen, full, x[u]);
            if (DECAY) load4(mbase + (long long)c * kChunk + u * 128, o, clen, full, mt[DECAY ? u : 0]);
            nib[u] = (full || o < clen) ? __ldg(wbase + c * (kChunk / 32) + u * 4) : 0u;
        }
    };
    float step = 0.f;
    auto update_chunk = [&](int c, float (&x)[U][4], float (&mt)[UM][4], unsigned (&nib)[U]) {
        const int clen = min(kChunk, t.len - c * kChunk);
        const bool full = clen == kChunk;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const unsigned n = nib[u] >> sh;
#pragma unroll
            for (int k = 0; k < 4; ++k) {   // x - step*sign: subtract step with the sign bit flipped in
                const float signed_step =
                    __uint_as_float(__float_as_uint(step) ^ ((n << (31 - k)) & 0x80000000u));
                x[u][k] = apply_one<DECAY>(a, x[u][k], signed_step, &mt[DECAY ? u : 0][k]);
            }
            store4(xbase + (long long)c * kChunk + u * 128, o0 + u * 128, clen, full, x[u]);
            if (DECAY)
                store4(mbase + (long long)c * kChunk + u * 128, o0 + u * 128, clen, full, mt[DECAY ? u : 0]);
        }
    };

    float xA[U][4], xB[U][4], mA[UM][4], mB[UM][4];
    unsigned nA[U], nB[U];
    load_chunk(0, xA, mA, nA);
    step = __fmul_rn(a.eta, block_scale());            // its latency overlaps the first loads
    for (int c = 0; c < nchunks; c += 2) {
        if (c + 1 < nchunks) load_chunk(c + 1, xB, mB, nB);
        update_chunk(c, xA, mA, nA);
        if (c + 1 < nchunks) {
            if (c + 2 < nchunks) load_chunk(c + 2, xA, mA, nA);
            update_chunk(c + 1, xB, mB, nB);
        }
    }
}

// ------------------------------------------------------------------ residual materialisation
// dst_j = p_j - s_b * sign(p_j): the residual e_{t+1} in its plain form (tests, checkpoints).
// One tile per CTA.
static __global__ void __launch_bounds__(kThreads) ef_residual_kernel(const ResidualArgs a) {
    pdl_enter();
    const Tile t = a.tiles[blockIdx.x];
    if (!work_item_ok(t, a.lim, 1 << 30)) return;
    const float s = a.rscale[t.block];
    for (int o = threadIdx.x; o < t.len; o += kThreads)
        a.dst[t.start + o] = residual_of(a.pb[t.start + o], s);
}

// Fused message of a block range: dst gets, block after block, [scale | packed words].
// One tile per CTA (a tile has at most kTileChunks*1024*U/32 words).
constexpr int kMaxPackTargets = 64;
struct PackArgs {
    const uint32_t* words;
    const float* scales;
    uint32_t* dst[kMaxPackTargets];   // n_dst copies of the message are written (own or peer memory)
    int n_dst;
    const Tile* tiles;
    const Block* blocks;
    int tile0;
    long long msg_base;
    DebugLimits lim;
};
static __global__ void __launch_bounds__(kThreads) ef_pack_kernel(const PackArgs a) {
    pdl_enter();
    const Tile t = a.tiles[blockIdx.x + a.tile0];
    if (!work_item_ok(t, a.lim, 1 << 30)) return;
    const Block b = a.blocks[t.block];
    const long long unit = message_unit(t.word, t.block) + 1 - a.msg_base;
    const int nwords = (t.len + 31) >> 5;
    for (int k = threadIdx.x; k < nwords; k += kThreads) {
        const uint32_t w = a.words[t.word + k];
        for (int q = 0; q < a.n_dst; ++q) a.dst[q][unit + k] = w;
    }
    if (threadIdx.x == 0 && t.start == b.start) {
        const uint32_t s = __float_as_uint(a.scales[t.block]);
        for (int q = 0; q < a.n_dst; ++q) a.dst[q][message_unit(b.word, t.block) - a.msg_base] = s;
    }
}

// Cut blocks: dst[b] = the piece's fp64 sum of |p| (0 for blocks held whole), and the scale of
// such a block from the sum over all pieces.  One thread per block.
static __global__ void __launch_bounds__(kThreads) ef_block_sums_kernel(const Block* __restrict__ blocks,
                                                                        const double* __restrict__ partials,
                                                                        int tc, int B, double* __restrict__ dst) {
    pdl_enter();
    const int b = blockIdx.x * kThreads + threadIdx.x;
    if (b < B) dst[b] = blocks[b].partial ? partials[(long long)blocks[b].tile_begin * tc] : 0.0;
}
static __global__ void __launch_bounds__(kThreads) ef_complete_scales_kernel(const Block* __restrict__ blocks,
                                                                             const double* __restrict__ totals,
                                                                             int B, float* __restrict__ scale_out,
                                                                             float* __restrict__ rscale) {
    pdl_wait();                        // writes a worker's scales: no early trigger (see pdl_wait above)
    const int b = blockIdx.x * kThreads + threadIdx.x;
    if (b < B && blocks[b].partial) {
        const float s = (float)(totals[b] / (double)blocks[b].div);
        scale_out[b] = s;
        rscale[b] = s;
    }
}

// Import of a residual (ef_set_state): adding +0 maps -0 to +0 and changes nothing else, which
// keeps the "no -0 in a residual buffer" invariant of the sign-bit tests above.
static __global__ void __launch_bounds__(kThreads) ef_import_kernel(const float* __restrict__ src,
                                                             float* __restrict__ dst, long long n) {
    pdl_wait();                        // writes a worker's state: no early trigger (see pdl_wait above)
    for (long long j = blockIdx.x * (long long)kThreads + threadIdx.x; j < n;
         j += (long long)gridDim.x * kThreads)
        dst[j] = __fadd_rn(src[j], 0.0f);
}

}  // namespace efk
