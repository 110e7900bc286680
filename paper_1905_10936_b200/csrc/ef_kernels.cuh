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
// (p_{t,j} < 0), which is exactly the bit that was sent.  Each launch is therefore one
// streaming pass: read g, m, p_prev; write m, p; write 1 bit per element; plus one fp64
// partial sum per tile.  The partial sums of a block are added in a fixed order, either by a
// tiny follow-up kernel (large grids: the kernel boundary orders the partial sums for free,
// whereas a device-wide fence in every CTA costs about 8% of the streaming rate) or, for small
// launch-bound grids, by the last CTA to finish the block (one atomic ticket, no waiting).
//
// Arithmetic is IEEE binary32 with explicit round-to-nearest intrinsics in a fixed order so
// that results do not depend on compiler contraction; block sums are binary64.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

namespace efk {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr unsigned kFull = 0xffffffffu;

// A tile is a run of at most 1024*U consecutive elements inside one block.  Tiles of a block
// start at multiples of the tile length from the block's first element, so a tile always
// starts on a packed-word boundary.
struct __align__(16) Tile {
    long long start;   // flat index of the first element
    long long word;    // index of the first packed word
    int len;           // elements in this tile (1 .. 1024*U)
    int block;         // block id
    int pad0, pad1;
};
static_assert(sizeof(Tile) == 32, "Tile must be 32 bytes");

struct __align__(16) Block {
    long long start;   // flat index of the first element
    long long len;     // d_b
    long long word;    // index of the block's first packed word
    int tile_begin;    // first tile of this block
    int tile_count;    // number of tiles
};
static_assert(sizeof(Block) == 32, "Block must be 32 bytes");

struct WorkerArgs {
    const float* g;        // gradient g_{t,i}
    float* m;              // momentum m_i (in/out)
    float* pb;             // deferred residual: p_{t-1,i} in, p_{t,i} out
    uint32_t* words;       // packed signs of p_{t,i}
    float* scale_out;      // per-block scales of the message
    float* rscale;         // per-block scale that belongs to pb (in: t-1, out: t)
    double* partials;      // one fp64 partial L1 sum per tile
    unsigned* tickets;     // one arrival counter per block (0 between launches)
    const Tile* tiles;
    const Block* blocks;
    float mu;
    int fused;             // 1: last CTA of a block finalises its scale; 0: ef_scale_kernel does
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
};

struct ScaleArgs {
    const double* partials;
    const Block* blocks;
    const int* multi;        // ids of the blocks that span more than one tile
    float* scale_out;
    float* rscale;
};

struct ApplyArgs {
    float* x;
    const uint32_t* words;   // server packed signs
    const float* scales;     // server scales
    const Tile* tiles;
    float eta;
};

struct ResidualArgs {
    const float* pb;
    const float* rscale;
    float* dst;
    const Tile* tiles;
};

// ------------------------------------------------------------------ small helpers
// Streaming accesses go through L2 only (.cg): every byte is used once per launch, and on
// B200 this measured about 2% faster than the evict-first (.cs) forms.
__device__ __forceinline__ float4 ld_stream(const float* p) {
    return __ldcg(reinterpret_cast<const float4*>(p));
}
__device__ __forceinline__ void st_stream(float* p, float4 v) {
    __stcg(reinterpret_cast<float4*>(p), v);
}

// e_{t+1,j} = p_{t,j} - s * sign(p_{t,j}) with sign(+-0) = +1 (Algorithm 4; Appendix A).
__device__ __forceinline__ float residual_of(float pb, float s) {
    return (pb < 0.f) ? __fadd_rn(pb, s) : __fsub_rn(pb, s);
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

// Adds the partial sums of block b in a fixed order (thread k takes tiles k, k+256, ...; then
// the CTA tree) and writes the scale s_b = ||p_b||_1 / d_b (Section 3.2).  Called by a whole CTA.
__device__ __forceinline__ void sum_partials_and_write(const Block& b, int block_id,
                                                       const double* __restrict__ partials,
                                                       float* __restrict__ scale_out,
                                                       float* __restrict__ rscale,
                                                       double* s_sum) {
    double v = 0.0;
    for (int k = threadIdx.x; k < b.tile_count; k += kThreads)
        v += __ldcg(&partials[b.tile_begin + k]);
    const double S = cta_sum(v, s_sum);
    if (threadIdx.x == 0) {
        const float s = (float)(S / (double)b.len);
        scale_out[block_id] = s;
        rscale[block_id] = s;
    }
}

// End of a tile: turns the tile's |p| sum into the block scale or a published partial sum.
// Single-tile blocks are finished directly.  For larger blocks the tile's partial sum is
// stored; if `fused`, the CTA that arrives last at the block's ticket also adds all partial
// sums (no CTA ever waits for another one), otherwise ef_scale_kernel does that after this
// launch.
__device__ __forceinline__ void finish_block(double acc, int tile_index, const Tile& t,
                                             const Block* __restrict__ blocks,
                                             double* __restrict__ partials,
                                             unsigned* __restrict__ tickets,
                                             float* __restrict__ scale_out,
                                             float* __restrict__ rscale, int fused) {
    __shared__ double s_sum[kWarps];
    __shared__ int s_last;
    const double S = cta_sum(acc, s_sum);
    if (threadIdx.x == 0) {
        const Block b = blocks[t.block];
        int last = 0;
        if (b.tile_count == 1) {
            const float s = (float)(S / (double)b.len);
            scale_out[t.block] = s;
            rscale[t.block] = s;
        } else {
            partials[tile_index] = S;
            if (fused) {
                __threadfence();
                const unsigned old = atomicAdd(&tickets[t.block], 1u);
                last = (old + 1u == (unsigned)b.tile_count);
            }
        }
        s_last = last;
    }
    if (!fused) return;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const Block b = blocks[t.block];
    sum_partials_and_write(b, t.block, partials, scale_out, rscale, s_sum);
    if (threadIdx.x == 0) tickets[t.block] = 0u;      // ready for the next launch
}

// Follow-up kernel of the non-fused mode: one CTA per multi-tile block.
__global__ void __launch_bounds__(kThreads) ef_scale_kernel(const ScaleArgs a) {
    __shared__ double s_sum[kWarps];
    const int block_id = a.multi[blockIdx.x];
    const Block b = a.blocks[block_id];
    sum_partials_and_write(b, block_id, a.partials, a.scale_out, a.rscale, s_sum);
}

// Packs the four sign bits each lane holds (nibble, element k in bit k) into 32-bit words:
// lanes 8q..8q+7 together hold 32 consecutive elements.  Returns the word in every lane of
// the group.
__device__ __forceinline__ unsigned pack_nibbles(unsigned nib, int lane) {
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

// ------------------------------------------------------------------ worker kernel
// One tile per CTA.  Warp w owns the 128*U consecutive elements starting at w*128*U; in row u
// lane l holds elements u*128 + 4l .. +3 (a 128-bit access, 512 contiguous bytes per warp).
template <int U, bool FULL>
__device__ __forceinline__ double worker_rows(const WorkerArgs& a, const Tile& t, float sp) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int o0 = warp * (128 * U) + lane * 4;
    const float* gp = a.g + t.start + o0;
    float* mp = a.m + t.start + o0;
    float* pp = a.pb + t.start + o0;
    float g[U][4], m[U][4], p[U][4];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        load4(gp + u * 128, o0 + u * 128, t.len, FULL, g[u]);
        load4(mp + u * 128, o0 + u * 128, t.len, FULL, m[u]);
        load4(pp + u * 128, o0 + u * 128, t.len, FULL, p[u]);
    }
    double acc = 0.0;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int o = o0 + u * 128;
        unsigned nib = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float e = residual_of(p[u][k], sp);                // e_{t,i}
            m[u][k] = __fmaf_rn(a.mu, m[u][k], g[u][k]);             // m_t = mu m_{t-1} + g
            const float v = __fmaf_rn(a.mu, m[u][k], g[u][k]);       // mu m_t + g
            float pv = __fadd_rn(v, e);                              // p_t
            if (!FULL && o + k >= t.len) pv = 0.f;
            p[u][k] = pv;
            nib |= (pv < 0.f ? 1u : 0u) << k;
        }
        acc += ((double)fabsf(p[u][0]) + (double)fabsf(p[u][1])) +
               ((double)fabsf(p[u][2]) + (double)fabsf(p[u][3]));
        const unsigned w = pack_nibbles(nib, lane);
        store4(mp + u * 128, o, t.len, FULL, m[u]);
        store4(pp + u * 128, o, t.len, FULL, p[u]);
        if ((lane & 7) == 0 && (FULL || o < t.len)) a.words[t.word + (o >> 5)] = w;
    }
    return acc;
}

// Fallback for tiles that do not start on a 16-byte boundary: 32-bit accesses, one ballot per
// 32 elements.
__device__ __forceinline__ double worker_rows_scalar(const WorkerArgs& a, const Tile& t, float sp) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rows = (t.len + 31) >> 5;
    double acc = 0.0;
    for (int r = warp; r < rows; r += kWarps) {
        const int o = r * 32 + lane;
        const bool valid = o < t.len;
        float pv = 0.f;
        if (valid) {
            const long long j = t.start + o;
            const float g = a.g[j];
            const float e = residual_of(a.pb[j], sp);
            const float m = __fmaf_rn(a.mu, a.m[j], g);
            pv = __fadd_rn(__fmaf_rn(a.mu, m, g), e);
            a.m[j] = m;
            a.pb[j] = pv;
        }
        acc += (double)fabsf(pv);
        const unsigned w = __ballot_sync(kFull, valid && pv < 0.f);
        if (lane == 0) a.words[t.word + r] = w;
    }
    return acc;
}

template <int U>
__global__ void __launch_bounds__(kThreads) ef_worker_kernel(const WorkerArgs a) {
    const Tile t = a.tiles[blockIdx.x];
    const float sp = a.rscale[t.block];
    double acc;
    if ((t.start & 3) != 0)
        acc = worker_rows_scalar(a, t, sp);
    else if (t.len == 1024 * U)
        acc = worker_rows<U, true>(a, t, sp);
    else
        acc = worker_rows<U, false>(a, t, sp);
    finish_block(acc, blockIdx.x, t, a.blocks, a.partials, a.tickets, a.scale_out, a.rscale, a.fused);
}

// ------------------------------------------------------------------ server kernel
// a_j = sum over ascending i of (bit_i ? -c_i : +c_i), c_i = fl(scale_{i,b} / M), the first
// term taken as is (Algorithm 4, server line: (1/M) sum_i Delta_{t,i}).
//
// For M <= 8 the 2^M possible values of a_j inside one block are tabulated once per CTA in
// shared memory (each entry is the same chain of fp32 additions, so the table is exact) and an
// element costs one lookup instead of M dependent additions with 2 bit operations each.  The
// index of element k of a lane is the byte k of R, where bit (8k + i) of R is worker i's sign
// bit: each worker's nibble n (its 4 sign bits for the lane's 4 elements) is spread with
// (n * 0x00204081) & 0x01010101, which moves bit k to bit 8k without carries, and shifted
// left by i.
constexpr int kMaxLutWorkers = 8;

__device__ __forceinline__ void build_scaled(const ServerArgs& a, int block, int M, float* s_c) {
    for (int i = threadIdx.x; i < M; i += kThreads)
        s_c[i] = __fdiv_rn(a.wscales[(long long)i * a.sstride + block], (float)M);
}

template <int MT>
__device__ __forceinline__ void build_lut(const float* s_c, float* s_lut) {
    for (int pat = threadIdx.x; pat < (1 << MT); pat += kThreads) {
        float v = (pat & 1) ? -s_c[0] : s_c[0];
#pragma unroll
        for (int i = 1; i < MT; ++i) v = __fadd_rn(v, ((pat >> i) & 1) ? -s_c[i] : s_c[i]);
        s_lut[pat] = v;
    }
}

template <int U, int MT, bool FULL>
__device__ __forceinline__ double server_rows_lut(const ServerArgs& a, const Tile& t, float sp,
                                                  float* s_c, float* s_lut) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int o0 = warp * (128 * U) + lane * 4;
    const int sh = (lane & 7) * 4;
    float* pp = a.pb + t.start + o0;
    const uint32_t* wp = a.wwords + t.word + (o0 >> 5);
    float p[U][4];
    unsigned w[U][MT];
    // all global loads first; the table is built while they are in flight
#pragma unroll
    for (int u = 0; u < U; ++u) {
        load4(pp + u * 128, o0 + u * 128, t.len, FULL, p[u]);
#pragma unroll
        for (int i = 0; i < MT; ++i)
            w[u][i] = (FULL || o0 + u * 128 < t.len) ? __ldg(wp + (long long)i * a.wstride + u * 4) : 0u;
    }
    build_scaled(a, t.block, MT, s_c);
    __syncthreads();
    build_lut<MT>(s_c, s_lut);
    __syncthreads();
    double acc = 0.0;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int o = o0 + u * 128;
        unsigned R = 0;
#pragma unroll
        for (int i = 0; i < MT; ++i) {
            const unsigned n = (w[u][i] >> sh) & 0xFu;
            R |= (n * (0x00204081u << i)) & (0x01010101u << i);
        }
        unsigned nib = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float avg = s_lut[(R >> (8 * k)) & 0xFFu];
            float pv = __fadd_rn(avg, residual_of(p[u][k], sp));      // ptilde_t
            if (!FULL && o + k >= t.len) pv = 0.f;
            p[u][k] = pv;
            nib |= (pv < 0.f ? 1u : 0u) << k;
        }
        acc += ((double)fabsf(p[u][0]) + (double)fabsf(p[u][1])) +
               ((double)fabsf(p[u][2]) + (double)fabsf(p[u][3]));
        const unsigned word = pack_nibbles(nib, lane);
        store4(pp + u * 128, o, t.len, FULL, p[u]);
        if ((lane & 7) == 0 && (FULL || o < t.len)) a.words[t.word + (o >> 5)] = word;
    }
    return acc;
}

// Direct evaluation for any M (and for tiles that are not 16-byte aligned).
__device__ __forceinline__ void average4(const ServerArgs& a, const float* s_c, long long wi,
                                         int sh, float (&avg)[4]) {
    const uint32_t* wp = a.wwords + wi;
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

template <int U, bool FULL>
__device__ __forceinline__ double server_rows(const ServerArgs& a, const Tile& t, float sp,
                                              const float* s_c) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int o0 = warp * (128 * U) + lane * 4;
    const int sh = (lane & 7) * 4;
    float* pp = a.pb + t.start + o0;
    float p[U][4];
#pragma unroll
    for (int u = 0; u < U; ++u) load4(pp + u * 128, o0 + u * 128, t.len, FULL, p[u]);
    double acc = 0.0;
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int o = o0 + u * 128;
        float avg[4] = {0.f, 0.f, 0.f, 0.f};
        if (FULL || o < t.len) average4(a, s_c, t.word + (o >> 5), sh, avg);
        unsigned nib = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            float pv = __fadd_rn(avg[k], residual_of(p[u][k], sp));   // ptilde_t
            if (!FULL && o + k >= t.len) pv = 0.f;
            p[u][k] = pv;
            nib |= (pv < 0.f ? 1u : 0u) << k;
        }
        acc += ((double)fabsf(p[u][0]) + (double)fabsf(p[u][1])) +
               ((double)fabsf(p[u][2]) + (double)fabsf(p[u][3]));
        const unsigned w = pack_nibbles(nib, lane);
        store4(pp + u * 128, o, t.len, FULL, p[u]);
        if ((lane & 7) == 0 && (FULL || o < t.len)) a.words[t.word + (o >> 5)] = w;
    }
    return acc;
}

__device__ __forceinline__ double server_rows_scalar(const ServerArgs& a, const Tile& t, float sp,
                                                     const float* s_c) {
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
                const unsigned w = __ldg(a.wwords + (long long)i * a.wstride + t.word + r);
                const float v = ((w >> lane) & 1u) ? -s_c[i] : s_c[i];
                avg = (i == 0) ? v : __fadd_rn(avg, v);
            }
            const long long j = t.start + o;
            pv = __fadd_rn(avg, residual_of(a.pb[j], sp));
            a.pb[j] = pv;
        }
        acc += (double)fabsf(pv);
        const unsigned w = __ballot_sync(kFull, valid && pv < 0.f);
        if (lane == 0) a.words[t.word + r] = w;
    }
    return acc;
}

// MT = number of workers when 1 <= M <= 8 (table path), MT = 0 for any other M.
template <int U, int MT>
__global__ void __launch_bounds__(kThreads) ef_server_kernel(const ServerArgs a) {
    extern __shared__ float s_c[];                     // M scaled worker scales
    __shared__ float s_lut[MT > 0 ? (1 << MT) : 1];
    const Tile t = a.tiles[blockIdx.x];
    const float sp = a.rscale[t.block];
    double acc;
    if (MT > 0 && (t.start & 3) == 0) {
        if (t.len == 1024 * U)
            acc = server_rows_lut<U, (MT > 0 ? MT : 1), true>(a, t, sp, s_c, s_lut);
        else
            acc = server_rows_lut<U, (MT > 0 ? MT : 1), false>(a, t, sp, s_c, s_lut);
    } else {
        build_scaled(a, t.block, a.M, s_c);
        __syncthreads();
        if ((t.start & 3) != 0)
            acc = server_rows_scalar(a, t, sp, s_c);
        else if (t.len == 1024 * U)
            acc = server_rows<U, true>(a, t, sp, s_c);
        else
            acc = server_rows<U, false>(a, t, sp, s_c);
    }
    finish_block(acc, blockIdx.x, t, a.blocks, a.partials, a.tickets, a.scale_out, a.rscale, a.fused);
}

// ------------------------------------------------------------------ parameter update
// x_{t+1,j} = x_{t,j} - eta * stilde_b * sign(ptilde_j)  (Algorithm 4, worker line after the pull)
template <int U>
__global__ void __launch_bounds__(kThreads) ef_apply_kernel(const ApplyArgs a) {
    const Tile t = a.tiles[blockIdx.x];
    const float step = __fmul_rn(a.eta, a.scales[t.block]);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if ((t.start & 3) != 0) {
        const int rows = (t.len + 31) >> 5;
        for (int r = warp; r < rows; r += kWarps) {
            const int o = r * 32 + lane;
            if (o < t.len) {
                const unsigned w = __ldg(a.words + t.word + r);
                const long long j = t.start + o;
                a.x[j] = ((w >> lane) & 1u) ? __fadd_rn(a.x[j], step) : __fsub_rn(a.x[j], step);
            }
        }
        return;
    }
    const bool full = (t.len == 1024 * U);
    const int o0 = warp * (128 * U) + lane * 4;
    const int sh = (lane & 7) * 4;
    float* xp = a.x + t.start + o0;
    float x[U][4];
    unsigned nib[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int o = o0 + u * 128;
        load4(xp + u * 128, o, t.len, full, x[u]);
        nib[u] = (full || o < t.len) ? (__ldg(a.words + t.word + (o >> 5)) >> sh) : 0u;
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
#pragma unroll
        for (int k = 0; k < 4; ++k)
            x[u][k] = ((nib[u] >> k) & 1u) ? __fadd_rn(x[u][k], step) : __fsub_rn(x[u][k], step);
        store4(xp + u * 128, o0 + u * 128, t.len, full, x[u]);
    }
}

// ------------------------------------------------------------------ residual materialisation
// dst_j = p_j - s_b * sign(p_j): the residual e_{t+1} in its plain form (tests, checkpoints).
template <int U>
__global__ void __launch_bounds__(kThreads) ef_residual_kernel(const ResidualArgs a) {
    const Tile t = a.tiles[blockIdx.x];
    const float s = a.rscale[t.block];
    for (int o = threadIdx.x; o < t.len; o += kThreads)
        a.dst[t.start + o] = residual_of(a.pb[t.start + o], s);
}

}  // namespace efk
