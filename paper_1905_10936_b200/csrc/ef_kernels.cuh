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
// partial sum per tile.  The last CTA to finish a block (found with one atomic ticket, no
// waiting) adds the block's partial sums in a fixed order and writes the scale.
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
__device__ __forceinline__ float4 ld_stream(const float* p) {
    return __ldcs(reinterpret_cast<const float4*>(p));
}
__device__ __forceinline__ void st_stream(float* p, float4 v) {
    __stcs(reinterpret_cast<float4*>(p), v);
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

// Combines the tile's |p| sum into the block scale s_b = ||p_b||_1 / d_b (Section 3.2).
// Single-tile blocks are finished directly.  Otherwise the tile's partial sum is published and
// the CTA that arrives last at the block's ticket adds all partial sums in tile order.  No CTA
// waits for another one.
__device__ __forceinline__ void finish_block(double acc, int tile_index, const Tile& t,
                                             const Block* __restrict__ blocks,
                                             double* __restrict__ partials,
                                             unsigned* __restrict__ tickets,
                                             float* __restrict__ scale_out,
                                             float* __restrict__ rscale) {
    __shared__ double s_sum[kWarps];
    __shared__ int s_last;
    double S = cta_sum(acc, s_sum);
    if (threadIdx.x == 0) {
        const Block b = blocks[t.block];
        if (b.tile_count == 1) {
            const float s = (float)(S / (double)b.len);
            scale_out[t.block] = s;
            rscale[t.block] = s;
            s_last = 0;
        } else {
            partials[tile_index] = S;
            __threadfence();
            const unsigned old = atomicAdd(&tickets[t.block], 1u);
            s_last = (old + 1u == (unsigned)b.tile_count);
        }
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const Block b = blocks[t.block];
    double v = 0.0;
    for (int k = threadIdx.x; k < b.tile_count; k += kThreads)
        v += __ldcg(&partials[b.tile_begin + k]);
    S = cta_sum(v, s_sum);
    if (threadIdx.x == 0) {
        const float s = (float)(S / (double)b.len);
        scale_out[t.block] = s;
        rscale[t.block] = s;
        tickets[t.block] = 0u;      // ready for the next launch
    }
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
    finish_block(acc, blockIdx.x, t, a.blocks, a.partials, a.tickets, a.scale_out, a.rscale);
}

// ------------------------------------------------------------------ server kernel
// a_j = sum over ascending i of (bit_i ? -c_i : +c_i), c_i = fl(scale_{i,b} / M), the first
// term taken as is (Algorithm 4, server line: (1/M) sum_i Delta_{t,i}).
template <int MT>
__device__ __forceinline__ void average4(const ServerArgs& a, const float* s_c, long long wi,
                                         int sh, float (&avg)[4]) {
    const int M = MT > 0 ? MT : a.M;
    const uint32_t* wp = a.wwords + wi;
#pragma unroll(MT > 0 ? MT : 4)
    for (int i = 0; i < M; ++i) {
        const unsigned nib = __ldg(wp + (long long)i * a.wstride) >> sh;
        const unsigned cb = __float_as_uint(s_c[i]);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float v = __uint_as_float(cb ^ ((nib << (31 - k)) & 0x80000000u));
            avg[k] = (i == 0) ? v : __fadd_rn(avg[k], v);
        }
    }
}

template <int U, int MT, bool FULL>
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
        if (FULL || o < t.len) average4<MT>(a, s_c, t.word + (o >> 5), sh, avg);
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

template <int U, int MT>
__global__ void __launch_bounds__(kThreads) ef_server_kernel(const ServerArgs a) {
    extern __shared__ float s_c[];
    const Tile t = a.tiles[blockIdx.x];
    const int M = MT > 0 ? MT : a.M;
    for (int i = threadIdx.x; i < M; i += kThreads)
        s_c[i] = __fdiv_rn(a.wscales[(long long)i * a.sstride + t.block], (float)M);
    const float sp = a.rscale[t.block];
    __syncthreads();
    double acc;
    if ((t.start & 3) != 0)
        acc = server_rows_scalar(a, t, sp, s_c);
    else if (t.len == 1024 * U)
        acc = server_rows<U, MT, true>(a, t, sp, s_c);
    else
        acc = server_rows<U, MT, false>(a, t, sp, s_c);
    finish_block(acc, blockIdx.x, t, a.blocks, a.partials, a.tickets, a.scale_out, a.rscale);
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
