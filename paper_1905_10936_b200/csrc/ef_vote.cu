// signum / signSGD with majority vote (the paper's comparison method, Sections 1, 4.1 and 4.2;
// Table 1: 2Md bits per iteration) on the same context, state and packed layout as the
// error-feedback path:
//   worker i :  m_i <- mu m_i + g_i ;  message = packed sign(m_i)           (ef_vote_worker_step)
//   server   :  vote = sign(sum_i sign(m_i)) ;  x <- x - eta vote           (ef_vote_server_step)
// sign(+-0) = +1 and a tied vote (even M) is sent as +1 (the message is one bit).
//
// Both kernels are single streaming passes: the worker reads g and m and writes m and one bit
// per element (12.125 bytes per element); the server reads M bits and x and writes x and one
// bit (8 + (M+1)/8 bytes per element).  The vote itself is computed on whole 32-bit words: the
// M packed words of a group of 32 elements are added into bit-sliced counters (plane p holds
// bit p of every element's count of negative votes) with a ripple of half adders, and the
// comparison count >= floor(M/2)+1 is evaluated on the planes.  For M <= 16 the counters come
// from a carry-save adder network (M = 7: eight logic operations for the 32 votes of a word),
// for larger M from a ripple of half adders; either way there is no per-element work at all.
#include "ef_internal.h"

#include <algorithm>

namespace {

using efk::Tile;
using efk::kFull;
using efk::kThreads;
using efk::kWarps;
using namespace efh;

struct VoteWorkerArgs {
    const float* g;
    float* m;
    uint32_t* words;
    const Tile* tiles;
    float mu;
    long long g_stride, state_stride, word_stride;   // blockIdx.y selects the worker
    efk::DebugLimits lim;
};

struct VoteServerArgs {
    const uint32_t* wwords;   // worker 0; worker i at + i*wstride
    long long wstride;
    int M;
    unsigned threshold;       // floor(M/2) + 1 negative votes make the majority negative
    uint32_t* words;          // the vote, packed
    float* x;
    const Tile* tiles;
    float eta;
    efk::DebugLimits lim;
};

// Sign bits (value < 0, so that -0 counts as +1) of four values as a nibble, element k in bit k.
__device__ __forceinline__ unsigned negative_nibble(const float (&v)[4]) {
    return (v[0] < 0.f ? 1u : 0u) | (v[1] < 0.f ? 2u : 0u) | (v[2] < 0.f ? 4u : 0u) |
           (v[3] < 0.f ? 8u : 0u);
}

// ------------------------------------------------------------------ worker
// One chunk per CTA, same thread-to-element mapping as the error-feedback worker kernel.
template <int U, bool FULL>
__device__ __forceinline__ void vote_worker_rows(const VoteWorkerArgs& a, const Tile& t) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int o0 = warp * (128 * U) + lane * 4;
    const float* gp = a.g + t.start + o0;
    float* mp = a.m + t.start + o0;
    float g[U][4], m[U][4];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        efk::load4(gp + u * 128, o0 + u * 128, t.len, FULL, g[u]);
        efk::load4(mp + u * 128, o0 + u * 128, t.len, FULL, m[u]);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int o = o0 + u * 128;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            float mv = __fmaf_rn(a.mu, m[u][k], g[u][k]);          // m_t = mu m_{t-1} + g_t
            if (!FULL && o + k >= t.len) mv = 0.f;
            m[u][k] = mv;
        }
        const unsigned w = efk::pack_nibbles(negative_nibble(m[u]), lane);
        efk::store4(mp + u * 128, o, t.len, FULL, m[u]);
        if ((lane & 7) == 0 && (FULL || o < t.len)) a.words[t.word + (o >> 5)] = w;
    }
}

__device__ __forceinline__ void vote_worker_rows_scalar(const VoteWorkerArgs& a, const Tile& t) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rows = (t.len + 31) >> 5;
    for (int r = warp; r < rows; r += kWarps) {
        const int o = r * 32 + lane;
        const bool valid = o < t.len;
        float mv = 0.f;
        if (valid) {
            const long long j = t.start + o;
            mv = __fmaf_rn(a.mu, a.m[j], a.g[j]);
            a.m[j] = mv;
        }
        const unsigned w = __ballot_sync(kFull, valid && mv < 0.f);
        if (lane == 0) a.words[t.word + r] = w;
    }
}

template <int U>
__global__ void __launch_bounds__(kThreads) ef_vote_worker_kernel(const VoteWorkerArgs a0) {
    efk::pdl_enter();
    VoteWorkerArgs a = a0;
    const long long wi = blockIdx.y;
    a.g += wi * a.g_stride;
    a.m += wi * a.state_stride;
    a.words += wi * a.word_stride;
    const Tile t = efk::chunk_of<U>(a.tiles[blockIdx.x / a.lim.tc], blockIdx.x % a.lim.tc);
    if (t.len <= 0 || !efk::work_item_ok(t, a.lim, 1024 * U)) return;
    if ((t.start & 3) != 0) vote_worker_rows_scalar(a, t);
    else if (t.len == 1024 * U) vote_worker_rows<U, true>(a, t);
    else vote_worker_rows<U, false>(a, t);
}

// ------------------------------------------------------------------ server
// Majority of M packed words, bit-parallel.  Two forms:
//  * M known at compile time (1..16): a carry-save adder network.  Words of equal weight are
//    compressed three at a time by full adders (sum = x^y^z stays, carry = maj(x,y,z) moves one
//    weight up: two logic operations for three words) until one word per weight is left: the
//    planes of the count.  M = 7 takes 4 full adders, M = 15 takes 12.
//  * any M: a ripple of half adders into P counter planes (2^P > M), eight workers' words loaded
//    at a time.
// Then count >= threshold is evaluated on the planes.
template <int N>
struct CsaLevel {     // a[0..N): words of one weight -> a[0]; the floor(N/2) carries go to up[0..)
    __device__ __forceinline__ static void run(unsigned* a, unsigned* up) {
        if constexpr (N >= 3) {
            constexpr int F = N / 3, R = N % 3;
            unsigned s[F + R];
#pragma unroll
            for (int i = 0; i < F; ++i) {
                const unsigned x = a[3 * i], y = a[3 * i + 1], z = a[3 * i + 2];
                s[i] = x ^ y ^ z;
                up[i] = (x & y) | (z & (x ^ y));
            }
#pragma unroll
            for (int i = 0; i < R; ++i) s[F + i] = a[3 * F + i];
#pragma unroll
            for (int i = 0; i < F + R; ++i) a[i] = s[i];
            CsaLevel<F + R>::run(a, up + F);
        } else if constexpr (N == 2) {
            const unsigned x = a[0], y = a[1];
            a[0] = x ^ y;
            up[0] = x & y;
        }
    }
};
template <int N, int PLANE>
struct CsaCount {     // a[0..N) of weight 2^PLANE -> planes[PLANE..]
    __device__ __forceinline__ static void run(unsigned* a, unsigned* planes) {
        unsigned up[N / 2 + 1];
        CsaLevel<N>::run(a, up);
        planes[PLANE] = a[0];
        if constexpr (N / 2 > 0) CsaCount<N / 2, PLANE + 1>::run(up, planes);
    }
};
__host__ __device__ constexpr int planes_of(int M) { int p = 1; while ((1 << p) <= M) ++p; return p; }

// count >= threshold, from the least significant plane up:
//   ge_p = (c_p > t_p) | ((c_p == t_p) & ge_{p-1}),  ge_{-1} = 1
template <int P>
__device__ __forceinline__ unsigned planes_ge(const unsigned (&c)[P], unsigned threshold) {
    unsigned ge = 0xffffffffu;
#pragma unroll
    for (int p = 0; p < P; ++p) ge = ((threshold >> p) & 1u) ? (ge & c[p]) : (ge | c[p]);
    return ge;
}

// MT > 0: M = MT at compile time; MT == 0: any M with P planes.  Word position r (of R) of
// worker i is w0[r * rstride + i * wstride]; positions with active[r] == false are not read and
// vote 0.
template <int MT, int P, int R>
__device__ __forceinline__ void majority_words(const uint32_t* __restrict__ w0, int rstride,
                                               long long wstride, int M, unsigned threshold,
                                               const bool (&active)[R], unsigned (&out)[R]) {
    if constexpr (MT > 0) {
        unsigned w[R][MT];
#pragma unroll
        for (int i = 0; i < MT; ++i)
#pragma unroll
            for (int r = 0; r < R; ++r)
                w[r][i] = active[r] ? __ldg(w0 + r * rstride + (long long)i * wstride) : 0u;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            unsigned planes[planes_of(MT)];
            CsaCount<MT, 0>::run(w[r], planes);
            out[r] = planes_ge<planes_of(MT)>(planes, (unsigned)(MT / 2 + 1));
        }
    } else {
        unsigned c[R][P];
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int p = 0; p < P; ++p) c[r][p] = 0u;
        for (int i0 = 0; i0 < M; i0 += 8) {
            unsigned w[R][8];
#pragma unroll
            for (int k = 0; k < 8; ++k)
#pragma unroll
                for (int r = 0; r < R; ++r)
                    w[r][k] = (i0 + k < M && active[r])
                                  ? __ldg(w0 + r * rstride + (long long)(i0 + k) * wstride) : 0u;
#pragma unroll
            for (int k = 0; k < 8; ++k)
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    unsigned carry = w[r][k];          // count += word, one half adder per plane
#pragma unroll
                    for (int p = 0; p < P; ++p) {
                        const unsigned t = c[r][p] & carry;
                        c[r][p] ^= carry;
                        carry = t;
                    }
                }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) out[r] = planes_ge<P>(c[r], threshold);
    }
}

// x <- x - eta * vote for the four elements of a lane (nibble: bit k set = vote -1).
__device__ __forceinline__ void vote_apply4(float (&x)[4], unsigned nib, float eta) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float signed_eta = __uint_as_float(__float_as_uint(eta) ^ ((nib << (31 - k)) & 0x80000000u));
        x[k] = __fsub_rn(x[k], signed_eta);
    }
}

// One tile per CTA; the CTA walks the tile's chunks, one or two rows of 128 elements at a time.
// MT = M for 1 <= M <= 16 (adder network), else 0 with P counter planes.
template <int U, int MT, int P>
__global__ void __launch_bounds__(kThreads, 4) ef_vote_server_kernel(const VoteServerArgs a) {
    constexpr int kChunk = 1024 * U;
    efk::pdl_enter();
    const Tile t = a.tiles[blockIdx.x];
    if (!efk::work_item_ok(t, a.lim, a.lim.tc * kChunk)) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if ((t.start & 3) != 0) {                   // block does not start on a 16-byte boundary
        const int rows = (t.len + 31) >> 5;
        for (int r = warp; r < rows; r += kWarps) {
            const bool one[1] = {true};
            unsigned vv[1];
            majority_words<MT, P, 1>(a.wwords + t.word + r, 0, a.wstride, a.M, a.threshold, one, vv);
            const unsigned v = vv[0];
            const int o = r * 32 + lane;
            if (o < t.len) {
                const long long j = t.start + o;
                const float signed_eta = ((v >> lane) & 1u) ? -a.eta : a.eta;
                a.x[j] = __fsub_rn(a.x[j], signed_eta);
            }
            if (lane == 0) a.words[t.word + r] = v;
        }
        return;
    }
    const int o0 = warp * (128 * U) + lane * 4;
    const int sh = (lane & 7) * 4;
    for (int c = 0; c * kChunk < t.len; ++c) {
        const int clen = min(kChunk, t.len - c * kChunk);
        const bool full = clen == kChunk;
        float* xp = a.x + t.start + (long long)c * kChunk + o0;
        const long long wbase = t.word + c * (kChunk / 32) + (o0 >> 5);
        // rows per batch: all of a batch's worker words are loaded before any is used
        constexpr int RB = (MT > 0 && MT <= 8) ? 2 : 1;
        static_assert(U % RB == 0, "rows are handled in batches");
        float x[U][4];
#pragma unroll
        for (int u = 0; u < U; ++u) efk::load4(xp + u * 128, o0 + u * 128, clen, full, x[u]);
#pragma unroll
        for (int u0 = 0; u0 < U; u0 += RB) {
            bool active[RB];                                // false: the 32-element group is past the end
            unsigned v[RB];
#pragma unroll
            for (int r = 0; r < RB; ++r) active[r] = full || ((o0 + (u0 + r) * 128) & ~31) < clen;
            majority_words<MT, P, RB>(a.wwords + wbase + u0 * 4, 4, a.wstride, a.M, a.threshold, active, v);
#pragma unroll
            for (int r = 0; r < RB; ++r) {
                const int u = u0 + r, o = o0 + u * 128;
                if (!active[r]) continue;
                vote_apply4(x[u], v[r] >> sh, a.eta);
                efk::store4(xp + u * 128, o, clen, full, x[u]);
                if ((lane & 7) == 0) a.words[wbase + u * 4] = v[r];
            }
        }
    }
}

template <int MT, int P>
void launch_vote_server_t(ef_ctx* c, const VoteServerArgs& a) {
    launch_kernel(c, ef_vote_server_kernel<kU, MT, P>, dim3((unsigned)c->L.num_tiles), 0, a);
}

int launch_vote_worker(ef_ctx* c, int i, const float* grad, int count, long long g_stride) {
    VoteWorkerArgs a;
    a.g = grad; a.m = c->m(i); a.words = c->words(i); a.tiles = c->tiles(); a.mu = c->mu;
    a.g_stride = g_stride; a.state_stride = (long long)c->L.dpad; a.word_stride = (long long)c->L.wpad;
    a.lim = c->limits();
    const dim3 grid((unsigned)(c->L.num_tiles * c->L.tile_chunks), (unsigned)count);
    launch_kernel(c, ef_vote_worker_kernel<kU>, grid, 0, a);
    EF_CUDA(c, cudaGetLastError());
    c->launches += 1;
    return EF_OK;
}

}  // namespace

extern "C" {

int ef_vote_worker_step(ef_ctx* c, int32_t i, const float* grad) {
    EF_API_RANGE();
    int rc = check_worker_call(c, i, grad, kModeVote);
    if (rc != EF_OK) return rc;
    if (!aligned16(grad)) return EF_ERR_ALIGNMENT;
    rc = launch_vote_worker(c, i, grad, 1, 0);
    if (rc != EF_OK) return rc;
    mark_stepped(c, i, kModeVote);
    return EF_OK;
}

int ef_vote_worker_step_host(ef_ctx* c, int32_t i, const float* grad) {
    EF_API_RANGE();
    int rc = check_worker_call(c, i, grad, kModeVote);
    if (rc != EF_OK) return rc;
    if (!(c->flags & EF_FLAG_HOST_STAGING)) return EF_ERR_BAD_STATE;
    float* staged = nullptr;
    rc = stage_host_gradient(c, grad, &staged);
    if (rc != EF_OK) return rc;
    rc = launch_vote_worker(c, i, staged, 1, 0);
    if (rc != EF_OK) return rc;
    rc = host_gradient_consumed(c);
    if (rc != EF_OK) return rc;
    mark_stepped(c, i, kModeVote);
    return EF_OK;
}

int ef_vote_worker_step_all(ef_ctx* c, const float* grads, int64_t stride) {
    EF_API_RANGE();
    if (!c || !grads || stride < c->L.d) return EF_ERR_INVALID_ARG;
    if (!aligned16(grads) || (stride & 3) != 0) return EF_ERR_ALIGNMENT;
    if (c->pending != 0) return EF_ERR_BAD_STATE;
    const int rc = launch_vote_worker(c, 0, grads, c->L.Ml, (long long)stride);
    if (rc != EF_OK) return rc;
    mark_all_stepped(c, kModeVote);
    return EF_OK;
}

int ef_vote_server_step(ef_ctx* c) {
    EF_API_RANGE();
    if (!c) return EF_ERR_INVALID_ARG;
    if (c->pending != c->L.M || c->mode != kModeVote) return EF_ERR_BAD_STATE;   // needs all M workers local
    const int M = c->L.M;
    VoteServerArgs a;
    a.wwords = c->words(0); a.wstride = (long long)c->L.wpad; a.M = M;
    a.threshold = (unsigned)(M / 2 + 1);
    a.words = c->words(c->srv()); a.x = c->x(); a.tiles = c->tiles(); a.eta = c->eta;
    a.lim = c->limits();
    switch (M <= 16 ? M : 16 + planes_of(M)) {
        case 1: launch_vote_server_t<1, 1>(c, a); break;
        case 2: launch_vote_server_t<2, 1>(c, a); break;
        case 3: launch_vote_server_t<3, 1>(c, a); break;
        case 4: launch_vote_server_t<4, 1>(c, a); break;
        case 5: launch_vote_server_t<5, 1>(c, a); break;
        case 6: launch_vote_server_t<6, 1>(c, a); break;
        case 7: launch_vote_server_t<7, 1>(c, a); break;
        case 8: launch_vote_server_t<8, 1>(c, a); break;
        case 9: launch_vote_server_t<9, 1>(c, a); break;
        case 10: launch_vote_server_t<10, 1>(c, a); break;
        case 11: launch_vote_server_t<11, 1>(c, a); break;
        case 12: launch_vote_server_t<12, 1>(c, a); break;
        case 13: launch_vote_server_t<13, 1>(c, a); break;
        case 14: launch_vote_server_t<14, 1>(c, a); break;
        case 15: launch_vote_server_t<15, 1>(c, a); break;
        case 16: launch_vote_server_t<16, 1>(c, a); break;
        case 16 + 5: launch_vote_server_t<0, 5>(c, a); break;      // 17 <= M < 32
        case 16 + 6: launch_vote_server_t<0, 6>(c, a); break;
        case 16 + 7: launch_vote_server_t<0, 7>(c, a); break;
        case 16 + 8: launch_vote_server_t<0, 8>(c, a); break;
        case 16 + 9: launch_vote_server_t<0, 9>(c, a); break;
        case 16 + 10: launch_vote_server_t<0, 10>(c, a); break;
        case 16 + 11: launch_vote_server_t<0, 11>(c, a); break;
        case 16 + 12: launch_vote_server_t<0, 12>(c, a); break;
        default: launch_vote_server_t<0, 13>(c, a); break;         // M <= EF_MAX_WORKERS = 4096 < 2^13
    }
    EF_CUDA(c, cudaGetLastError());
    c->launches += 1;
    end_iteration(c);
    return EF_OK;
}

}  // extern "C"
