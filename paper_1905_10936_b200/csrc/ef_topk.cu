// Top-k compressor with its error-feedback residual (Section 2, second example after
// Definition 1: the operator that keeps the k coordinates of largest absolute value; used in
// Algorithm 2 as  Delta = C(p),  e = p - Delta).
//
//   ef_topk_compress(v, n, k) -> idx[k] (increasing), val[k] = v[idx], resid = v - C(v)
//
// Among equal magnitudes the lower index is kept, so the result is unique and reproducible.
//
// Method (all integer work on the bit pattern of |v_j|, which orders like the magnitude):
//   1. radix select of the k-th largest key in three passes over v (11 + 11 + 9 bits): each pass
//      histograms one digit of the keys that still match the prefix found so far (shared-memory
//      histogram per CTA, merged into a global one), then one CTA finds the bin, from the top,
//      in which the count reaches what is still to keep, and fixes the next digit.  Result: the threshold key T and how many keys equal
//      to T have to be kept (need_eq).
//   2. a counting pass: per 4096-element chunk the number of keys > T and == T;
//   3. a scan of those counts over the chunks (one CTA);
//   4. a scatter pass: every chunk recomputes its flags, ranks its kept elements in index order
//      (ballots + population counts, no sorting) and writes idx, val and the residual.
// Traffic: five reads of v, one write of the residual, k index/value pairs: about 24 bytes per
// element.  Nothing waits on another CTA; kernel boundaries order the passes.
#include "ef_internal.h"

#include <algorithm>

namespace {

using efk::kFull;
using efk::kThreads;
using efk::kWarps;
using namespace efh;

constexpr int kBins = 2048;
constexpr int kPasses = 3;
__host__ __device__ constexpr int pass_shift(int p) { return p == 0 ? 20 : (p == 1 ? 9 : 0); }
__host__ __device__ constexpr int pass_bits(int p) { return p == 2 ? 9 : 11; }

struct TopkState {                 // lives in the workspace; written by the select kernel
    unsigned long long remaining;  // how many of the keys matching `prefix` are still to keep
    unsigned prefix;               // digits fixed so far (high bits of the threshold key)
    unsigned threshold;            // final: the k-th largest key T
    unsigned long long need_eq;    // final: number of keys == T to keep (lowest indices first)
};

struct TopkLayout {
    size_t off_hist = 0, off_state = 0, off_cgt = 0, off_ceq = 0, off_pgt = 0, off_peq = 0, total = 0;
    long long chunks = 0;
};

TopkLayout topk_layout(int64_t n) {
    TopkLayout L;
    L.chunks = (n + kChunkLen - 1) / kChunkLen;
    size_t o = 0;
    L.off_hist = o;  o += align_up(sizeof(unsigned long long) * kBins * kPasses);
    L.off_state = o; o += align_up(sizeof(TopkState));
    L.off_cgt = o;   o += align_up(sizeof(unsigned) * (size_t)L.chunks);
    L.off_ceq = o;   o += align_up(sizeof(unsigned) * (size_t)L.chunks);
    L.off_pgt = o;   o += align_up(sizeof(unsigned long long) * (size_t)L.chunks);
    L.off_peq = o;   o += align_up(sizeof(unsigned long long) * (size_t)L.chunks);
    L.total = o;
    return L;
}

__device__ __forceinline__ unsigned key_of(float v) { return __float_as_uint(v) & 0x7fffffffu; }

// Loads the four elements of this lane's row; elements past n read as a key that is never kept.
__device__ __forceinline__ void load_keys(const float* __restrict__ v, long long base, long long n,
                                          float (&x)[4], bool (&in)[4]) {
    if (base + 4 <= n) {
        const float4 q = efk::ld_stream(v + base);
        x[0] = q.x; x[1] = q.y; x[2] = q.z; x[3] = q.w;
        in[0] = in[1] = in[2] = in[3] = true;
    } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            in[k] = base + k < n;
            x[k] = in[k] ? v[base + k] : 0.f;
        }
    }
}

// ---- 1. one radix pass: histogram of digit PASS over the keys that match the prefix so far
template <int PASS>
__global__ void __launch_bounds__(kThreads) ef_topk_hist_kernel(const float* __restrict__ v, long long n,
                                                                long long chunks,
                                                                const TopkState* __restrict__ st,
                                                                unsigned long long* __restrict__ hist) {
    __shared__ unsigned s_hist[kBins];
    for (int b = threadIdx.x; b < kBins; b += kThreads) s_hist[b] = 0u;
    __syncthreads();
    constexpr int shift = pass_shift(PASS), bits = pass_bits(PASS);
    const unsigned prefix = PASS == 0 ? 0u : st->prefix;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (long long c = blockIdx.x; c < chunks; c += gridDim.x) {
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            const long long base = c * kChunkLen + warp * (128 * kU) + u * 128 + lane * 4;
            if (base >= n) continue;
            float x[4]; bool in[4];
            load_keys(v, base, n, x, in);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const unsigned key = key_of(x[k]);
                const bool match = PASS == 0 || (key >> (shift + bits)) == prefix;
                if (in[k] && match) atomicAdd(&s_hist[(key >> shift) & ((1u << bits) - 1u)], 1u);
            }
        }
    }
    __syncthreads();
    for (int b = threadIdx.x; b < (1 << bits); b += kThreads)
        if (s_hist[b]) atomicAdd(&hist[b], (unsigned long long)s_hist[b]);
}

// One CTA fixes the next digit: it finds, from the largest digit down, the bin in which the
// count of keys seen so far reaches `remaining`.  Thread t adds up bins 8t .. 8t+7; thread 0
// walks the 256 sums from the top and then the eight bins of the group it stops in.
template <int PASS>
__global__ void __launch_bounds__(kThreads) ef_topk_select_kernel(const unsigned long long* __restrict__ hist,
                                                                  TopkState* st, unsigned long long k) {
    constexpr int bits = pass_bits(PASS), nbins = 1 << bits, per = kBins / kThreads;
    __shared__ unsigned long long s_bin[kBins], s_grp[kThreads];
    unsigned long long g = 0;
#pragma unroll
    for (int j = 0; j < per; ++j) {
        const int b = threadIdx.x * per + j;
        const unsigned long long v = b < nbins ? hist[b] : 0ull;
        s_bin[b] = v;
        g += v;
    }
    s_grp[threadIdx.x] = g;
    __syncthreads();
    if (threadIdx.x != 0) return;
    unsigned long long remaining = PASS == 0 ? k : st->remaining;
    const unsigned prefix = PASS == 0 ? 0u : st->prefix;
    unsigned long long above = 0;
    int grp = kThreads - 1;
    for (; grp > 0; --grp) {
        if (above + s_grp[grp] >= remaining) break;
        above += s_grp[grp];
    }
    int b = grp * per + per - 1;
    for (; b > grp * per; --b) {
        if (above + s_bin[b] >= remaining) break;
        above += s_bin[b];
    }
    remaining -= above;                       // still to keep among the keys of bin b
    st->prefix = (prefix << bits) | (unsigned)b;
    st->remaining = remaining;
    if (PASS == kPasses - 1) {
        st->threshold = st->prefix;
        st->need_eq = remaining;
    }
}

// ---- 2. per chunk: how many keys are > T and == T
__global__ void __launch_bounds__(kThreads) ef_topk_count_kernel(const float* __restrict__ v, long long n,
                                                                 const TopkState* __restrict__ st,
                                                                 unsigned* __restrict__ cgt,
                                                                 unsigned* __restrict__ ceq) {
    __shared__ unsigned s_gt[kWarps], s_eq[kWarps];
    const unsigned T = st->threshold;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    unsigned gt = 0, eq = 0;
#pragma unroll
    for (int u = 0; u < kU; ++u) {
        const long long base = (long long)blockIdx.x * kChunkLen + warp * (128 * kU) + u * 128 + lane * 4;
        if (base >= n) continue;
        float x[4]; bool in[4];
        load_keys(v, base, n, x, in);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const unsigned key = key_of(x[k]);
            gt += (in[k] && key > T) ? 1u : 0u;
            eq += (in[k] && key == T) ? 1u : 0u;
        }
    }
    unsigned both = gt | (eq << 16);          // at most 512 elements per warp each: two 16-bit fields
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) both += __shfl_xor_sync(kFull, both, o);
    if (lane == 0) { s_gt[warp] = both & 0xffffu; s_eq[warp] = both >> 16; }
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned a = 0, b = 0;
        for (int w = 0; w < kWarps; ++w) { a += s_gt[w]; b += s_eq[w]; }
        cgt[blockIdx.x] = a;
        ceq[blockIdx.x] = b;
    }
}

// ---- 3. exclusive prefix sums of the two count arrays over the chunks (one CTA)
constexpr int kScanThreads = 1024;
__device__ __forceinline__ unsigned long long warp_inclusive_scan(unsigned long long v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long u = __shfl_up_sync(kFull, v, o);
        if (lane >= o) v += u;
    }
    return v;
}
__global__ void __launch_bounds__(kScanThreads) ef_topk_scan_kernel(const unsigned* __restrict__ cgt,
                                                                    const unsigned* __restrict__ ceq,
                                                                    unsigned long long* __restrict__ pgt,
                                                                    unsigned long long* __restrict__ peq,
                                                                    long long chunks) {
    __shared__ unsigned long long s_a[32], s_b[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long per = (chunks + kScanThreads - 1) / kScanThreads;
    const long long lo = min(chunks, (long long)threadIdx.x * per), hi = min(chunks, lo + per);
    unsigned long long a = 0, b = 0;
    for (long long c = lo; c < hi; ++c) { a += cgt[c]; b += ceq[c]; }
    // exclusive scan of the per-thread totals over the CTA: warps, then the warps' totals
    const unsigned long long ia = warp_inclusive_scan(a, lane), ib = warp_inclusive_scan(b, lane);
    if (lane == 31) { s_a[warp] = ia; s_b[warp] = ib; }
    __syncthreads();
    if (warp == 0) {
        const unsigned long long wa = warp_inclusive_scan(s_a[lane], lane), wb = warp_inclusive_scan(s_b[lane], lane);
        s_a[lane] = wa - s_a[lane];            // exclusive
        s_b[lane] = wb - s_b[lane];
    }
    __syncthreads();
    a = s_a[warp] + ia - a;
    b = s_b[warp] + ib - b;
    for (long long c = lo; c < hi; ++c) {
        pgt[c] = a; peq[c] = b;
        a += cgt[c]; b += ceq[c];
    }
}

// ---- 4. scatter: kept = key > T, or key == T and fewer than need_eq equal keys precede it
__global__ void __launch_bounds__(kThreads) ef_topk_scatter_kernel(const float* v, long long n,
                                                                   const TopkState* __restrict__ st,
                                                                   const unsigned long long* __restrict__ pgt,
                                                                   const unsigned long long* __restrict__ peq,
                                                                   long long* __restrict__ idx_out,
                                                                   float* __restrict__ val_out,
                                                                   float* resid, unsigned long long kmax) {
    // resid may alias v: every thread has read its own elements before it writes them.
    // element order inside a chunk: warp, then row, then lane, then the lane's four elements
    __shared__ unsigned s_eq[kWarps], s_gt[kWarps];
    const unsigned T = st->threshold;
    const unsigned long long need_eq = st->need_eq;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const unsigned lt_mask = (1u << lane) - 1u;
    float x[kU][4]; bool in[kU][4];
    unsigned feq[kU], fgt[kU];                 // nibbles of flags
    unsigned eq_lanes_before[kU], gt_lanes_before[kU], eq_row[kU], gt_row[kU];
    unsigned weq = 0, wgt = 0;                 // this warp's totals
#pragma unroll
    for (int u = 0; u < kU; ++u) {
        const long long base = (long long)blockIdx.x * kChunkLen + warp * (128 * kU) + u * 128 + lane * 4;
        feq[u] = fgt[u] = 0u;
        if (base < n) {
            load_keys(v, base, n, x[u], in[u]);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const unsigned key = key_of(x[u][k]);
                if (in[u][k] && key == T) feq[u] |= 1u << k;
                if (in[u][k] && key > T) fgt[u] |= 1u << k;
            }
        } else {
#pragma unroll
            for (int k = 0; k < 4; ++k) { in[u][k] = false; x[u][k] = 0.f; }
        }
        // keys of this row before this lane, and in the whole row: one ballot per element position
        eq_lanes_before[u] = gt_lanes_before[u] = eq_row[u] = gt_row[u] = 0u;
        if (__any_sync(kFull, (feq[u] | fgt[u]) != 0u)) {      // most rows keep nothing
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const unsigned be = __ballot_sync(kFull, (feq[u] >> k) & 1u);
                const unsigned bg = __ballot_sync(kFull, (fgt[u] >> k) & 1u);
                eq_lanes_before[u] += __popc(be & lt_mask); eq_row[u] += __popc(be);
                gt_lanes_before[u] += __popc(bg & lt_mask); gt_row[u] += __popc(bg);
            }
        }
        weq += eq_row[u];
        wgt += gt_row[u];
    }
    if (lane == 0) { s_eq[warp] = weq; s_gt[warp] = wgt; }
    __syncthreads();
    unsigned long long eq_before = peq[blockIdx.x], gt_before = pgt[blockIdx.x];
    for (int w = 0; w < warp; ++w) { eq_before += s_eq[w]; gt_before += s_gt[w]; }
#pragma unroll
    for (int u = 0; u < kU; ++u) {
        const long long base = (long long)blockIdx.x * kChunkLen + warp * (128 * kU) + u * 128 + lane * 4;
        unsigned long long eq_rank = eq_before + eq_lanes_before[u];     // equal keys before element 0 of this lane
        unsigned long long gt_rank = gt_before + gt_lanes_before[u];
        float r[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const bool is_eq = (feq[u] >> k) & 1u, is_gt = (fgt[u] >> k) & 1u;
            const bool kept = is_gt || (is_eq && eq_rank < need_eq);
            if (kept) {
                // kept elements before this one = (keys > T before it) + min(equal keys before it, need_eq)
                const unsigned long long pos = gt_rank + (eq_rank < need_eq ? eq_rank : need_eq);
                if (pos < kmax) {              // always true when the counts are consistent
                    idx_out[pos] = base + k;
                    val_out[pos] = x[u][k];
                }
            }
            r[k] = kept ? __fsub_rn(x[u][k], x[u][k]) : x[u][k];      // e = v - C(v)
            eq_rank += is_eq ? 1u : 0u;
            gt_rank += is_gt ? 1u : 0u;
        }
        if (resid != nullptr && base < n) {
            if (base + 4 <= n) efk::st_stream(resid + base, make_float4(r[0], r[1], r[2], r[3]));
            else
                for (int k = 0; k < 4; ++k) if (in[u][k]) resid[base + k] = r[k];
        }
        eq_before += eq_row[u];
        gt_before += gt_row[u];
    }
}

}  // namespace

extern "C" {

int ef_topk_workspace_bytes(int64_t n, size_t* bytes) {
    if (!bytes || n < 1) return EF_ERR_INVALID_ARG;
    *bytes = topk_layout(n).total;
    return EF_OK;
}

int ef_topk_compress(const float* v, int64_t n, int64_t k, int64_t* idx_out, float* val_out,
                     float* resid_out, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!v || n < 1 || k < 1 || k > n || !idx_out || !val_out) return EF_ERR_INVALID_ARG;
    const TopkLayout L = topk_layout(n);
    if (L.chunks > 0x7fffffffLL) return EF_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < L.total) return EF_ERR_WORKSPACE;
    if (!aligned16(v) || (resid_out && !aligned16(resid_out)) || ((uintptr_t)workspace & (kAlign - 1)))
        return EF_ERR_ALIGNMENT;
    int dev = -1, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return EF_ERR_CUDA;
    if (major != 10) return EF_ERR_UNSUPPORTED_DEVICE;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    char* ws = (char*)workspace;
    unsigned long long* hist = (unsigned long long*)(ws + L.off_hist);
    TopkState* state = (TopkState*)(ws + L.off_state);
    unsigned* cgt = (unsigned*)(ws + L.off_cgt);
    unsigned* ceq = (unsigned*)(ws + L.off_ceq);
    unsigned long long* pgt = (unsigned long long*)(ws + L.off_pgt);
    unsigned long long* peq = (unsigned long long*)(ws + L.off_peq);
    if (cudaMemsetAsync(ws, 0, L.off_cgt, st) != cudaSuccess) return EF_ERR_CUDA;   // histograms + state
    const unsigned hgrid = (unsigned)std::min<long long>(L.chunks, 148 * 8);
    const unsigned long long kk = (unsigned long long)k;
    ef_topk_hist_kernel<0><<<hgrid, kThreads, 0, st>>>(v, n, L.chunks, state, hist);
    ef_topk_select_kernel<0><<<1, kThreads, 0, st>>>(hist, state, kk);
    ef_topk_hist_kernel<1><<<hgrid, kThreads, 0, st>>>(v, n, L.chunks, state, hist + kBins);
    ef_topk_select_kernel<1><<<1, kThreads, 0, st>>>(hist + kBins, state, kk);
    ef_topk_hist_kernel<2><<<hgrid, kThreads, 0, st>>>(v, n, L.chunks, state, hist + 2 * kBins);
    ef_topk_select_kernel<2><<<1, kThreads, 0, st>>>(hist + 2 * kBins, state, kk);
    ef_topk_count_kernel<<<(unsigned)L.chunks, kThreads, 0, st>>>(v, n, state, cgt, ceq);
    ef_topk_scan_kernel<<<1, kScanThreads, 0, st>>>(cgt, ceq, pgt, peq, L.chunks);
    ef_topk_scatter_kernel<<<(unsigned)L.chunks, kThreads, 0, st>>>(v, n, state, pgt, peq,
                                                                    (long long*)idx_out, val_out, resid_out, kk);
    return cudaGetLastError() == cudaSuccess ? EF_OK : EF_ERR_CUDA;
}

}  // extern "C"
