// Top-k compressor with its error-feedback residual (Section 2, second example after
// Definition 1: the operator that keeps the k coordinates of largest absolute value; used in
// Algorithm 2 as  Delta = C(p),  e = p - Delta).
//
//   ef_topk_compress(v, n, k) -> idx[k] (increasing), val[k] = v[idx], resid = v - C(v)
//
// Among equal magnitudes the lower index is kept, so the result is unique and reproducible.
//
// Method (all integer work on the bit pattern of |v_j|, which orders like the magnitude):
//   1. radix select of the k-th largest key T, three digits of 11 + 11 + 9 bits:
//      a. histogram of the first digit over v; one CTA finds the bin P0, from the top, in which
//         the count reaches k.  Keys above that bin are kept for sure, keys below never; only the
//         keys IN the bin (the candidates, typically a few per cent of n) still matter.
//      b. second pass over v: histogram of the second digit of the candidates, the number of
//         sure keys per slice (the 512 elements of a 4096-element chunk that one warp handles),
//         and the candidates' keys copied to a compact list (one segment per slice; the order
//         inside a segment is arbitrary and nothing depends on it).  The third digit is then
//         histogrammed over the list, not over v.
//      Result: T and how many keys equal to T have to be kept (need_eq).
//   2. per slice the number of keys > T and == T, from the slice's sure count and its segment
//      of the list (no pass over v), and their totals per tile of 32 chunks;
//   3. a scan of the tile totals (one CTA);
//   4. a scatter pass: every warp recomputes the flags of its slices, ranks the kept elements in
//      index order (a shuffle scan of per-lane counts, no sorting) and writes idx, val and the
//      residual.
// Traffic: three reads of v, one write of the residual, k index/value pairs: about 16 bytes per
// element (the definition needs 8).  The list has room for n/8 candidates; when the bin holds
// more (e.g. a vector whose magnitudes are all equal) steps 1b's list is skipped and the third
// digit and the counts are taken from v itself (two more reads of v).  Which way a call goes is
// decided on the device, inside the kernels of the third digit and of the counts.
// Nothing waits on another CTA; kernel boundaries order the passes.
#include "ef_internal.h"

#include <algorithm>
#include <utility>
#include <type_traits>

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
    unsigned long long ncand;      // keys in the first digit's bin
    unsigned long long cursor;     // next free entry of the candidate list
    unsigned compact;              // 1: the candidates fit the list
};

constexpr int kTileOfChunks = 32;     // chunks per tile of the count scan
constexpr int kScatterChunks = 8;     // chunks per CTA of the scatter pass (divides kTileOfChunks)
static_assert(kTileOfChunks == 32 && kTileOfChunks % kScatterChunks == 0, "one warp adds a tile's counts");

struct TopkLayout {
    size_t off_hist = 0, off_state = 0, off_tgt = 0, off_teq = 0, off_cgt = 0, off_ceq = 0, off_pgt = 0,
           off_peq = 0, off_seg_start = 0, off_seg_cnt = 0, off_cand = 0, total = 0;
    long long chunks = 0, tiles = 0;
    unsigned long long cap = 0;    // entries of the candidate list
};

TopkLayout topk_layout(int64_t n) {
    TopkLayout L;
    L.chunks = (n + kChunkLen - 1) / kChunkLen;
    L.tiles = (L.chunks + kTileOfChunks - 1) / kTileOfChunks;
    // room for an eighth of the vector; short vectors always fit
    L.cap = (unsigned long long)std::max<int64_t>(n / 8, std::min<int64_t>(n, 65536));
    size_t o = 0;
    // zeroed at the start of every call: histograms, state, per-tile totals
    L.off_hist = o;  o += align_up(sizeof(unsigned long long) * kBins * kPasses);
    L.off_state = o; o += align_up(sizeof(TopkState));
    L.off_tgt = o;   o += align_up(sizeof(unsigned) * (size_t)L.tiles);
    L.off_teq = o;   o += align_up(sizeof(unsigned) * (size_t)L.tiles);
    // written before they are read; counts and list segments are kept per SLICE: the 512 elements
    // of a chunk that one warp handles (slice = chunk * kWarps + warp)
    L.off_cgt = o;   o += align_up(sizeof(unsigned) * (size_t)L.chunks * kWarps);
    L.off_ceq = o;   o += align_up(sizeof(unsigned) * (size_t)L.chunks * kWarps);
    L.off_pgt = o;   o += align_up(sizeof(unsigned long long) * (size_t)L.tiles);
    L.off_peq = o;   o += align_up(sizeof(unsigned long long) * (size_t)L.tiles);
    L.off_seg_start = o; o += align_up(sizeof(unsigned long long) * (size_t)L.chunks * kWarps);   // one segment
    L.off_seg_cnt = o;   o += align_up(sizeof(unsigned) * (size_t)L.chunks * kWarps);             // per warp and chunk
    L.off_cand = o;  o += align_up(sizeof(unsigned) * (size_t)L.cap);
    L.total = o;
    return L;
}

__device__ __forceinline__ unsigned key_of(float v) { return __float_as_uint(v) & 0x7fffffffu; }

// Loads the four elements of this lane's row; elements past n are flagged.
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

__device__ __forceinline__ unsigned warp_inclusive_scan32(unsigned v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned u = __shfl_up_sync(kFull, v, o);
        if (lane >= o) v += u;
    }
    return v;
}

// ---- 1a: histogram of digit PASS over the keys of v that match the prefix so far (a device
// function: the first pass is a kernel of its own, the third digit's fallback shares a kernel
// with the pass over the list).
template <int PASS>
__device__ __forceinline__ void hist_over_vector(const float* __restrict__ v, long long n, long long chunks,
                                                 unsigned prefix, unsigned* s_hist) {
    constexpr int shift = pass_shift(PASS), bits = pass_bits(PASS);
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
}

template <int PASS>
__global__ void __launch_bounds__(kThreads) ef_topk_hist_kernel(const float* __restrict__ v, long long n,
                                                                long long chunks,
                                                                const TopkState* __restrict__ st,
                                                                unsigned long long* __restrict__ hist) {
    __shared__ unsigned s_hist[kBins];
    for (int b = threadIdx.x; b < kBins; b += kThreads) s_hist[b] = 0u;
    __syncthreads();
    efk::pdl_enter();
    constexpr int bits = pass_bits(PASS);
    hist_over_vector<PASS>(v, n, chunks, PASS == 0 ? 0u : st->prefix, s_hist);
    __syncthreads();
    for (int b = threadIdx.x; b < (1 << bits); b += kThreads)
        if (s_hist[b]) atomicAdd(&hist[b], (unsigned long long)s_hist[b]);
}

// ---- Both passes below are bound by instruction issue, not by memory, if every element is
// classified by its own lane: only a few per cent of the elements matter (keys at or above the
// threshold bin resp. the threshold), but nearly every warp instruction of a per-element test
// has some lane that needs it.  So a lane first tests its four elements of a row together (the
// largest of the four keys against the bound), and the lanes whose row holds such a key copy the
// row to a staging area of their warp, packed densely in index order (ballot + population
// count).  The warp then classifies the staged rows, one row per lane: a handful of dense
// iterations instead of sixteen sparse ones.
struct WarpStage {
    uint4 row[128];                 // raw bits of the four elements of a staged lane-row
    unsigned short tag[128];        // (in-range nibble << 8) | (row u << 5) | lane
};

// Stages the lane-rows of this warp's part of a chunk whose largest key is >= lo (and that lie
// inside the vector).  Returns the number of staged rows (the same in every lane).
// FULL: the chunk lies wholly inside the vector (every chunk but the last): no range tests.
template <bool FULL>
__device__ __forceinline__ int stage_rows(const float (&x)[kU][4], unsigned fin, unsigned lo,
                                          WarpStage& st, int lane) {
    const unsigned lt_mask = (1u << lane) - 1u;
    int H = 0;
#pragma unroll
    for (int u = 0; u < kU; ++u) {
        const unsigned b0 = __float_as_uint(x[u][0]), b1 = __float_as_uint(x[u][1]),
                       b2 = __float_as_uint(x[u][2]), b3 = __float_as_uint(x[u][3]);
        const unsigned m = max(__vimax3_u32(b0 & 0x7fffffffu, b1 & 0x7fffffffu, b2 & 0x7fffffffu),
                               b3 & 0x7fffffffu);
        const unsigned nib = FULL ? 0xfu : (fin >> (4 * u)) & 0xfu;
        const bool hit = m >= lo && nib != 0u;
        const unsigned ballot = __ballot_sync(kFull, hit);
        if (hit) {
            const int e = H + __popc(ballot & lt_mask);
            st.row[e] = make_uint4(b0, b1, b2, b3);
            st.tag[e] = (unsigned short)((nib << 8) | (u << 5) | lane);
        }
        H += __popc(ballot);
    }
    __syncwarp();
    return H;
}

// ---- 1b. second pass over v.  Per chunk: histogram of the second digit of the candidates (keys
// whose first digit is P0), the number of sure keys (first digit > P0) into cgt, and -- if the
// candidates fit the list -- the candidates' keys on the list.

// This warp's 512 elements of chunk c, four rows of four per lane; fin: bit 4u + k = element exists.
__device__ __forceinline__ void load_chunk_keys(const float* __restrict__ v, long long n, long long c,
                                                int warp, int lane, float (&x)[kU][4], unsigned& fin) {
    if ((c + 1) * kChunkLen <= n) {            // the whole chunk is inside the vector
        const float* p = v + c * kChunkLen + warp * (128 * kU) + lane * 4;
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            const float4 q = efk::ld_stream(p + u * 128);
            x[u][0] = q.x; x[u][1] = q.y; x[u][2] = q.z; x[u][3] = q.w;
        }
        fin = 0xffffu;
        return;
    }
    fin = 0u;
#pragma unroll
    for (int u = 0; u < kU; ++u) {
        const long long base = c * kChunkLen + warp * (128 * kU) + u * 128 + lane * 4;
        bool in[4];
        if (base < n) load_keys(v, base, n, x[u], in);
        else {
#pragma unroll
            for (int k = 0; k < 4; ++k) { in[k] = false; x[u][k] = 0.f; }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) fin |= in[k] ? 1u << (4 * u + k) : 0u;
    }
}

// Every warp works for itself: it keeps its candidates of up to 32 chunks in a list of its own in
// shared memory, and when that is half full (or 32 chunks are logged) it reserves room on the
// global list with ONE atomic, copies the keys out and records where each logged chunk's keys
// went.  So a chunk has kWarps segments on the global list (one per warp), no CTA barrier lies on
// the path, and the global cursor sees one atomic per ~500 candidates.
constexpr int kWarpListKeys = 1024;     // a warp's slice of a chunk holds at most 512 keys: flushed above 512, it always fits
constexpr int kWarpListLog = 32;
struct WarpList {
    unsigned key[kWarpListKeys];
    long long seg[kWarpListLog];        // which segment (chunk * kWarps + warp) ...
    unsigned short off[kWarpListLog];   // ... starts where in key[] ...
    unsigned short cnt[kWarpListLog];   // ... and holds how many keys
};

__device__ __forceinline__ void flush_warp_list(WarpList& wl, int& fill, int& nlog, TopkState* st,
                                                unsigned long long* __restrict__ seg_start,
                                                unsigned* __restrict__ seg_cnt,
                                                unsigned* __restrict__ cand, int lane) {
    __syncwarp();
    if (fill > 0) {
        unsigned long long base = 0ull;
        if (lane == 0) base = atomicAdd(&st->cursor, (unsigned long long)fill);
        base = __shfl_sync(kFull, base, 0);
        for (int i = lane; i < fill; i += 32) cand[base + i] = wl.key[i];
        if (lane < nlog) {
            seg_start[wl.seg[lane]] = base + wl.off[lane];
            seg_cnt[wl.seg[lane]] = wl.cnt[lane];
        }
    }
    __syncwarp();
    fill = 0;
    nlog = 0;
}

__global__ void __launch_bounds__(kThreads) ef_topk_candidates_kernel(const float* __restrict__ v, long long n,
                                                                      long long chunks, TopkState* st,
                                                                      unsigned long long* __restrict__ hist,
                                                                      unsigned* __restrict__ cgt,
                                                                      unsigned long long* __restrict__ seg_start,
                                                                      unsigned* __restrict__ seg_cnt,
                                                                      unsigned* __restrict__ cand) {
    extern __shared__ __align__(16) unsigned char s_dyn[];
    // dynamic: [one list per warp][one staging area per warp]
    WarpList* s_lists = reinterpret_cast<WarpList*>(s_dyn);
    WarpStage* s_stage = reinterpret_cast<WarpStage*>(s_dyn + kWarps * sizeof(WarpList));
    __shared__ unsigned s_hist[kBins];
    for (int b = threadIdx.x; b < kBins; b += kThreads) s_hist[b] = 0u;
    efk::pdl_enter();
    const unsigned P0 = st->prefix;
    const unsigned lo = P0 << 20, hi_top = P0 + 1u;       // candidates: lo <= key and (key >> 20) < hi_top
    const bool compact = st->compact != 0u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    WarpStage& stage = s_stage[warp];
    WarpList& wl = s_lists[warp];
    float x[kU][4];
    unsigned fin = 0u;
    int fill = 0, nlog = 0;                    // the same in every lane of the warp
    if (blockIdx.x < chunks) load_chunk_keys(v, n, blockIdx.x, warp, lane, x, fin);
    __syncthreads();                           // the histogram is zero
    // the staged rows of this warp's slice of chunk c: second-digit histogram, candidates to the
    // warp's list, sure keys counted.  The next chunk's loads are issued once the rows are staged.
    auto classify = [&](auto full_c, long long c) {
        constexpr bool FULL = decltype(full_c)::value;
        if (compact && (fill > kWarpListKeys / 2 || nlog == kWarpListLog))
            flush_warp_list(wl, fill, nlog, st, seg_start, seg_cnt, cand, lane);
        const int H = stage_rows<FULL>(x, fin, lo, stage, lane);
        const long long next = c + gridDim.x;
        if (next < chunks) load_chunk_keys(v, n, next, warp, lane, x, fin);
        unsigned gt = 0u;
        const int fill0 = fill;
        for (int e0 = 0; e0 < H; e0 += 32) {
            const int e = e0 + lane;
            unsigned keys[4] = {0u, 0u, 0u, 0u};
            unsigned mine = 0u;                // bit k: element k of the staged row is a candidate
            if (e < H) {
                const uint4 q = stage.row[e];
                const unsigned nib = FULL ? 0xfu : stage.tag[e] >> 8;
                keys[0] = q.x & 0x7fffffffu; keys[1] = q.y & 0x7fffffffu;
                keys[2] = q.z & 0x7fffffffu; keys[3] = q.w & 0x7fffffffu;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const bool in = (nib >> k) & 1u;
                    const unsigned top = keys[k] >> 20;
                    gt += (in && top >= hi_top) ? 1u : 0u;
                    if (in && top == P0) {
                        mine |= 1u << k;
                        atomicAdd(&s_hist[(keys[k] >> 9) & (kBins - 1)], 1u);
                    }
                }
            }
            if (compact && __any_sync(kFull, mine != 0u)) {
                const unsigned cnt = (unsigned)__popc(mine);
                const unsigned incl = warp_inclusive_scan32(cnt, lane);
                int pos = fill + (int)(incl - cnt);
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if ((mine >> k) & 1u) wl.key[pos++] = keys[k];
                fill += (int)__shfl_sync(kFull, incl, 31);
            }
        }
        __syncwarp();                          // the staging area is rewritten by the next chunk
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) gt += __shfl_xor_sync(kFull, gt, o);
        if (lane == 0) {
            const long long seg = c * kWarps + warp;
            cgt[seg] = gt;
            if (!compact || fill == fill0) seg_cnt[seg] = 0u;
            else {
                wl.seg[nlog] = seg;
                wl.off[nlog] = (unsigned short)fill0;
                wl.cnt[nlog] = (unsigned short)(fill - fill0);
            }
        }
        if (compact && fill != fill0) nlog += 1;
    };
    for (long long c = blockIdx.x; c < chunks; c += gridDim.x) {
        // the choice must be the same in every thread of a warp (the paths hold warp-wide
        // operations): it is made on the chunk, not on the thread's own range flags
        if ((c + 1) * kChunkLen <= n) classify(std::true_type{}, c);
        else classify(std::false_type{}, c);
    }
    if (compact) flush_warp_list(wl, fill, nlog, st, seg_start, seg_cnt, cand, lane);
    __syncthreads();
    for (int b = threadIdx.x; b < kBins; b += kThreads)
        if (s_hist[b]) atomicAdd(&hist[b], (unsigned long long)s_hist[b]);
}
constexpr size_t kCandidatesSmem = kWarps * (sizeof(WarpList) + sizeof(WarpStage));

// ---- 1b, third digit: histogram over the candidate list, or over v when the list was not used.
__global__ void __launch_bounds__(kThreads) ef_topk_third_digit_kernel(const float* __restrict__ v, long long n,
                                                                       long long chunks,
                                                                       const unsigned* __restrict__ cand,
                                                                       const TopkState* __restrict__ st,
                                                                       unsigned long long* __restrict__ hist) {
    constexpr int nbins = 1 << pass_bits(2);
    __shared__ unsigned s_hist[nbins];
    for (int b = threadIdx.x; b < nbins; b += kThreads) s_hist[b] = 0u;
    __syncthreads();
    efk::pdl_enter();
    const unsigned prefix = st->prefix;            // 22 bits
    if (st->compact) {
        const unsigned long long ncand = st->ncand;
        for (unsigned long long i = (unsigned long long)blockIdx.x * kThreads + threadIdx.x; i < ncand;
             i += (unsigned long long)gridDim.x * kThreads) {
            const unsigned key = cand[i];
            if ((key >> pass_bits(2)) == prefix) atomicAdd(&s_hist[key & (nbins - 1u)], 1u);
        }
    } else {
        hist_over_vector<2>(v, n, chunks, prefix, s_hist);
    }
    __syncthreads();
    for (int b = threadIdx.x; b < nbins; b += kThreads)
        if (s_hist[b]) atomicAdd(&hist[b], (unsigned long long)s_hist[b]);
}

// One CTA fixes the next digit: it finds, from the largest digit down, the bin in which the
// count of keys seen so far reaches `remaining`.  Thread t adds up the eight bins of group
// 255 - t (so thread order is from the top down); a scan over the threads gives every group the
// count above it, the one thread whose group holds the crossing walks its eight bins.
template <int PASS>
__global__ void __launch_bounds__(kThreads) ef_topk_select_kernel(const unsigned long long* __restrict__ hist,
                                                                  TopkState* st, unsigned long long k,
                                                                  unsigned long long cap) {
    constexpr int bits = pass_bits(PASS), nbins = 1 << bits, per = kBins / kThreads;
    __shared__ unsigned long long s_warp[kWarps];
    __shared__ int s_found;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int grp = kThreads - 1 - threadIdx.x;
    efk::pdl_enter();
    unsigned long long bin[per];
    unsigned long long g = 0;
#pragma unroll
    for (int j = 0; j < per; ++j) {
        const int b = grp * per + j;
        bin[j] = b < nbins ? hist[b] : 0ull;
        g += bin[j];
    }
    if (threadIdx.x == 0) s_found = 0;
    unsigned long long incl = g;               // keys in this group and all groups above it
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long u = __shfl_up_sync(kFull, incl, o);
        if (lane >= o) incl += u;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    for (int w = 0; w < warp; ++w) incl += s_warp[w];
    const unsigned long long remaining = PASS == 0 ? k : st->remaining;
    unsigned long long above = incl - g;
    // the crossing group; if the counts never reach `remaining` (they always do for k <= n) the lowest group
    const bool mine = above < remaining && (incl >= remaining || grp == 0);
    if (!mine) return;
    if (atomicExch(&s_found, 1) != 0) return;  // defensive: exactly one thread writes
    int j = per - 1;
    for (; j > 0; --j) {
        if (above + bin[j] >= remaining) break;
        above += bin[j];
    }
    const unsigned prefix = PASS == 0 ? 0u : st->prefix;
    st->prefix = (prefix << bits) | (unsigned)(grp * per + j);
    st->remaining = remaining - above;         // still to keep among the keys of the bin
    if (PASS == 0) {
        st->ncand = bin[j];
        st->compact = bin[j] <= cap ? 1u : 0u;
    }
    if (PASS == kPasses - 1) {
        st->threshold = st->prefix;
        st->need_eq = remaining - above;
    }
}

// ---- 2. per slice (the 512 elements of a chunk that one warp handles): how many keys are > T and
// == T, and the totals per tile for the scan.  A CTA takes kWarps consecutive chunks.  With the
// list: one warp per chunk, four lanes per slice, adds the slice's candidates above T to its sure
// count.  Without: the CTA counts its chunks in v one by one, every warp its own slice.
__global__ void __launch_bounds__(kThreads) ef_topk_count_kernel(const float* __restrict__ v, long long n,
                                                                 long long chunks,
                                                                 const unsigned* __restrict__ cand,
                                                                 const TopkState* __restrict__ st,
                                                                 const unsigned long long* __restrict__ seg_start,
                                                                 const unsigned* __restrict__ seg_cnt,
                                                                 unsigned* __restrict__ cgt,
                                                                 unsigned* __restrict__ ceq,
                                                                 unsigned* __restrict__ tgt,
                                                                 unsigned* __restrict__ teq) {
    efk::pdl_enter();
    const unsigned T = st->threshold;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (st->compact) {
        const long long c = (long long)blockIdx.x * kWarps + warp;
        if (c >= chunks) return;
        // the chunk's kWarps slices, four lanes each
        static_assert(kWarps == 8, "four lanes per slice");
        const long long sl = c * kWarps + (lane >> 2);
        const unsigned cnt = seg_cnt[sl];
        const unsigned* seg = cand + (cnt ? seg_start[sl] : 0ull);
        unsigned both = 0u;                   // at most 512 each: two 16-bit fields
        for (unsigned i = lane & 3; i < cnt; i += 4) {
            const unsigned key = seg[i];
            both += (key > T ? 1u : 0u) + (key == T ? 1u << 16 : 0u);
        }
        both += __shfl_xor_sync(kFull, both, 1);
        both += __shfl_xor_sync(kFull, both, 2);
        if ((lane & 3) == 0) {
            both += cgt[sl];                  // the slice's sure keys
            cgt[sl] = both & 0xffffu;
            ceq[sl] = both >> 16;
        } else {
            both = 0u;
        }
#pragma unroll
        for (int o = 16; o > 2; o >>= 1) both += __shfl_xor_sync(kFull, both, o);
        if (lane == 0) {                      // at most 4096 each
            if (both & 0xffffu) atomicAdd(&tgt[c / kTileOfChunks], both & 0xffffu);
            if (both >> 16) atomicAdd(&teq[c / kTileOfChunks], both >> 16);
        }
        return;
    }
    for (int j = 0; j < kWarps; ++j) {
        const long long c = (long long)blockIdx.x * kWarps + j;
        if (c >= chunks) return;
        unsigned gt = 0, eq = 0;
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            const long long base = c * kChunkLen + warp * (128 * kU) + u * 128 + lane * 4;
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
        unsigned both = gt | (eq << 16);      // at most 512 elements per warp each: two 16-bit fields
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) both += __shfl_xor_sync(kFull, both, o);
        if (lane == 0) {
            cgt[c * kWarps + warp] = both & 0xffffu;
            ceq[c * kWarps + warp] = both >> 16;
            if (both & 0xffffu) atomicAdd(&tgt[c / kTileOfChunks], both & 0xffffu);
            if (both >> 16) atomicAdd(&teq[c / kTileOfChunks], both >> 16);
        }
    }
}

// ---- 3. exclusive prefix sums of the two per-tile count arrays (a tile is kTileOfChunks chunks;
// one CTA).  The CTA walks the arrays in pieces of kScanThreads * kScanPer entries: every thread takes kScanPer
// consecutive entries, the threads' totals are scanned over the CTA (warps, then the warps'
// totals), and the piece's total is carried to the next piece.
constexpr int kScanThreads = 1024;
constexpr int kScanPer = 8;
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
    __shared__ unsigned long long s_carry[2];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) { s_carry[0] = 0ull; s_carry[1] = 0ull; }
    __syncthreads();
    efk::pdl_enter();
    for (long long piece = 0; piece < chunks; piece += (long long)kScanThreads * kScanPer) {
        const long long lo = piece + (long long)threadIdx.x * kScanPer;
        unsigned ga[kScanPer], gb[kScanPer];
        unsigned long long a = 0, b = 0;
#pragma unroll
        for (int j = 0; j < kScanPer; ++j) {
            ga[j] = lo + j < chunks ? cgt[lo + j] : 0u;
            gb[j] = lo + j < chunks ? ceq[lo + j] : 0u;
            a += ga[j]; b += gb[j];
        }
        const unsigned long long ia = warp_inclusive_scan(a, lane), ib = warp_inclusive_scan(b, lane);
        if (lane == 31) { s_a[warp] = ia; s_b[warp] = ib; }
        __syncthreads();
        if (warp == 0) {
            const unsigned long long ta = s_a[lane], tb = s_b[lane];
            const unsigned long long wa = warp_inclusive_scan(ta, lane), wb = warp_inclusive_scan(tb, lane);
            s_a[lane] = wa - ta;               // exclusive
            s_b[lane] = wb - tb;
        }
        __syncthreads();
        a = s_carry[0] + s_a[warp] + ia - a;   // entries before this thread's first one
        b = s_carry[1] + s_b[warp] + ib - b;
#pragma unroll
        for (int j = 0; j < kScanPer; ++j) {
            if (lo + j < chunks) { pgt[lo + j] = a; peq[lo + j] = b; }
            a += ga[j]; b += gb[j];
        }
        __syncthreads();                       // everyone has read the carry and the warp offsets
        if (threadIdx.x == kScanThreads - 1) { s_carry[0] = a; s_carry[1] = b; }
        __syncthreads();
    }
}

// ---- 4. scatter: kept = key > T, or key == T and fewer than need_eq equal keys precede it.
// Element order inside a chunk: warp, then row, then lane, then the lane's four elements, i.e.
// slice after slice.  A CTA handles kScatterChunks consecutive chunks; every warp walks its own
// slices of them with the next slice's loads in flight, without any CTA barrier: the number of
// kept keys before each slice is known up front from the per-slice counts (the tile's prefix,
// the tile's slices before the CTA's, and a scan over the CTA's own 64 slices by its first warp).
struct ScatterArgs {
    const float* v;
    long long n, chunks;
    const TopkState* st;
    const unsigned* cgt;               // per slice
    const unsigned* ceq;
    const unsigned long long* pgt;     // per tile
    const unsigned long long* peq;
    long long* idx_out;
    float* val_out;
    float* resid;                      // may alias v: every thread has read its own elements before it writes them
    unsigned long long kmax;
};

// One slice (this warp's 512 elements of chunk c), its elements in x/fin.  gt_base / eq_base: keys
// > T and == T before the slice.  Lane-rows without a key >= T keep nothing: their residual is the
// input, stored at once.  The others are staged in index order and handled one row per lane:
// ranks are running counts from one shuffle scan per 32 staged rows.
template <bool FULL>
__device__ __forceinline__ void scatter_slice(const ScatterArgs& a, long long c, unsigned T,
                                              unsigned long long need_eq, const float (&x)[kU][4],
                                              unsigned fin, WarpStage& stage,
                                              unsigned long long gt_base, unsigned long long eq_base) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long wbase = c * kChunkLen + warp * (128 * kU);
    const int H = stage_rows<FULL>(x, fin, T, stage, lane);
    // residual of the rows that keep nothing (a staged row is recognised by its largest key again)
    if (a.resid != nullptr) {
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            const long long base = wbase + u * 128 + lane * 4;
            const unsigned nib = FULL ? 0xfu : (fin >> (4 * u)) & 0xfu;
            const unsigned m = max(__vimax3_u32(__float_as_uint(x[u][0]) & 0x7fffffffu,
                                                __float_as_uint(x[u][1]) & 0x7fffffffu,
                                                __float_as_uint(x[u][2]) & 0x7fffffffu),
                                   __float_as_uint(x[u][3]) & 0x7fffffffu);
            if (m >= T || nib == 0u) continue;
            if (nib == 0xfu) efk::st_stream(a.resid + base, make_float4(x[u][0], x[u][1], x[u][2], x[u][3]));
            else
                for (int k = 0; k < 4; ++k) if ((nib >> k) & 1u) a.resid[base + k] = x[u][k];
        }
    }
    // position of a kept element = gt_rank + min(eq_rank, need_eq), split into a 64-bit part that
    // is fixed for the slice and small local counts:
    //   gt_base + min(eq_base, need_eq)  +  gt_local + min(eq_local, eq_room)
    const unsigned long long pos_base = gt_base + (eq_base < need_eq ? eq_base : need_eq);
    const unsigned eq_room = eq_base < need_eq ? (unsigned)min(need_eq - eq_base, 1024ull) : 0u;
    unsigned gt_local = 0u, eq_local = 0u;     // staged keys > T / == T in the rows before this iteration
    for (int e0 = 0; e0 < H; e0 += 32) {
        const int e = e0 + lane;
        uint4 q = make_uint4(0u, 0u, 0u, 0u);
        unsigned tag = 0u, fgt = 0u, feq = 0u;
        if (e < H) {
            q = stage.row[e];
            tag = stage.tag[e];
            const unsigned key[4] = {q.x & 0x7fffffffu, q.y & 0x7fffffffu, q.z & 0x7fffffffu, q.w & 0x7fffffffu};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                fgt |= key[k] > T ? 1u << k : 0u;
                feq |= key[k] == T ? 1u << k : 0u;
            }
            if (!FULL) { fgt &= tag >> 8; feq &= tag >> 8; }
        }
        const unsigned cnt = (unsigned)__popc(fgt) | ((unsigned)__popc(feq) << 16);
        const unsigned incl = warp_inclusive_scan32(cnt, lane);
        const unsigned tot = __shfl_sync(kFull, incl, 31);
        if (e < H) {
            unsigned gt_rank = gt_local + ((incl - cnt) & 0xffffu);
            unsigned eq_rank = eq_local + ((incl - cnt) >> 16);
            const long long base = wbase + ((tag >> 5) & 3u) * 128 + (tag & 31u) * 4;
            const float xv[4] = {__uint_as_float(q.x), __uint_as_float(q.y), __uint_as_float(q.z), __uint_as_float(q.w)};
            float r[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const bool is_eq = (feq >> k) & 1u, is_gt = (fgt >> k) & 1u;
                const bool kept = is_gt || (is_eq && eq_rank < eq_room);
                if (kept) {
                    const unsigned long long pos = pos_base + gt_rank + (eq_rank < eq_room ? eq_rank : eq_room);
                    if (pos < a.kmax) {        // always true when the counts are consistent
                        a.idx_out[pos] = base + k;
                        a.val_out[pos] = xv[k];
                    }
                }
                r[k] = kept ? __fsub_rn(xv[k], xv[k]) : xv[k];      // e = v - C(v)
                eq_rank += is_eq ? 1u : 0u;
                gt_rank += is_gt ? 1u : 0u;
            }
            if (a.resid != nullptr) {
                if (FULL || (tag >> 8) == 0xfu) efk::st_stream(a.resid + base, make_float4(r[0], r[1], r[2], r[3]));
                else
                    for (int k = 0; k < 4; ++k) if ((tag >> (8 + k)) & 1u) a.resid[base + k] = r[k];
            }
        }
        gt_local += tot & 0xffffu;
        eq_local += tot >> 16;
    }
    __syncwarp();                              // the staging area is rewritten by the next slice
}

__global__ void __launch_bounds__(kThreads, 3) ef_topk_scatter_kernel(const ScatterArgs a) {
    constexpr int kSlices = kScatterChunks * kWarps;            // 64: two per lane of the first warp
    static_assert(kSlices == 64, "the first warp scans two slices per lane");
    __shared__ unsigned long long s_gt[kSlices], s_eq[kSlices]; // keys > T / == T before each slice of the CTA
    __shared__ WarpStage s_stage[kWarps];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long c0 = (long long)blockIdx.x * kScatterChunks;
    const int nch = (int)min((long long)kScatterChunks, a.chunks - c0);
    float xA[kU][4], xB[kU][4];
    unsigned finA, finB = 0u;
    efk::pdl_enter();
    load_chunk_keys(a.v, a.n, c0, warp, lane, xA, finA);
    if (warp == 0) {
        // before the CTA's first slice: the tile's prefix plus the tile's slices before it
        const long long tile = c0 / kTileOfChunks, first = tile * kTileOfChunks * kWarps, mine = c0 * kWarps;
        unsigned long long g = 0ull, e = 0ull;
        for (long long i = first + lane; i < mine; i += 32) { g += a.cgt[i]; e += a.ceq[i]; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            g += __shfl_xor_sync(kFull, g, o);
            e += __shfl_xor_sync(kFull, e, o);
        }
        g += a.pgt[tile];
        e += a.peq[tile];
        // exclusive scan over the CTA's own slices, lane l holding slices 2l and 2l + 1
        const long long last = a.chunks * kWarps;
        const unsigned g0 = mine + 2 * lane < last ? a.cgt[mine + 2 * lane] : 0u;
        const unsigned g1 = mine + 2 * lane + 1 < last ? a.cgt[mine + 2 * lane + 1] : 0u;
        const unsigned e0 = mine + 2 * lane < last ? a.ceq[mine + 2 * lane] : 0u;
        const unsigned e1 = mine + 2 * lane + 1 < last ? a.ceq[mine + 2 * lane + 1] : 0u;
        const unsigned ig = warp_inclusive_scan32(g0 + g1, lane), ie = warp_inclusive_scan32(e0 + e1, lane);
        s_gt[2 * lane] = g + (ig - g0 - g1);
        s_gt[2 * lane + 1] = g + (ig - g1);
        s_eq[2 * lane] = e + (ie - e0 - e1);
        s_eq[2 * lane + 1] = e + (ie - e1);
    }
    const unsigned T = a.st->threshold;
    const unsigned long long need_eq = a.st->need_eq;
    __syncthreads();                           // the only barrier: from here on every warp runs for itself
    for (int j = 0; j < nch; j += 2) {
        if (j + 1 < nch) load_chunk_keys(a.v, a.n, c0 + j + 1, warp, lane, xB, finB);
        // whole chunk or not: decided on the chunk, identically in every lane (the paths hold warp-wide operations)
        if ((c0 + j + 1) * kChunkLen <= a.n)
            scatter_slice<true>(a, c0 + j, T, need_eq, xA, finA, s_stage[warp], s_gt[j * kWarps + warp], s_eq[j * kWarps + warp]);
        else
            scatter_slice<false>(a, c0 + j, T, need_eq, xA, finA, s_stage[warp], s_gt[j * kWarps + warp], s_eq[j * kWarps + warp]);
        if (j + 1 < nch) {
            if (j + 2 < nch) load_chunk_keys(a.v, a.n, c0 + j + 2, warp, lane, xA, finA);
            if ((c0 + j + 2) * kChunkLen <= a.n)
                scatter_slice<true>(a, c0 + j + 1, T, need_eq, xB, finB, s_stage[warp], s_gt[(j + 1) * kWarps + warp], s_eq[(j + 1) * kWarps + warp]);
            else
                scatter_slice<false>(a, c0 + j + 1, T, need_eq, xB, finB, s_stage[warp], s_gt[(j + 1) * kWarps + warp], s_eq[(j + 1) * kWarps + warp]);
        }
    }
}

// ---- short vectors: everything in ONE CTA.  Up to kSmallN elements the nine launches above
// cost more than the work; here one CTA of 1024 threads runs the three digit passes over v
// (shared-memory histogram, selection by a scan over the CTA; v is re-read from L2), then goes
// through v once more in index order, 4096 elements per round, ranks the kept elements (a scan
// within each warp, then over the warps' totals, running totals over the rounds) and writes idx,
// val and the residual.  Same keys, same tie rule, hence the same result as the general path.
// (All keys of a vector fall into a few dozen bins of the first digit, so the histogram's
// shared-memory atomics serialise: the cost grows with n and the general path wins from about
// 2^15 elements on.  Keeping the vector in registers across the passes did not change that.)
constexpr int kSmallThreads = 1024;
constexpr long long kSmallN = 16384;

__global__ void __launch_bounds__(kSmallThreads) ef_topk_small_kernel(const float* v, long long n,
                                                                      unsigned long long k,
                                                                      long long* __restrict__ idx_out,
                                                                      float* __restrict__ val_out, float* resid) {
    __shared__ unsigned s_hist[kBins];
    __shared__ unsigned s_warp[32];            // per-warp totals (histogram scan, then packed gt | eq << 16)
    __shared__ unsigned s_prefix, s_remaining;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned prefix = 0u, remaining = (unsigned)k;          // k <= n <= kSmallN
#pragma unroll 1
    for (int pass = 0; pass < kPasses; ++pass) {
        const int shift = pass_shift(pass), bits = pass_bits(pass);
        for (int b = tid; b < kBins; b += kSmallThreads) s_hist[b] = 0u;
        __syncthreads();
        for (long long i = 4LL * tid; i < n; i += 4 * kSmallThreads) {
            float x[4]; bool in[4];
            load_keys(v, i, n, x, in);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const unsigned key = key_of(x[j]);
                if (in[j] && (pass == 0 || (key >> (shift + bits)) == prefix))
                    atomicAdd(&s_hist[(key >> shift) & ((1u << bits) - 1u)], 1u);
            }
        }
        __syncthreads();
        // thread t owns bins 2047 - 2t and 2046 - 2t: from the top down; scan over the CTA
        const unsigned h0 = s_hist[kBins - 1 - 2 * tid], h1 = s_hist[kBins - 2 - 2 * tid];
        unsigned incl = warp_inclusive_scan32(h0 + h1, lane);
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            const unsigned t = s_warp[lane];
            const unsigned w = warp_inclusive_scan32(t, lane);
            s_warp[lane] = w - t;              // exclusive
        }
        __syncthreads();
        incl += s_warp[warp];
        const unsigned above = incl - h0 - h1; // keys in the bins above this thread's pair
        // the bin in which the count from the top reaches `remaining`
        if (above < remaining && incl >= remaining) {
            const bool first = above + h0 >= remaining;
            const unsigned bin = kBins - 1 - 2 * tid - (first ? 0 : 1);
            s_prefix = (prefix << bits) | bin;
            s_remaining = remaining - above - (first ? 0u : h0);
        }
        __syncthreads();
        prefix = s_prefix;
        remaining = s_remaining;
        __syncthreads();
    }
    const unsigned T = prefix;
    const unsigned need_eq = remaining;
    unsigned gt_run = 0u, eq_run = 0u;         // keys > T / == T before this round
    for (long long base0 = 0; base0 < n; base0 += 4 * kSmallThreads) {
        const long long base = base0 + 4 * tid;
        float x[4] = {0.f, 0.f, 0.f, 0.f};
        bool in[4] = {false, false, false, false};
        if (base < n) load_keys(v, base, n, x, in);
        unsigned fgt = 0u, feq = 0u, nib = 0u;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const unsigned key = key_of(x[j]);
            nib |= in[j] ? 1u << j : 0u;
            fgt |= key > T ? 1u << j : 0u;
            feq |= key == T ? 1u << j : 0u;
        }
        fgt &= nib; feq &= nib;
        const unsigned cnt = (unsigned)__popc(fgt) | ((unsigned)__popc(feq) << 16);
        const unsigned incl = warp_inclusive_scan32(cnt, lane);
        __syncthreads();                       // the previous round's totals have been read
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        unsigned before = 0u, total = 0u;
#pragma unroll 8
        for (int w = 0; w < 32; ++w) {
            const unsigned t = s_warp[w];
            before += w < warp ? t : 0u;
            total += t;
        }
        unsigned gt_rank = gt_run + ((before + incl - cnt) & 0xffffu);
        unsigned eq_rank = eq_run + ((before + incl - cnt) >> 16);
        float y[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const bool is_gt = (fgt >> j) & 1u, is_eq = (feq >> j) & 1u;
            const bool kept = is_gt || (is_eq && eq_rank < need_eq);
            if (kept) {
                const unsigned long long pos = (unsigned long long)gt_rank + (eq_rank < need_eq ? eq_rank : need_eq);
                if (pos < k) {                 // always true when the counts are consistent
                    idx_out[pos] = base + j;
                    val_out[pos] = x[j];
                }
            }
            y[j] = kept ? __fsub_rn(x[j], x[j]) : x[j];        // e = v - C(v)
            gt_rank += is_gt ? 1u : 0u;
            eq_rank += is_eq ? 1u : 0u;
        }
        if (resid != nullptr && nib != 0u) {
            if (nib == 0xfu) *reinterpret_cast<float4*>(resid + base) = make_float4(y[0], y[1], y[2], y[3]);
            else
                for (int j = 0; j < 4; ++j) if ((nib >> j) & 1u) resid[base + j] = y[j];
        }
        gt_run += total & 0xffffu;
        eq_run += total >> 16;
    }
}

// Launch with programmatic stream serialization: every kernel of the call starts with
// efk::pdl_enter() (or sets up its shared memory first), so a kernel's launch latency and set-up
// overlap the tail of the one before it and its reads still follow that kernel's completion.
template <typename... KArgs, typename... Args>
cudaError_t launch_after(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t st,
                         Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
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
    EF_API_RANGE();
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
    {
        // the candidates kernel needs more dynamic shared memory than the default limit: once per device
        static bool raised[64] = {};
        if (dev < 0 || dev >= 64) return EF_ERR_UNSUPPORTED_DEVICE;
        if (!raised[dev]) {
            if (cudaFuncSetAttribute(ef_topk_candidates_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)kCandidatesSmem) != cudaSuccess)
                return EF_ERR_CUDA;
            raised[dev] = true;
        }
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (n <= kSmallN) {                        // short vectors: one CTA does it all (the workspace stays unused)
        ef_topk_small_kernel<<<1, kSmallThreads, 0, st>>>(v, n, (unsigned long long)k, (long long*)idx_out,
                                                          val_out, resid_out);
        return cudaGetLastError() == cudaSuccess ? EF_OK : EF_ERR_CUDA;
    }
    char* ws = (char*)workspace;
    unsigned long long* hist = (unsigned long long*)(ws + L.off_hist);
    TopkState* state = (TopkState*)(ws + L.off_state);
    unsigned* tgt = (unsigned*)(ws + L.off_tgt);
    unsigned* teq = (unsigned*)(ws + L.off_teq);
    unsigned* cgt = (unsigned*)(ws + L.off_cgt);
    unsigned* ceq = (unsigned*)(ws + L.off_ceq);
    unsigned long long* pgt = (unsigned long long*)(ws + L.off_pgt);
    unsigned long long* peq = (unsigned long long*)(ws + L.off_peq);
    unsigned long long* seg_start = (unsigned long long*)(ws + L.off_seg_start);
    unsigned* seg_cnt = (unsigned*)(ws + L.off_seg_cnt);
    unsigned* cand = (unsigned*)(ws + L.off_cand);
    if (cudaMemsetAsync(ws, 0, L.off_cgt, st) != cudaSuccess) return EF_ERR_CUDA;   // histograms, state, tile totals
    const unsigned hgrid = (unsigned)std::min<long long>(L.chunks, 148 * 8);
    const unsigned cgrid = (unsigned)std::min<long long>(L.chunks, 148 * 3);       // three CTAs of 59 KB per SM
    const unsigned long long kk = (unsigned long long)k;
    launch_after(ef_topk_hist_kernel<0>, hgrid, kThreads, 0, st, v, (long long)n, L.chunks, (const TopkState*)state, hist);
    launch_after(ef_topk_select_kernel<0>, 1, kThreads, 0, st, (const unsigned long long*)hist, state, kk, L.cap);
    launch_after(ef_topk_candidates_kernel, cgrid, kThreads, kCandidatesSmem, st, v, (long long)n, L.chunks, state,
                 hist + kBins, cgt, seg_start, seg_cnt, cand);
    launch_after(ef_topk_select_kernel<1>, 1, kThreads, 0, st, (const unsigned long long*)(hist + kBins), state, kk, L.cap);
    launch_after(ef_topk_third_digit_kernel, hgrid, kThreads, 0, st, v, (long long)n, L.chunks, (const unsigned*)cand,
                 (const TopkState*)state, hist + 2 * kBins);
    launch_after(ef_topk_select_kernel<2>, 1, kThreads, 0, st, (const unsigned long long*)(hist + 2 * kBins), state, kk,
                 L.cap);
    launch_after(ef_topk_count_kernel, (unsigned)((L.chunks + kWarps - 1) / kWarps), kThreads, 0, st, v, (long long)n,
                 L.chunks, (const unsigned*)cand, (const TopkState*)state, (const unsigned long long*)seg_start,
                 (const unsigned*)seg_cnt, cgt, ceq, tgt, teq);
    launch_after(ef_topk_scan_kernel, 1, kScanThreads, 0, st, (const unsigned*)tgt, (const unsigned*)teq, pgt, peq,
                 L.tiles);
    ScatterArgs sa;
    sa.v = v; sa.n = n; sa.chunks = L.chunks; sa.st = state; sa.cgt = cgt; sa.ceq = ceq; sa.pgt = pgt; sa.peq = peq;
    sa.idx_out = (long long*)idx_out; sa.val_out = val_out; sa.resid = resid_out; sa.kmax = kk;
    launch_after(ef_topk_scatter_kernel, (unsigned)((L.chunks + kScatterChunks - 1) / kScatterChunks), kThreads, 0, st,
                 sa);
    return cudaGetLastError() == cudaSuccess ? EF_OK : EF_ERR_CUDA;
}

}  // extern "C"
