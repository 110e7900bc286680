// CPU oracle for the two comparison compressors the paper names next to its own:
//   * signSGD / signum with majority vote (Section 1 "Related work"; baselines (iii), (iv) of
//     Section 4.1 and baseline (ii) of Section 4.2; Table 1: 2Md bits per iteration), and
//   * the top-k operator, the second example of a delta-approximate compressor after
//     Definition 1 (Section 2): it "only preserves the k coordinates with the largest absolute
//     values".
//
// TEST INFRASTRUCTURE ONLY.  Plain, slow, single-threaded; shares no code with the CUDA library
// and is never linked, imported or executed by the product path.
//
// ---- signum with majority vote -----------------------------------------------------------
// The paper does not print the algorithm (it cites it); what it fixes is: only the 1-bit
// gradient sign travels in both directions (Section 1), the momentum variant is called signum,
// the cost is 2Md bits per iteration (Table 1), and with an odd number of workers a majority
// vote never produces zero (Section 4.2).  Written out, one iteration is
//   worker i :  m_{t,i} = mu m_{t-1,i} + g_{t,i}          (momentum in the form Section 3.3 uses)
//               push sign(m_{t,i})                         (1 bit per coordinate)
//   server   :  v_t = sign( sum_i sign(m_{t,i}) )          (coordinate-wise majority), push v_t
//   worker   :  x_{t+1} = x_t - eta v_t
// mu = 0 gives signSGD with majority vote.
// Readings where the paper is silent (conventions of this repository, PARITY UNPINNED BY THE
// PAPER):
//   * sign(+-0) = +1 on the workers, as in the blockwise compressor (Appendix A: signs in
//     {-1,+1}, one bit);
//   * a tie of the vote (even M only) is sent as +1: the message is 1 bit per coordinate, so it
//     cannot carry the zero the vote would produce, which is the loss Section 4.2 alludes to;
//   * the momentum is m = mu m + g rather than the cited work's m = beta m + (1-beta) g; the two
//     differ by the positive factor 1/(1-beta), which no sign depends on;
//   * packed layout and block partition exactly as in ef_oracle.cpp (blocks only fix where
//     words start; the method itself never looks at them);
//   * element arithmetic in binary32: m = fmaf(mu, m, g), x = x -+ eta.
//
// ---- top-k ---------------------------------------------------------------------------------
// C(v) keeps the k entries of largest |v_j| and zeroes the others; the error-feedback residual
// is e = v - C(v) (Algorithm 2, worker lines 3 and 5, with C = top-k).  Readings: among equal
// magnitudes the lower index wins (the paper does not say; PARITY UNPINNED); +0 and -0 have the
// same magnitude; the kept entries are listed in increasing index order; NaN is unspecified.
//
// Build: g++ -O2 -ffp-contract=off -shared -fPIC (together with ef_oracle.cpp).

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <new>
#include <numeric>
#include <vector>

namespace {

struct Signum {
    int64_t d = 0, W = 0, t = 0;
    int32_t B = 0, M = 0;
    float mu = 0.f, eta = 0.f;
    std::vector<int64_t> off, woff;
    std::vector<float> x;
    std::vector<std::vector<float>> m;
    std::vector<std::vector<uint32_t>> words;
    std::vector<uint32_t> swords;
    std::vector<uint8_t> stepped;
};

}  // namespace

extern "C" {

void* sgo_init(int64_t d, int32_t B, const int64_t* offsets, int32_t M, float mu, float eta)
{
    if (d < 1 || B < 1 || M < 1 || !offsets || offsets[0] != 0 || offsets[B] != d) return nullptr;
    for (int32_t b = 0; b < B; ++b) if (offsets[b + 1] <= offsets[b]) return nullptr;
    if (!(mu >= 0.f && mu < 1.f) || !(eta > 0.f) || !std::isfinite(eta)) return nullptr;
    Signum* o = new (std::nothrow) Signum();
    if (!o) return nullptr;
    o->d = d; o->B = B; o->M = M; o->mu = mu; o->eta = eta;
    o->off.assign(offsets, offsets + B + 1);
    o->woff.assign(B + 1, 0);
    for (int32_t b = 0; b < B; ++b)
        o->woff[b + 1] = o->woff[b] + (offsets[b + 1] - offsets[b] + 31) / 32;
    o->W = o->woff[B];
    o->x.assign(d, 0.f);
    o->m.assign(M, std::vector<float>(d, 0.f));
    o->words.assign(M, std::vector<uint32_t>(o->W, 0u));
    o->swords.assign(o->W, 0u);
    o->stepped.assign(M, 0);
    return o;
}

void sgo_destroy(void* h) { delete static_cast<Signum*>(h); }
int64_t sgo_num_words(void* h) { return static_cast<Signum*>(h)->W; }
int64_t sgo_step_count(void* h) { return static_cast<Signum*>(h)->t; }

// Worker i: momentum, then the packed signs of the momentum.  Returns 0, or -1 on misuse.
int32_t sgo_worker_step(void* h, int32_t i, const float* grad)
{
    Signum* o = static_cast<Signum*>(h);
    if (!o || !grad || i < 0 || i >= o->M || o->stepped[i]) return -1;
    float* m = o->m[i].data();
    uint32_t* words = o->words[i].data();
    for (int64_t w = 0; w < o->W; ++w) words[w] = 0u;
    for (int32_t b = 0; b < o->B; ++b) {
        for (int64_t j = o->off[b]; j < o->off[b + 1]; ++j) {
            m[j] = std::fmaf(o->mu, m[j], grad[j]);            // m_t = mu m_{t-1} + g_t
            const int64_t k = j - o->off[b];
            if (m[j] < 0.0f) words[o->woff[b] + (k >> 5)] |= (1u << (k & 31));   // sign(m_t)
        }
    }
    o->stepped[i] = 1;
    return 0;
}

// Server: coordinate-wise majority of the M sign vectors, then x <- x - eta * vote.
int32_t sgo_server_step(void* h)
{
    Signum* o = static_cast<Signum*>(h);
    if (!o) return -1;
    for (int32_t i = 0; i < o->M; ++i) if (!o->stepped[i]) return -1;
    for (int64_t w = 0; w < o->W; ++w) o->swords[w] = 0u;
    for (int32_t b = 0; b < o->B; ++b) {
        for (int64_t j = o->off[b]; j < o->off[b + 1]; ++j) {
            const int64_t k = j - o->off[b];
            const int64_t w = o->woff[b] + (k >> 5);
            int32_t sum = 0;                                   // sum_i sign(m_{t,i,j}) in {-M..M}
            for (int32_t i = 0; i < o->M; ++i)
                sum += ((o->words[i][w] >> (k & 31)) & 1u) ? -1 : +1;
            const bool neg = sum < 0;                          // tie (sum == 0) is sent as +1
            if (neg) o->swords[w] |= (1u << (k & 31));
            o->x[j] = neg ? (o->x[j] + o->eta) : (o->x[j] - o->eta);   // x - eta * vote
        }
    }
    for (int32_t i = 0; i < o->M; ++i) o->stepped[i] = 0;
    o->t += 1;
    return 0;
}

float*    sgo_params(void* h)              { return static_cast<Signum*>(h)->x.data(); }
float*    sgo_momentum(void* h, int32_t i) { return static_cast<Signum*>(h)->m[i].data(); }
uint32_t* sgo_words(void* h, int32_t i)    { Signum* o = static_cast<Signum*>(h);
                                             return i < 0 ? o->swords.data() : o->words[i].data(); }

// Top-k of v[0..n): writes the k kept indices (increasing) and their values, and the residual
// resid = v - C(v) (n floats; may be null).  Returns 0, or -1 on bad arguments.
int32_t tko_compress(const float* v, int64_t n, int64_t k, int64_t* idx_out, float* val_out,
                     float* resid)
{
    if (!v || n < 1 || k < 1 || k > n || !idx_out || !val_out) return -1;
    std::vector<int64_t> order(n);
    std::iota(order.begin(), order.end(), (int64_t)0);
    // largest magnitude first; equal magnitudes keep index order (stable)
    std::stable_sort(order.begin(), order.end(),
                     [v](int64_t a, int64_t b) { return std::fabs(v[a]) > std::fabs(v[b]); });
    std::vector<int64_t> kept(order.begin(), order.begin() + k);
    std::sort(kept.begin(), kept.end());
    if (resid) for (int64_t j = 0; j < n; ++j) resid[j] = v[j];
    for (int64_t r = 0; r < k; ++r) {
        idx_out[r] = kept[r];
        val_out[r] = v[kept[r]];
        if (resid) resid[kept[r]] = v[kept[r]] - v[kept[r]];   // e = v - C(v): +0 where kept
    }
    return 0;
}

}  // extern "C"
