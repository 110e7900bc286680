// CPU oracle for dist-EF-blockSGDM (Algorithm 4 of arXiv 1905.10936).
//
// TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, single-threaded statement of
// what one two-way compressed step computes.  It shares no code with the CUDA library and
// must never be linked, imported or executed by the product path; only the tests, the
// smoke check and the benchmark's CPU-baseline leg use it.
//
// It follows Algorithm 4 line by line, in the paper's notation:
//   worker i :  m_{t,i} = mu m_{t-1,i} + g_{t,i}                          (Alg. 4, worker line 1)
//               p_{t,i} = mu m_{t,i} + g_{t,i} + (eta_{t-1}/eta_t) e_{t,i} (Alg. 4, worker line 2)
//               Delta_{t,i} = C_B(p_{t,i})   pushed to the server          (Alg. 4, worker line 3)
//               e_{t+1,i} = p_{t,i} - Delta_{t,i}                          (Alg. 4, worker line 5)
//   server   :  ptilde_t = (1/M) sum_i Delta_{t,i} + (eta_{t-1}/eta_t) etilde_t
//               Deltatilde_t = C_B(ptilde_t) pushed to the workers
//               etilde_{t+1} = ptilde_t - Deltatilde_t
//   worker   :  x_{t+1} = x_t - eta_t Deltatilde_t                         (Alg. 4, worker line 4)
// with the blockwise compressor of Section 3.2:
//   C_B(v) = [ ||v_{G_b}||_1 / d_b * sign(v_{G_b}) ]_{b=1..B}.
//
// Stepsize sequence (Algorithms 2-4, "stepsize sequence {eta_t}"): efo_set_eta changes the
// stepsize of the coming iteration; both residuals are then rescaled by
// r = fl(eta_{t-1} / eta_t) as they are added: p = fma(r, e, mu m + g), ptilde = fma(r, etilde, a).
// Weight decay (Appendix A): kept out of the compressor; every worker keeps an extra momentum
//   mtilde_t = mu mtilde_{t-1} + lambda x_t,   x_{t+1} = x_t - eta_t (Deltatilde_t + mu mtilde_t + lambda x_t),
// done once here because all replicas of x are identical.
//
// Diagnostics (Section 3.2, Fig. 1), off by default and switched on by efo_set_diagnostics: a
// worker call then also records, per block, ||p_b||_1, ||p_b||_2^2, ||g_b||_1 and ||g_b||_2^2
// (binary64 sums; they are not part of Algorithm 4 and change none of its results), from which follow
//   phi(p) = min_b ||p_b||_1^2 / (d_b ||p_b||_2^2)            (Prop. 1),
//   delta of the non-block compressor = ||p||_1^2 / (d ||p||_2^2)   (Section 3.2),
//   coefficient of variation of |g| in block b = sqrt(d_b ||g_b||_2^2 / ||g_b||_1^2 - 1).
//
// Readings where the paper is silent (each is a convention of this repository):
//   * until efo_set_eta is called the stepsize is constant, so eta_{t-1}/eta_t = 1; at t = 0 the
//     paper's ratio (eta_{-1} = 0) multiplies e_0 = etilde_0 = 0, which the ratio 1 reproduces;
//   * the rescaled residual enters through one fused multiply-add, p = fma(r, e, u), with
//     r = fl(eta_{t-1}/eta_t) computed once in fp32 (for r = 1 this is fl(u + e), bit for bit);
//   * with weight decay the update is evaluated as
//       wd = fl(lambda x); mtilde = fma(mu, mtilde, wd); v = fma(mu, mtilde, wd);
//       x <- fl( fl(x -+ fl(eta s_b)) - fl(eta v) );
//   * state and element arithmetic are IEEE binary32 in the fixed order written below, block
//     L1 sums are accumulated sequentially in binary64 and rounded once to binary32 (the scale
//     is a float32 on the wire, Section 3.2);
//   * sign(+-0) = +1: Appendix A maps signs to {-1, +1} in one bit;
//   * the server average uses c_{i,b} = fl(s_{i,b} / M) and adds +-c_{i,b} in ascending i;
//   * all workers hold the same x, so the parameter update is done once, by the server call;
//   * blocks are contiguous index ranges given by B+1 offsets, every d_b >= 1;
//   * packed layout: block b owns ceil(d_b/32) words; element k of the block is bit (k mod 32)
//     (LSB = bit 0) of word floor(k/32); bit = 1 means negative (decodes to -1); unused high
//     bits of the last word are 0.
// PARITY UNPINNED BY THE PAPER for: this packed layout (bit polarity, bit order, word alignment),
// the order of the server average, the binary64 accumulation of the block sums, the single
// rounding of the rescaled residual (one fma rather than a product and a sum), and the operation
// order of the weight-decay update.  The paper is silent on all five; they are pinned, as
// conventions of this repository, only by worked examples and by hand-built cases in which the
// alternative gives a different binary32 result.
//
// "Hint" protocol (for step-locked comparison with another implementation): an element whose
// |p| is below 1e-6 times its block's scale may legitimately round to either sign when two
// implementations differ in the last bit of p.  When a hint (the other side's packed words)
// is given and the bits differ at such an element, the oracle adopts the hinted bit for the
// residual, the output word and the parameter update, and records the element index.  Outside
// that zone the hint is ignored.  Either sign satisfies e' = p - Delta.
//
// Build: g++ -O2 -ffp-contract=off -shared -fPIC  (no fast-math; fmaf is the only fused op).

#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

namespace {

struct Oracle {
    int64_t d = 0;
    int32_t B = 0;
    int32_t M = 0;
    float mu = 0.f;
    float eta = 0.f;                     // eta_t of the coming iteration
    float eta_prev = 0.f;                // eta_{t-1}: stepsize of the last completed iteration
    float lambda = 0.f;                  // weight decay (0 = off)
    std::vector<float> mt;               // weight-decay momentum mtilde (allocated when lambda > 0)
    int64_t W = 0;                       // total packed words
    int64_t t = 0;                       // completed iterations
    std::vector<int64_t> off;            // B+1 element offsets
    std::vector<int64_t> woff;           // B+1 word offsets
    std::vector<float> x;                // parameters
    std::vector<std::vector<float>> m;   // per-worker momentum
    std::vector<std::vector<float>> e;   // per-worker residual
    std::vector<float> et;               // server residual (etilde)
    std::vector<float> p;                // scratch: corrected vector of the current call
    std::vector<std::vector<uint32_t>> words;   // per-worker packed signs
    std::vector<std::vector<float>> scales;     // per-worker block scales
    std::vector<uint32_t> swords;        // server packed signs
    std::vector<float> sscales;          // server block scales
    std::vector<uint8_t> stepped;        // worker i has pushed in this iteration
    // Diagnostics of the last worker call of each worker (the quantities behind Fig. 1):
    // per block ||p_b||_1, ||p_b||_2^2, ||g_b||_1, ||g_b||_2^2, accumulated in binary64.
    std::vector<std::vector<double>> diag;   // [M][4*B]
    bool want_diag = false;                  // record them (efo_set_diagnostics)
};

// Compress p[lo,hi) of block b (Section 3.2), write the block's scale and packed signs,
// and replace the residual r[lo,hi) by p - Delta.  Optionally updates x (server call).
// Returns the number of adopted elements appended to `adopted`.
int64_t compress_block(const float* p, int64_t lo, int64_t hi,
                       float* scale_out, uint32_t* words_out /* block's first word */,
                       float* resid, float* x, float eta, float mu, float lambda, float* mt,
                       const uint32_t* hint /* block's first word or null */,
                       int64_t* adopted, int64_t adopted_cap, int64_t adopted_n)
{
    const int64_t db = hi - lo;
    double S = 0.0;
    for (int64_t j = lo; j < hi; ++j) S += (double)std::fabs(p[j]);
    const float s = (float)(S / (double)db);
    *scale_out = s;

    const int64_t nw = (db + 31) / 32;
    for (int64_t w = 0; w < nw; ++w) words_out[w] = 0u;

    const float zone = 1e-6f * s;
    const float step = eta * s;          // only used when x != nullptr
    for (int64_t j = lo; j < hi; ++j) {
        const int64_t k = j - lo;
        bool neg = p[j] < 0.0f;
        if (hint) {
            const bool hneg = (hint[k >> 5] >> (k & 31)) & 1u;
            if (hneg != neg && std::fabs(p[j]) < zone) {
                neg = hneg;
                if (adopted && adopted_n < adopted_cap) adopted[adopted_n] = j;
                ++adopted_n;
            }
        }
        if (neg) words_out[k >> 5] |= (1u << (k & 31));
        resid[j] = neg ? (p[j] + s) : (p[j] - s);
        if (x) {
            if (lambda > 0.0f) {                       // Appendix A: decay outside the compressor
                const float wd = lambda * x[j];
                mt[j] = std::fmaf(mu, mt[j], wd);      // mtilde_t = mu mtilde_{t-1} + lambda x_t
                const float v = std::fmaf(mu, mt[j], wd);
                const float xs = neg ? (x[j] + step) : (x[j] - step);
                const float ev = eta * v;
                x[j] = xs - ev;
            } else {
                x[j] = neg ? (x[j] + step) : (x[j] - step);
            }
        }
    }
    return adopted_n;
}

}  // namespace

extern "C" {

void* efo_init(int64_t d, int32_t B, const int64_t* offsets, int32_t M, float mu, float eta)
{
    if (d < 1 || B < 1 || M < 1 || !offsets) return nullptr;
    if (offsets[0] != 0 || offsets[B] != d) return nullptr;
    for (int32_t b = 0; b < B; ++b) if (offsets[b + 1] <= offsets[b]) return nullptr;
    if (!(mu >= 0.f && mu < 1.f) || !(eta > 0.f) || !std::isfinite(eta)) return nullptr;
    Oracle* o = new (std::nothrow) Oracle();
    if (!o) return nullptr;
    o->d = d; o->B = B; o->M = M; o->mu = mu; o->eta = eta; o->eta_prev = eta;
    o->off.assign(offsets, offsets + B + 1);
    o->woff.assign(B + 1, 0);
    for (int32_t b = 0; b < B; ++b)
        o->woff[b + 1] = o->woff[b] + (offsets[b + 1] - offsets[b] + 31) / 32;
    o->W = o->woff[B];
    o->x.assign(d, 0.f);
    o->et.assign(d, 0.f);
    o->p.assign(d, 0.f);
    o->m.assign(M, std::vector<float>(d, 0.f));
    o->e.assign(M, std::vector<float>(d, 0.f));
    o->words.assign(M, std::vector<uint32_t>(o->W, 0u));
    o->scales.assign(M, std::vector<float>(B, 0.f));
    o->swords.assign(o->W, 0u);
    o->sscales.assign(B, 0.f);
    o->stepped.assign(M, 0);
    o->diag.assign(M, std::vector<double>(4 * (size_t)B, 0.0));
    return o;
}

void efo_destroy(void* h) { delete static_cast<Oracle*>(h); }

int64_t efo_num_words(void* h) { return static_cast<Oracle*>(h)->W; }
int64_t efo_step_count(void* h) { return static_cast<Oracle*>(h)->t; }

// Worker i, one iteration.  grad: d floats.  hint: W words or null.  Returns the number of
// adopted elements (their flat indices go to adopted[0..cap)), or -1 on misuse.
int64_t efo_worker_step(void* h, int32_t i, const float* grad, const uint32_t* hint,
                        int64_t* adopted, int64_t adopted_cap)
{
    Oracle* o = static_cast<Oracle*>(h);
    if (!o || !grad || i < 0 || i >= o->M || o->stepped[i]) return -1;
    float* m = o->m[i].data();
    float* e = o->e[i].data();
    float* p = o->p.data();
    const float mu = o->mu;
    const float r = o->eta_prev / o->eta;                    // eta_{t-1} / eta_t
    int64_t n_adopted = 0;
    for (int32_t b = 0; b < o->B; ++b) {
        const int64_t lo = o->off[b], hi = o->off[b + 1];
        for (int64_t j = lo; j < hi; ++j) {
            m[j] = std::fmaf(mu, m[j], grad[j]);             // m_t = mu m_{t-1} + g_t
            const float u = std::fmaf(mu, m[j], grad[j]);    // mu m_t + g_t
            p[j] = std::fmaf(r, e[j], u);                    // + (eta_{t-1}/eta_t) e_t
        }
        if (o->want_diag) {   // plain sums over the block, independent of the compression below
            double p1 = 0.0, p2 = 0.0, g1 = 0.0, g2 = 0.0;
            for (int64_t j = lo; j < hi; ++j) {
                p1 += (double)std::fabs(p[j]);      p2 += (double)p[j] * (double)p[j];
                g1 += (double)std::fabs(grad[j]);   g2 += (double)grad[j] * (double)grad[j];
            }
            double* dg = o->diag[i].data() + 4 * (size_t)b;
            dg[0] = p1; dg[1] = p2; dg[2] = g1; dg[3] = g2;
        }
        n_adopted = compress_block(p, lo, hi, &o->scales[i][b],
                                   o->words[i].data() + o->woff[b], e, nullptr, 0.f, 0.f, 0.f,
                                   nullptr,
                                   hint ? hint + o->woff[b] : nullptr,
                                   adopted, adopted_cap, n_adopted);
    }
    o->stepped[i] = 1;
    return n_adopted;
}

// Server, one iteration (requires all M workers to have pushed).  Also applies the update
// x_{t+1} = x_t - eta Deltatilde_t.  Returns adopted count, or -1 on misuse.
int64_t efo_server_step(void* h, const uint32_t* hint, int64_t* adopted, int64_t adopted_cap)
{
    Oracle* o = static_cast<Oracle*>(h);
    if (!o) return -1;
    for (int32_t i = 0; i < o->M; ++i) if (!o->stepped[i]) return -1;
    float* p = o->p.data();
    float* et = o->et.data();
    const int32_t M = o->M;
    const float r = o->eta_prev / o->eta;                    // eta_{t-1} / eta_t
    std::vector<float> c(M);
    int64_t n_adopted = 0;
    for (int32_t b = 0; b < o->B; ++b) {
        const int64_t lo = o->off[b], hi = o->off[b + 1];
        for (int32_t i = 0; i < M; ++i) c[i] = o->scales[i][b] / (float)M;
        for (int64_t j = lo; j < hi; ++j) {
            const int64_t k = j - lo;
            float a = 0.f;
            for (int32_t i = 0; i < M; ++i) {
                const uint32_t w = o->words[i][o->woff[b] + (k >> 5)];
                const float v = ((w >> (k & 31)) & 1u) ? -c[i] : c[i];   // decoded Delta_{t,i} / M
                a = (i == 0) ? v : (a + v);
            }
            p[j] = std::fmaf(r, et[j], a);                    // ptilde_t = a + (eta_{t-1}/eta_t) etilde_t
        }
        n_adopted = compress_block(p, lo, hi, &o->sscales[b],
                                   o->swords.data() + o->woff[b], et, o->x.data(), o->eta,
                                   o->mu, o->lambda, o->lambda > 0.f ? o->mt.data() : nullptr,
                                   hint ? hint + o->woff[b] : nullptr,
                                   adopted, adopted_cap, n_adopted);
    }
    for (int32_t i = 0; i < M; ++i) o->stepped[i] = 0;
    o->eta_prev = o->eta;
    o->t += 1;
    return n_adopted;
}

// Stepsize of the coming iteration (between iterations only).  Returns 0, or -1 on misuse.
int32_t efo_set_eta(void* h, float eta)
{
    Oracle* o = static_cast<Oracle*>(h);
    if (!o || !(eta > 0.f) || !std::isfinite(eta)) return -1;
    for (int32_t i = 0; i < o->M; ++i) if (o->stepped[i]) return -1;
    o->eta = eta;
    return 0;
}

// Weight decay lambda >= 0 (Appendix A); allocates mtilde = 0 on first use.
int32_t efo_set_weight_decay(void* h, float lambda)
{
    Oracle* o = static_cast<Oracle*>(h);
    if (!o || !(lambda >= 0.f) || !std::isfinite(lambda)) return -1;
    for (int32_t i = 0; i < o->M; ++i) if (o->stepped[i]) return -1;
    o->lambda = lambda;
    if (lambda > 0.f && o->mt.empty()) o->mt.assign(o->d, 0.f);
    return 0;
}

// Diagnostic sums on/off (off after efo_init); they never change what Algorithm 4 computes.
void efo_set_diagnostics(void* h, int32_t on) { static_cast<Oracle*>(h)->want_diag = on != 0; }

double* efo_diagnostics(void* h, int32_t i) { return static_cast<Oracle*>(h)->diag[i].data(); }

float* efo_decay_momentum(void* h) { Oracle* o = static_cast<Oracle*>(h);
                                     return o->mt.empty() ? nullptr : o->mt.data(); }

// Raw views into the oracle's state (valid until efo_destroy).
float*    efo_params(void* h)               { return static_cast<Oracle*>(h)->x.data(); }
float*    efo_momentum(void* h, int32_t i)  { return static_cast<Oracle*>(h)->m[i].data(); }
float*    efo_residual(void* h, int32_t i)  { Oracle* o = static_cast<Oracle*>(h);
                                              return i < 0 ? o->et.data() : o->e[i].data(); }
uint32_t* efo_words(void* h, int32_t i)     { Oracle* o = static_cast<Oracle*>(h);
                                              return i < 0 ? o->swords.data() : o->words[i].data(); }
float*    efo_scales(void* h, int32_t i)    { Oracle* o = static_cast<Oracle*>(h);
                                              return i < 0 ? o->sscales.data() : o->scales[i].data(); }
// The corrected vector p (or ptilde) of the most recent call, before compression.
float*    efo_last_p(void* h)               { return static_cast<Oracle*>(h)->p.data(); }

}  // extern "C"
