// Runs the CPU oracles (Algorithm 4, signum with majority vote, top-k) on ragged layouts under
// AddressSanitizer and UndefinedBehaviorSanitizer: the test compiles this file together with the
// oracle sources with -fsanitize=address,undefined and fails on any report.  Prints "ok".
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <vector>

extern "C" {
void* efo_init(int64_t d, int32_t B, const int64_t* offsets, int32_t M, float mu, float eta);
void efo_destroy(void* h);
int64_t efo_num_words(void* h);
int64_t efo_worker_step(void* h, int32_t i, const float* grad, const uint32_t* hint, int64_t* adopted,
                        int64_t cap);
int64_t efo_server_step(void* h, const uint32_t* hint, int64_t* adopted, int64_t cap);
int32_t efo_set_eta(void* h, float eta);
int32_t efo_set_weight_decay(void* h, float lambda);
void efo_set_diagnostics(void* h, int32_t on);
uint32_t* efo_words(void* h, int32_t i);
float* efo_params(void* h);
void* sgo_init(int64_t d, int32_t B, const int64_t* offsets, int32_t M, float mu, float eta);
void sgo_destroy(void* h);
int32_t sgo_worker_step(void* h, int32_t i, const float* grad);
int32_t sgo_server_step(void* h);
int32_t tko_compress(const float* v, int64_t n, int64_t k, int64_t* idx, float* val, float* resid);
}

static uint32_t rng_state = 12345u;
static float rnd() {                      // small deterministic generator, values in (-1, 1)
    rng_state = rng_state * 1664525u + 1013904223u;
    return (float)((int32_t)(rng_state >> 8) - (1 << 23)) / (float)(1 << 23);
}

int main() {
    const std::vector<std::vector<int64_t>> layouts = {
        {1}, {1, 1, 1}, {3, 5, 31, 33, 63, 65}, {32, 64, 96}, {1000, 7, 4097}, {40}};
    for (const auto& sizes : layouts) {
        std::vector<int64_t> off(1, 0);
        for (int64_t s : sizes) off.push_back(off.back() + s);
        const int64_t d = off.back();
        const int32_t B = (int32_t)sizes.size();
        for (int32_t M : {1, 2, 5}) {
            void* h = efo_init(d, B, off.data(), M, 0.9f, 0.1f);
            void* s = sgo_init(d, B, off.data(), M, 0.5f, 0.01f);
            if (!h || !s) return 1;
            efo_set_diagnostics(h, M == 2);
            if (M == 5) efo_set_weight_decay(h, 0.01f);
            const int64_t W = efo_num_words(h);
            std::vector<float> g(d);
            std::vector<uint32_t> hint(W);
            std::vector<int64_t> adopted(8);
            for (int t = 0; t < 4; ++t) {
                if (t == 2) efo_set_eta(h, 0.05f);
                for (int32_t i = 0; i < M; ++i) {
                    for (auto& v : g) v = rnd();
                    for (auto& w : hint) { rng_state = rng_state * 1664525u + 1013904223u; w = rng_state; }
                    efo_worker_step(h, i, g.data(), (t & 1) ? hint.data() : nullptr, adopted.data(), 8);
                    sgo_worker_step(s, i, g.data());
                }
                efo_server_step(h, (t & 1) ? hint.data() : nullptr, adopted.data(), 8);
                sgo_server_step(s);
            }
            volatile float sink = efo_params(h)[d - 1] + (float)efo_words(h, -1)[W - 1];
            (void)sink;
            efo_destroy(h);
            sgo_destroy(s);
        }
        std::vector<float> v(d), val(d), resid(d);
        std::vector<int64_t> idx(d);
        for (auto& x : v) x = rnd();
        for (int64_t k : {(int64_t)1, (d + 1) / 2, d})
            if (tko_compress(v.data(), d, k, idx.data(), val.data(), resid.data()) != 0) return 2;
    }
    // misuse must be refused, not crash
    int64_t off2[2] = {0, 4};
    if (efo_init(4, 1, off2, 0, 0.9f, 0.1f) != nullptr) return 3;
    if (tko_compress(nullptr, 4, 1, nullptr, nullptr, nullptr) != -1) return 4;
    std::printf("ok\n");
    return 0;
}
