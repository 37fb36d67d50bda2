// Drives every entry point of the CPU oracle on small inputs. Built together with
// oracle/ga_oracle.cpp under -fsanitize=address,undefined by tests/test_sanitizers.py: any
// out-of-bounds access, use after free, leak or undefined operation in the oracle ends the
// program with a report and a non-zero status.
#include <cstdint>
#include <cstdio>
#include <vector>

extern "C" {
void* gao_create(int64_t d, int n_workers, double lr, double momentum, double beta, int variant, int precision);
void gao_destroy(void* p);
void gao_set_c_order(void* p, int c_order);
void gao_set_lr(void* p, double lr);
void gao_set_nesterov(void* p, int on);
void gao_set_weight_decay(void* p, double wd);
void gao_set_params(void* p, const float* theta0);
void gao_pull(void* p, int worker);
int64_t gao_push(void* p, int worker, const float* grad);
void gao_gap(void* p, int worker, double* out);
int64_t gao_k_done(void* p);
int64_t gao_iter(void* p, int worker);
void gao_set_state(void* p, const double* th, const double* v, const double* m, const double* saved,
                   const int64_t* iter, int64_t k_done, int64_t k_c, const double* v_workers);
int gao_set_layers(void* p, const int64_t* offsets, int n);
void gao_layer_state(void* p, double* gaps, double* m_layer);
void gao_set_adam(void* p, double beta2, double adam_eps);
void gao_set_dana_sum(void* p, int mode);
int64_t gao_k_c(void* p);
void gao_stats(void* p, double* sum_gap, double* max_gap);
int gao_get(void* p, int which, double* out);
void gao_sent_f32(void* p, int worker, float* out);
}

static uint64_t next(uint64_t& s) { s = s * 6364136223846793005ULL + 1442695040888963407ULL; return s >> 33; }

int main() {
    const int64_t d = 37;
    const int n = 3;
    uint64_t seed = 7;
    std::vector<float> g(d), th0(d), sent(d);
    std::vector<double> out(d), gaps(4), ml(4);
    for (auto& x : th0) x = (float)((double)(next(seed) % 2001) / 1000.0 - 1.0);
    long checksum = 0;
    for (int precision : {32, 64}) {
        for (int variant = 0; variant <= 10; ++variant) {
            for (int c_order = 0; c_order < 2; ++c_order) {
                if (c_order == 1 && variant != 2 && variant != 6 && variant != 9) continue;
                void* o = gao_create(d, n, 0.1, 0.9, 0.999, variant, precision);
                if (!o) return 2;
                gao_set_c_order(o, c_order);
                gao_set_dana_sum(o, variant == 5 ? 0 : 1);
                gao_set_adam(o, 0.99, 1e-7);
                if (variant < 4 || variant == 10) gao_set_nesterov(o, 1);
                gao_set_weight_decay(o, 1e-4);
                if (variant == 10) {
                    const int64_t off[4] = {0, 5, 6, d};
                    if (gao_set_layers(o, off, 3) != 0) return 3;
                    const int64_t bad[3] = {0, 9, 8};
                    if (gao_set_layers(o, bad, 2) == 0) return 4;
                }
                gao_set_params(o, th0.data());
                for (int k = 0; k < 12; ++k) {
                    const int i = (int)(next(seed) % n);
                    for (auto& x : g) x = (float)((double)(next(seed) % 2001) / 1000.0 - 1.0);
                    checksum += (long)gao_push(o, i, g.data());
                    if (k % 4 != 3) gao_pull(o, i);
                    if (k == 5) gao_set_lr(o, 0.01);
                }
                for (int which : {0, 1, 2, 3, 4, 4 + n - 1, 100000, 200000, 99}) gao_get(o, which, out.data());
                gao_gap(o, 1, out.data());
                gao_sent_f32(o, 2, sent.data());
                double s, m;
                gao_stats(o, &s, &m);
                if (variant == 10) gao_layer_state(o, gaps.data(), ml.data());
                checksum += (long)gao_k_done(o) + (long)gao_k_c(o) + (long)gao_iter(o, 0);
                gao_destroy(o);
            }
        }
    }
    gao_destroy(nullptr);
    if (gao_create(0, 1, 0.1, 0.9, 0.999, 2, 32) || gao_create(4, 1, 0.1, 0.9, 0.999, 11, 32) ||
        gao_create(4, 1, 0.1, 0.9, 0.999, 2, 16)) return 5;
    std::printf("sanitize driver ok %ld\n", checksum);
    return 0;
}
