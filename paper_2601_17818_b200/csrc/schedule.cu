// Host-side arithmetic of the pruning schedule and of the cost model (Algorithm 1, Appendix E: Eq. 7-10).
#include <cmath>

#include "vitcop.h"

extern "C" {

int vitcop_stage_count(int m, double pi) { return (int)std::floor((double)m * pi); }

double vitcop_flops_layer(double N, double d) { return 4.0 * N * N * d + 16.0 * N * d * d; }

double vitcop_visual_tokens_at_layer(int l, double m, double pi1, double pi2, double pi3, int l_s, int l_d) {
    if (l < l_s) return pi1 * m;
    if (l < l_d) return pi2 * m;
    return pi3 * m;
}

double vitcop_flops_total(double m, double n_text, double d, double pi1, double pi2, double pi3, int l_s, int l_d,
                          int n_layers) {
    double total = 0.0;
    for (int l = 1; l <= n_layers; ++l)
        total += vitcop_flops_layer(vitcop_visual_tokens_at_layer(l, m, pi1, pi2, pi3, l_s, l_d) + n_text, d);
    return total;
}

double vitcop_cr_int(double pi1, double pi2, double pi3, int l_s, int l_d, int n_layers) {
    double kept = 0.0;
    for (int l = 1; l <= n_layers; ++l) kept += vitcop_visual_tokens_at_layer(l, 1.0, pi1, pi2, pi3, l_s, l_d);
    return 1.0 - kept / (double)n_layers;
}

}  // extern "C"
