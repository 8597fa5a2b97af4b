// Iteration-cost bound of Theorem 3.2 and the quantities around it (Section
// 3): closed forms over a handful of scalars, evaluated on the host.  They take
// the perturbation norms that scar_recover_partial / scar_perturbation_norm
// report and turn them into the worst-case number of extra iterations.
#include <cmath>
#include <limits>

#include "scar.h"

namespace {

const double kNaN = std::numeric_limits<double>::quiet_NaN();

bool rate_ok(double c) { return c > 0.0 && c < 1.0; }

}  // namespace

extern "C" {

double scar_baseline_iterations(double dist0, double eps, double c) {
    if (!rate_ok(c) || !(dist0 > 0.0) || !(eps > 0.0)) return kNaN;
    return std::log(dist0 / eps) / std::log(1.0 / c);
}

double scar_discounted_perturbation(const double *norms, const uint64_t *iters, uint64_t n, double c) {
    if (!rate_ok(c) || (n && (!norms || !iters))) return kNaN;
    double sum = 0.0;
    for (uint64_t i = 0; i < n; ++i) {
        if (!(norms[i] >= 0.0)) return kNaN;
        // c^(-l) as exp(-l log c): one rounding instead of l of them
        sum += std::exp(-(double)iters[i] * std::log(c)) * norms[i];
    }
    return sum;
}

double scar_iteration_cost_bound(double delta_T, double dist0, double c) {
    if (!rate_ok(c) || !(dist0 > 0.0) || !(delta_T >= 0.0)) return kNaN;
    return std::log1p(delta_T / dist0) / std::log(1.0 / c);
}

double scar_irreducible_error(double delta_max, double c) {
    if (!rate_ok(c) || !(delta_max >= 0.0)) return kNaN;
    return c / (1.0 - c) * delta_max;
}

}  // extern "C"
