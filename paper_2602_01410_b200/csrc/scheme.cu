// Host side of scheme generation (paper Sec. 4.2, 4.3, 5): turns the norms collected on the GPU into
// the per-layer, per-option quality losses and picks one option per layer.  No GPU work here.
//
//   loss divergence of a layer under an option (Sec. 4.2):
//       sqrt( (|dL/dX| |dX_err| / sqrt(M K))^2 + (|dL/dW| |dW_err| / sqrt(N K))^2 ) / |L|
//   weight divergence of a layer (Sec. 4.3):
//       (1/layers) * alpha * sqrt(1 - beta2^t) / (1 - beta1^t) * |T| |g_err| / sqrt(N K) / |W|
//   selection (Sec. 5.2): minimise sum q[i][j] x[i][j]  s.t.  sum e[i][j] x[i][j] >= E_t, one option per
//   layer; with pipeline stages (Sec. 5.3) every stage must reach E_t / stages on its own.
//
// The selection is a multiple-choice knapsack.  Efficiencies are integers here (FLOPs run in FP4 under
// the option), so the solver is exact: it walks the layers keeping the Pareto frontier of
// (work reached, quality lost so far) - a state survives only if no other state reaches at least as
// much work at no more loss - and reads the cheapest state at or above the target at the end.  With a
// handful of distinct layer shapes the frontier stays small (it is bounded by the number of distinct
// work sums); a cap turns pathological inputs into an error instead of an endless run.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <limits>
#include <vector>

#include "common.cuh"

namespace snip {
namespace {

struct State {
    int64_t work;     // capped at the target: beyond it more work buys nothing
    double loss;
    int32_t parent;   // index into the previous layer's frontier
    int32_t option;
};

constexpr size_t kMaxFrontier = 4u << 20;

// One group of layers [first, last) against its own target.  Appends the chosen options to choice[first..last).
int solve_group(int n, const double *q, const int64_t *w, int first, int last, int64_t target, int *choice, double *loss_out, int64_t *work_out)
{
    std::vector<std::vector<State>> layers;
    layers.reserve(last - first + 1);
    layers.push_back({State{0, 0.0, -1, -1}});
    std::vector<State> cand;
    for (int i = first; i < last; ++i) {
        const std::vector<State> &prev = layers.back();
        cand.clear();
        cand.reserve(prev.size() * (size_t)n);
        for (int32_t s = 0; s < (int32_t)prev.size(); ++s)
            for (int j = 0; j < n; ++j) {
                const int64_t wij = w[(int64_t)i * n + j];
                const double qij = q[(int64_t)i * n + j];
                if (wij < 0 || !(qij >= 0.0) || !std::isfinite(qij)) return SNIP_ERR_ARG;
                int64_t nw = prev[s].work + wij;
                if (nw > target) nw = target;
                cand.push_back(State{nw, prev[s].loss + qij, s, j});
            }
        // frontier: by work descending, keep a state only if it loses strictly less than every state with more work
        std::sort(cand.begin(), cand.end(), [](const State &a, const State &b) {
            if (a.work != b.work) return a.work > b.work;
            if (a.loss != b.loss) return a.loss < b.loss;
            if (a.parent != b.parent) return a.parent < b.parent;
            return a.option < b.option;
        });
        std::vector<State> next;
        double best = std::numeric_limits<double>::infinity();
        for (const State &c : cand)
            if (c.loss < best) { next.push_back(c); best = c.loss; }
        if (next.size() > kMaxFrontier) return SNIP_ERR_UNSUPPORTED;
        layers.push_back(std::move(next));
    }
    // the frontier is sorted by work descending / loss descending: the cheapest state that reaches the target
    const std::vector<State> &fin = layers.back();
    int32_t pick = -1;
    for (int32_t s = 0; s < (int32_t)fin.size(); ++s)
        if (fin[s].work >= target) pick = s;   // later entries with the same (capped) work cannot exist; keep the last = cheapest
    if (pick < 0) return SNIP_ERR_UNSUPPORTED;   // the target cannot be reached even with every layer at its largest option
    *loss_out = fin[pick].loss;
    int64_t work = 0;
    for (int i = last - 1; i >= first; --i) {
        const State &st = layers[i - first + 1][pick];
        choice[i] = st.option;
        work += w[(int64_t)i * n + st.option];
        pick = st.parent;
    }
    *work_out = work;
    return SNIP_OK;
}

}  // namespace
}  // namespace snip

extern "C" double snip_loss_divergence(double grad_x_norm, double err_x_norm, int64_t M, int64_t K, double grad_w_norm, double err_w_norm, int64_t N,
                                       double loss)
{
    const double tx = grad_x_norm * err_x_norm / std::sqrt((double)M * (double)K);
    const double tw = grad_w_norm * err_w_norm / std::sqrt((double)N * (double)K);
    return std::sqrt(tx * tx + tw * tw) / std::fabs(loss);
}

extern "C" double snip_weight_divergence(double sens_norm, double grad_err_norm, int64_t N, int64_t K, double lr, double beta1, double beta2, int64_t step,
                                         double weight_norm, int64_t num_layers)
{
    const double bias = std::sqrt(1.0 - std::pow(beta2, (double)step)) / (1.0 - std::pow(beta1, (double)step));
    const double dw = lr * bias * sens_norm * grad_err_norm / std::sqrt((double)N * (double)K);
    return dw / weight_norm / (double)num_layers;
}

extern "C" int snip_select_scheme(int m, int n, const double *q, const int64_t *w, int64_t target, int num_groups, int *choice, double *q_total,
                                  int64_t *w_total)
{
    using namespace snip;
    if (m <= 0 || n <= 0 || !q || !w || !choice || target < 0) return SNIP_ERR_ARG;
    if (num_groups < 1 || (m % num_groups) != 0) return SNIP_ERR_SHAPE;
    const int per = m / num_groups;
    // every stage must reach target / stages on its own (rounded up: the constraint is >=)
    const int64_t group_target = (target + num_groups - 1) / num_groups;
    double loss = 0.0;
    int64_t work = 0;
    for (int k = 0; k < num_groups; ++k) {
        double gl = 0.0;
        int64_t gw = 0;
        const int rc = solve_group(n, q, w, k * per, (k + 1) * per, group_target, choice, &gl, &gw);
        if (rc != SNIP_OK) return rc;
        loss += gl;
        work += gw;
    }
    if (q_total) *q_total = loss;
    if (w_total) *w_total = work;
    return SNIP_OK;
}
