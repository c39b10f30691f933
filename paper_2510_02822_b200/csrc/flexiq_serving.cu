// Run-time ratio controller and the request queue of the serving experiment (Sec. 8).
// Host code only: the controller is a table lookup per decision, the queue one pass over the
// arrival times with two cursors (next request to dispatch, start of the rate window).
#include "flexiq_internal.h"

#include <new>
#include <vector>

struct flexiq_controller {
    uint32_t magic;
    int n_levels, n_rates, level;
    double threshold, window;
    std::vector<double> rate_grid;  // [n_rates] ascending
    std::vector<double> latency;    // [n_levels][n_rates]
};

namespace {

constexpr uint32_t kControllerMagic = 0x46514354u;  // "FQCT"

flexiq_controller *as_controller(flexiq_controller_t h)
{
    return h && h->magic == kControllerMagic ? h : nullptr;
}

// profiled latency of one level at `rate`: linear between grid rates, end values outside
double profiled_latency(const flexiq_controller &c, int level, double rate)
{
    const double *g = c.rate_grid.data(), *y = c.latency.data() + (size_t)level * c.n_rates;
    const int n = c.n_rates;
    if (rate <= g[0]) return y[0];
    if (rate >= g[n - 1]) return y[n - 1];
    int hi = 1;
    while (rate > g[hi]) ++hi;
    const double t = (rate - g[hi - 1]) / (g[hi] - g[hi - 1]);
    return y[hi - 1] + t * (y[hi] - y[hi - 1]);
}

int decide(flexiq_controller &c, double rate)
{
    if (profiled_latency(c, c.level, rate) > c.threshold) {
        if (c.level + 1 < c.n_levels) ++c.level;
    } else if (c.level > 0 && profiled_latency(c, c.level - 1, rate) <= c.threshold) {
        --c.level;
    }
    return c.level;
}

}  // namespace

using flexiq::set_error;

extern "C" int flexiq_controller_create(flexiq_controller_t *out, int n_levels, int n_rates, const double *rate_grid_host,
                                        const double *latency_host, double threshold, double window_s, int initial_level)
{
    if (!out) return set_error(FLEXIQ_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    if (n_levels < 1 || n_rates < 1) return set_error(FLEXIQ_ERR_INVALID_ARG, "n_levels %d and n_rates %d must be positive", n_levels, n_rates);
    if (!rate_grid_host || !latency_host) return set_error(FLEXIQ_ERR_INVALID_ARG, "rate_grid_host or latency_host is NULL");
    if (!(window_s > 0.0)) return set_error(FLEXIQ_ERR_INVALID_ARG, "window_s %g must be positive", window_s);
    if (!(threshold == threshold)) return set_error(FLEXIQ_ERR_INVALID_ARG, "threshold is not a number");
    if (initial_level < 0 || initial_level >= n_levels)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "initial_level %d outside [0, %d)", initial_level, n_levels);
    for (int i = 1; i < n_rates; ++i)
        if (!(rate_grid_host[i] > rate_grid_host[i - 1]))
            return set_error(FLEXIQ_ERR_INVALID_ARG, "rate_grid_host is not strictly ascending at index %d", i);
    flexiq_controller *c = new (std::nothrow) flexiq_controller();
    if (!c) return set_error(FLEXIQ_ERR_CUDA, "out of host memory");
    c->magic = kControllerMagic;
    c->n_levels = n_levels; c->n_rates = n_rates; c->level = initial_level;
    c->threshold = threshold; c->window = window_s;
    c->rate_grid.assign(rate_grid_host, rate_grid_host + n_rates);
    c->latency.assign(latency_host, latency_host + (size_t)n_levels * n_rates);
    *out = c;
    return FLEXIQ_OK;
}

extern "C" int flexiq_controller_destroy(flexiq_controller_t ctrl)
{
    flexiq_controller *c = as_controller(ctrl);
    if (!c) return set_error(FLEXIQ_ERR_INVALID_ARG, "not a live flexiq controller handle");
    c->magic = 0;
    delete c;
    return FLEXIQ_OK;
}

extern "C" int flexiq_controller_level(flexiq_controller_t ctrl, int *level)
{
    flexiq_controller *c = as_controller(ctrl);
    if (!c) return set_error(FLEXIQ_ERR_INVALID_ARG, "not a live flexiq controller handle");
    if (!level) return set_error(FLEXIQ_ERR_INVALID_ARG, "level is NULL");
    *level = c->level;
    return FLEXIQ_OK;
}

extern "C" int flexiq_controller_update(flexiq_controller_t ctrl, double rate, int *level)
{
    flexiq_controller *c = as_controller(ctrl);
    if (!c) return set_error(FLEXIQ_ERR_INVALID_ARG, "not a live flexiq controller handle");
    if (!(rate >= 0.0)) return set_error(FLEXIQ_ERR_INVALID_ARG, "rate %g is negative or not a number", rate);
    const int l = decide(*c, rate);
    if (level) *level = l;
    return FLEXIQ_OK;
}

extern "C" int flexiq_serving_simulate(flexiq_controller_t ctrl, int fixed_level, int64_t n, const double *arrival_host,
                                       int n_levels, int max_batch, const double *service_host, double *response_host,
                                       int32_t *level_host)
{
    flexiq_controller *c = nullptr;
    if (ctrl) {
        c = as_controller(ctrl);
        if (!c) return set_error(FLEXIQ_ERR_INVALID_ARG, "not a live flexiq controller handle");
        if (c->n_levels != n_levels)
            return set_error(FLEXIQ_ERR_INVALID_ARG, "the controller has %d levels, the service table %d", c->n_levels, n_levels);
    }
    if (n < 0) return set_error(FLEXIQ_ERR_INVALID_ARG, "n = %lld is negative", (long long)n);
    if (n_levels < 1 || max_batch < 1) return set_error(FLEXIQ_ERR_INVALID_ARG, "n_levels %d and max_batch %d must be positive", n_levels, max_batch);
    if (!c && (fixed_level < 0 || fixed_level >= n_levels))
        return set_error(FLEXIQ_ERR_INVALID_ARG, "fixed_level %d outside [0, %d)", fixed_level, n_levels);
    if (n == 0) return FLEXIQ_OK;
    if (!arrival_host || !service_host || !response_host || !level_host)
        return set_error(FLEXIQ_ERR_INVALID_ARG, "arrival_host, service_host, response_host or level_host is NULL");
    for (int64_t i = 1; i < n; ++i)
        if (!(arrival_host[i] >= arrival_host[i - 1]))
            return set_error(FLEXIQ_ERR_INVALID_ARG, "arrival_host is not ascending at index %lld", (long long)i);

    int level = c ? c->level : fixed_level;
    double free_at = 0.0, last_decision = 0.0;
    int64_t i = 0;        // next request to dispatch
    int64_t w_lo = 0;     // first arrival inside the rate window (start - window, start]
    int64_t w_hi = 0;     // first arrival after `start`
    while (i < n) {
        const double start = free_at > arrival_host[i] ? free_at : arrival_host[i];
        int64_t b = 1;
        while (i + b < n && b < max_batch && arrival_host[i + b] <= start) ++b;
        if (c && start - last_decision >= c->window) {
            // the starts ascend, so both cursors only move forward
            while (w_hi < n && arrival_host[w_hi] <= start) ++w_hi;
            while (w_lo < w_hi && !(arrival_host[w_lo] > start - c->window)) ++w_lo;
            level = decide(*c, (double)(w_hi - w_lo) / c->window);
            last_decision = start;
        }
        const double done = start + service_host[(size_t)level * max_batch + (b - 1)];
        for (int64_t r = i; r < i + b; ++r) {
            response_host[r] = done - arrival_host[r];
            level_host[r] = level;
        }
        free_at = done;
        i += b;
    }
    return FLEXIQ_OK;
}
