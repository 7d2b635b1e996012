// Hysteresis-guided reconfiguration policy (host only): decides when to move between pre-specified
// topologies from per-step Rollout / Training times.
#include <cmath>
#include <new>

#include "dr_internal.h"

struct dr_ctl {
    dr_ctl_config cfg;
    int32_t index;
    uint32_t streak;
    int32_t streak_dir;
    uint64_t held;
    uint64_t since_resize;
    bool resized_before;
};

extern "C" {

int dr_ctl_create(const dr_ctl_config* cfg, dr_ctl** out)
{
    if (!out) {
        dr::set_error("NULL out");
        return DR_ERR_INVALID;
    }
    *out = nullptr;
    if (!cfg || cfg->struct_size != sizeof(dr_ctl_config) || cfg->n_topologies == 0 || cfg->initial >= cfg->n_topologies ||
        !(cfg->enter_threshold > 0) || !(cfg->exit_threshold >= 0) || cfg->exit_threshold > cfg->enter_threshold ||
        cfg->consecutive == 0) {
        dr::set_error("bad controller configuration");
        return DR_ERR_INVALID;
    }
    dr_ctl* c = new (std::nothrow) dr_ctl();
    if (!c) return DR_ERR_NOMEM;
    c->cfg = *cfg;
    c->index = (int32_t)cfg->initial;
    c->streak = 0;
    c->streak_dir = 0;
    c->held = 0;
    c->since_resize = 0;
    c->resized_before = false;
    *out = c;
    return DR_OK;
}

int dr_ctl_observe(dr_ctl* c, double t_rollout, double t_train, int32_t* move, uint32_t* topology)
{
    if (!c || !(t_rollout >= 0) || !(t_train >= 0)) {
        dr::set_error("NULL controller or negative / NaN step time");
        return DR_ERR_INVALID;
    }
    const dr_ctl_config& g = c->cfg;
    c->held++;
    if (c->resized_before) c->since_resize++;
    const double top = t_rollout > t_train ? t_rollout : t_train;
    const double imbalance = top > 0 ? (t_rollout - t_train) / top : 0.0;
    enum { QUIET, HOLD, SIGNAL } kind;
    int32_t dir = 0;
    if (imbalance > g.enter_threshold) {
        kind = SIGNAL;
        dir = 1;
    } else if (imbalance < -g.enter_threshold) {
        kind = SIGNAL;
        dir = -1;
    } else if (std::fabs(imbalance) < g.exit_threshold) {
        kind = QUIET;
    } else {
        kind = HOLD;  // inside the hysteresis band: the streak neither grows nor resets
    }
    if (kind == QUIET) {
        c->streak = 0;
        c->streak_dir = 0;
    } else if (kind == SIGNAL) {
        if (dir == c->streak_dir) {
            c->streak++;
        } else {
            c->streak = 1;
            c->streak_dir = dir;
        }
    }
    int32_t m = 0;
    const int64_t next = (int64_t)c->index + c->streak_dir;
    if (c->streak >= g.consecutive && c->held >= g.dwell_steps &&
        (!c->resized_before || c->since_resize >= g.cooldown_steps) && next >= 0 && next < (int64_t)g.n_topologies) {
        m = c->streak_dir;
        c->index = (int32_t)next;
        c->held = 0;
        c->since_resize = 0;
        c->resized_before = true;
        c->streak = 0;
        c->streak_dir = 0;
    }
    if (move) *move = m;
    if (topology) *topology = (uint32_t)c->index;
    return DR_OK;
}

int dr_ctl_break_even(double resize_cost_s, double step_before_s, double step_after_s, double* steps)
{
    if (!steps || !(resize_cost_s >= 0)) {
        dr::set_error("bad argument");
        return DR_ERR_INVALID;
    }
    const double saved = step_before_s - step_after_s;
    *steps = saved > 0 ? resize_cost_s / saved : INFINITY;
    return DR_OK;
}

int dr_ctl_destroy(dr_ctl* c)
{
    delete c;
    return DR_OK;
}

}  // extern "C"
