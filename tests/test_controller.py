"""Hysteresis controller (Sec. 3.4): the Python oracle against what the paper fixes (break-even of about
11 steps from its own numbers, cooldown above 10, no thrashing under transient noise, only sustained
one-directional imbalance triggers, never leaves the candidate set), and the C implementation against
the oracle on random traces."""
import math
import os
import sys

import numpy as np
import pytest

import paper_2607_22614_b200 as dr
from oracle.controller import Config, Controller, break_even_steps


def _run_oracle(cfg, trace):
    c = Controller(cfg)
    return [(c.observe(r, t), c.index) for r, t in trace]


def _run_lib(cfg, trace):
    rc, h = dr.dr_ctl_create(cfg.n_topologies, cfg.initial, cfg.enter, cfg.exit, cfg.consecutive, cfg.dwell, cfg.cooldown)
    assert rc == 0
    out = []
    for r, t in trace:
        rc, move, topo = dr.dr_ctl_observe(h, r, t)
        assert rc == 0
        out.append((move, topo))
    dr.dr_ctl_destroy(h)
    return out


def test_paper_numbers(golden):
    g = {r[0]: float(r[1]) for r in golden("resize_numbers.txt")}
    be = break_even_steps(g["critical_path_blocking_s"], g["step_before_s"], g["step_after_s"])
    assert g["break_even_steps_about"] <= be < g["break_even_steps_about"] + 1          # 187 / 15.91 = 11.75
    assert Config(3).cooldown > g["cooldown_steps_more_than"] and Config(3).cooldown >= math.floor(be)
    assert abs((g["naive_blocking_s"] - g["critical_path_blocking_s"]) / g["naive_blocking_s"] * 100
               - g["overhead_hidden_percent"]) < 0.5
    assert abs((g["step_before_s"] / g["step_after_s"] - 1) * 100 - g["throughput_gain_percent"]) < 0.1
    rc, steps = dr.dr_ctl_break_even(g["critical_path_blocking_s"], g["step_before_s"], g["step_after_s"])
    assert rc == 0 and steps == be
    assert dr.dr_ctl_break_even(100.0, 10.0, 12.0)[1] == math.inf == break_even_steps(100.0, 10.0, 12.0)


def test_sustained_imbalance_triggers_once_then_cooldown_holds():
    cfg = Config(3, initial=0, consecutive=3, dwell=5, cooldown=11)
    trace = [(39.84, 20.0)] * 40                     # Rollout much slower than Training, for 40 steps
    moves = [m for m, _ in _run_oracle(cfg, trace)]
    first = moves.index(1)
    assert first == 4                                 # dwell (5 steps) is the binding constraint: decided on step 5
    second = moves.index(1, first + 1)
    assert second - first == 11                       # the cooldown separates consecutive resizes
    assert sum(moves) == 2 and moves.count(1) == 2    # and the set of 3 topologies is never left
    assert _run_oracle(cfg, trace)[-1][1] == 2


def test_transient_noise_and_band_oscillation_never_trigger():
    cfg = Config(3, initial=1, consecutive=3, dwell=0, cooldown=11)
    spikes = ([(30.0, 20.0)] * 2 + [(20.0, 20.0)]) * 20           # two noisy steps, then a quiet one
    assert all(m == 0 for m, _ in _run_oracle(cfg, spikes))
    flip = [(30.0, 20.0), (20.0, 30.0)] * 30                      # alternating direction
    assert all(m == 0 for m, _ in _run_oracle(cfg, flip))
    band = [(23.0, 20.0)] * 50                                    # imbalance 0.13: inside the hysteresis band
    assert all(m == 0 for m, _ in _run_oracle(cfg, band))
    # a band step does not break a streak: signal, signal, band, signal -> resize on the third signal
    cfg2 = Config(3, initial=1, consecutive=3, dwell=0, cooldown=0)
    moves = [m for m, _ in _run_oracle(cfg2, [(30.0, 20.0), (30.0, 20.0), (23.0, 20.0), (30.0, 20.0)])]
    assert moves == [0, 0, 0, 1]


def test_direction_and_bounds():
    cfg = Config(2, initial=1, consecutive=2, dwell=0, cooldown=0)
    out = _run_oracle(cfg, [(10.0, 30.0)] * 6)                     # Training is the bottleneck: move towards Training
    assert [m for m, _ in out] == [0, -1, 0, 0, 0, 0] and out[-1][1] == 0   # then pinned at the edge
    out = _run_oracle(Config(2, initial=1, consecutive=1, dwell=0, cooldown=0), [(30.0, 10.0)] * 3)
    assert all(m == 0 for m, _ in out)                             # already most-Rollout


@pytest.mark.parametrize("seed", range(8))
def test_library_equals_oracle_on_random_traces(seed):
    rng = np.random.default_rng(seed)
    cfg = Config(int(rng.integers(1, 6)), 0, enter=float(rng.uniform(0.05, 0.4)), exit=0.0, consecutive=int(rng.integers(1, 5)),
                 dwell=int(rng.integers(0, 8)), cooldown=int(rng.integers(0, 15)))
    cfg.exit = float(rng.uniform(0, cfg.enter))
    cfg.initial = int(rng.integers(0, cfg.n_topologies))
    # slowly drifting load with noise, so that streaks, band steps and reversals all occur
    t = np.arange(600)
    roll = 20 + 10 * np.sin(t / 37.0 + seed) + rng.normal(0, 2.5, t.size)
    train = 20 + 10 * np.cos(t / 53.0) + rng.normal(0, 2.5, t.size)
    trace = [(float(max(a, 0.0)), float(max(b, 0.0))) for a, b in zip(roll, train)]
    want = _run_oracle(cfg, trace)
    assert _run_lib(cfg, trace) == want
    assert any(m != 0 for m, _ in want) or cfg.n_topologies == 1


def test_controller_argument_errors():
    E = dr.binding
    assert dr.dr_ctl_create(0)[0] == E.DR_ERR_INVALID
    assert dr.dr_ctl_create(3, initial=3)[0] == E.DR_ERR_INVALID
    assert dr.dr_ctl_create(3, enter=0.1, exit=0.2)[0] == E.DR_ERR_INVALID
    rc, h = dr.dr_ctl_create(3)
    assert rc == 0
    assert dr.dr_ctl_observe(h, float("nan"), 1.0)[0] == E.DR_ERR_INVALID
    assert dr.dr_ctl_observe(h, -1.0, 1.0)[0] == E.DR_ERR_INVALID
    assert dr.dr_ctl_observe(h, 0.0, 0.0)[:2] == (0, 0)
    dr.dr_ctl_destroy(h)
