"""TEST INFRASTRUCTURE -- not part of the product path.

Plain Python statement of the hysteresis-guided reconfiguration policy of Sec. 3.4: resizing is a
decision among a fixed, ordered list of candidate topologies, filtered by hysteresis thresholds, a dwell
time, a cooldown interval and a consecutive-signal requirement, so that only sustained, one-directional
imbalance triggers a switch (Sec. 3.4); the cooldown is longer than 10 steps, above the break-even of
about 11 sustained steps (Sec. 5, Exp#3).  The paper gives the ingredients, not the formulas; the reading
below is the one this repository adopts:

  imbalance  = (t_rollout - t_train) / max(t_rollout, t_train); positive: Rollout is the bottleneck
  signal     = +1 if imbalance >  enter, -1 if imbalance < -enter, "quiet" if |imbalance| < exit,
               otherwise "hold" (inside the hysteresis band: the streak neither grows nor resets)
  streak     = number of consecutive signals of one direction (a quiet step or the other direction resets it)
  a resize by one position in the streak's direction happens when streak >= consecutive, the topology has
  been held for >= dwell steps, the last resize is >= cooldown steps ago, and the neighbour exists.

Topologies are indexed from most-Training to most-Rollout (e.g. 6:2, 5:3, 4:4); +1 moves a GPU to Rollout.
"""
from __future__ import annotations

from dataclasses import dataclass


@dataclass
class Config:
    n_topologies: int
    initial: int = 0
    enter: float = 0.2
    exit: float = 0.1
    consecutive: int = 3
    dwell: int = 5
    cooldown: int = 11


class Controller:
    def __init__(self, cfg: Config):
        self.cfg = cfg
        self.index = cfg.initial
        self.streak = 0
        self.streak_dir = 0
        self.held = 0            # steps spent in the current topology
        self.since_resize = None  # steps since the last resize, None before the first

    def observe(self, t_rollout: float, t_train: float) -> int:
        """Feed one step's times; returns -1, 0 or +1 (the move decided at this step)."""
        c = self.cfg
        self.held += 1
        if self.since_resize is not None:
            self.since_resize += 1
        top = max(t_rollout, t_train)
        imbalance = (t_rollout - t_train) / top if top > 0 else 0.0
        if imbalance > c.enter:
            direction = 1
        elif imbalance < -c.enter:
            direction = -1
        elif abs(imbalance) < c.exit:
            direction = 0
        else:
            direction = None  # hold
        if direction == 0:
            self.streak, self.streak_dir = 0, 0
        elif direction is not None:
            if direction == self.streak_dir:
                self.streak += 1
            else:
                self.streak, self.streak_dir = 1, direction
        move = 0
        if (self.streak >= c.consecutive and self.held >= c.dwell
                and (self.since_resize is None or self.since_resize >= c.cooldown)
                and 0 <= self.index + self.streak_dir < c.n_topologies):
            move = self.streak_dir
            self.index += move
            self.held = 0
            self.since_resize = 0
            self.streak, self.streak_dir = 0, 0
        return move


def break_even_steps(resize_cost_s: float, step_before_s: float, step_after_s: float) -> float:
    """Sustained steps after which the time saved per step has paid for one resize (Exp#3)."""
    saved = step_before_s - step_after_s
    return float("inf") if saved <= 0 else resize_cost_s / saved
