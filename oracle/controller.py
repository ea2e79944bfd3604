"""Oracle for the adaptive runtime controller (Eq. 6-9, Algorithm 2).

TEST INFRASTRUCTURE: only tests, the smoke check and the CPU-baseline leg of the
benchmark may import this module.  It shares no code with the library.

Plain Python floats (fp64).  The controller keeps four numbers

    g_bar   EMA of the gradient norm            (Eq. 6)
    g_last  the last gradient norm observed
    c_bar   EMA of the worker's batch time      (Eq. 8)
    c_prev  the last batch time observed

and takes two decisions per batch r, in the order of Algorithm 2:

    S_r  (only when r is a candidate refresh boundary, Eq. 7)
         0 if r > 0 and g_bar > 0 and g_last < tau_g * g_bar, else 1
    H_r  (every batch, Eq. 9)
         1 if r > 0 and c_bar > 0 and c_prev > tau_c * c_bar, else 0

then, after the batch has run, folds its gradient norm g_r and its measured time
c_r into the two EMAs.  An EMA whose previous value is exactly 0 restarts from
the new sample (first case of Eq. 6 and Eq. 8).

Readings where the paper is silent:
  * candidate boundaries are the batches r with r % K == 0 (K = the
    synchronisation interval of the experiments section); r = 0 is one, and
    Eq. 7 gives S_0 = 1;
  * alpha and beta have no printed value; callers pass them.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple


def ema(prev: float, x: float, factor: float) -> float:
    """Eq. 6 / Eq. 8: restart from x when the previous average is 0."""
    if prev == 0.0:
        return x
    return factor * x + (1.0 - factor) * prev


def sync_decision(r: int, g_last: float, g_bar: float, tau_g: float) -> int:
    """Eq. 7."""
    if r > 0 and g_bar > 0.0 and g_last < tau_g * g_bar:
        return 0
    return 1


def load_detect(r: int, c_prev: float, c_bar: float, tau_c: float) -> int:
    """Eq. 9."""
    if r > 0 and c_bar > 0.0 and c_prev > tau_c * c_bar:
        return 1
    return 0


@dataclass
class ControllerOracle:
    alpha: float
    beta: float
    tau_g: float
    tau_c: float
    K: int
    g_bar: float = 0.0
    g_last: float = 0.0
    c_bar: float = 0.0
    c_prev: float = 0.0

    def begin_batch(self, r: int) -> Tuple[int, Optional[int], int]:
        """Algorithm 2, the decisions taken before batch r runs: (is_boundary, S_r or None, H_r)."""
        boundary = 1 if r % self.K == 0 else 0
        s = sync_decision(r, self.g_last, self.g_bar, self.tau_g) if boundary else None
        h = load_detect(r, self.c_prev, self.c_bar, self.tau_c)
        return boundary, s, h

    def end_batch(self, g_r: float, c_r: float) -> None:
        """Algorithm 2, the bookkeeping after backpropagation and after the batch time is measured."""
        self.g_bar = ema(self.g_bar, g_r, self.alpha)
        self.g_last = g_r
        self.c_bar = ema(self.c_bar, c_r, self.beta)
        self.c_prev = c_r


def run(alpha: float, beta: float, tau_g: float, tau_c: float, K: int, g: Sequence[float],
        c: Sequence[float]) -> List[Tuple[int, Optional[int], int, float, float]]:
    """Decisions and EMAs for whole sequences: per batch (boundary, S, H, g_bar after, c_bar after)."""
    o = ControllerOracle(alpha, beta, tau_g, tau_c, K)
    out = []
    for r, (gr, cr) in enumerate(zip(g, c)):
        b, s, h = o.begin_batch(r)
        o.end_batch(gr, cr)
        out.append((b, s, h, o.g_bar, o.c_bar))
    return out
