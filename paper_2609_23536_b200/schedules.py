"""Schedule orders for one simulated pipeline stage: lists of ("F" | "dI" | "dW", microbatch).

A schedule is input to the layer, not part of it: the paper's contract holds for any
order in which F(m) precedes dI(m) precedes dW(m) (Sec. 4.2: the split-backward
schedules share one implementation and differ only in event order).  This module holds
no arithmetic of the method.
"""
from __future__ import annotations

from typing import List, Tuple

Action = Tuple[str, int]


def sched(M: int, warmup: int, defer: int) -> List[Action]:
    """`warmup` forwards first; then per round: F(next) if any, dI(next), and dW(next)
    whenever more than `defer` input-grads are waiting for their weight-grad; the
    remaining dW are flushed in order.  dW order is monotone in the microbatch index.

    sched(4, 1, 0) = F0 F1 dI0 dW0 F2 dI1 dW1 F3 dI2 dW2 dI3 dW3   (1F1B, full backward)
    sched(M, 3, 3)                                                 (zero-bubble H1 style stage)
    """
    out: List[Action] = []
    f = di = dw = 0
    for _ in range(min(warmup, M)):
        out.append(("F", f))
        f += 1
    while di < M:
        if f < M:
            out.append(("F", f))
            f += 1
        out.append(("dI", di))
        di += 1
        if di - dw > defer:
            out.append(("dW", dw))
            dw += 1
    while dw < M:
        out.append(("dW", dw))
        dw += 1
    return out


def full_backward(schedule: List[Action]) -> List[Action]:
    """Same F and dI order, with every dW moved to directly after its dI."""
    out: List[Action] = []
    for a, m in schedule:
        if a == "dW":
            continue
        out.append((a, m))
        if a == "dI":
            out.append(("dW", m))
    return out


def peak_live(schedule: List[Action]) -> int:
    """Largest number of tapes alive at once (F allocates, dW releases)."""
    live = peak = 0
    for a, _ in schedule:
        if a == "F":
            live += 1
            peak = max(peak, live)
        elif a == "dW":
            live -= 1
    return peak
