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


# ------------------------------------------------------------------------------------------------ multi-chunk orders
# With several model chunks per device (Sec. 4.2: Interleaved-1F1B and ZB-V place two local chunks on a device,
# each with its own tape pool) an action also names its chunk: ("F" | "dI" | "dW", microbatch, chunk).
ChunkAction = Tuple[str, int, int]


def interleaved_1f1b(M: int, stages: int, stage: int, chunks: int = 2, defer: int = 0) -> List[ChunkAction]:
    """Order seen by pipeline stage `stage` of `stages` under interleaved 1F1B with `chunks` local chunks.

    Microbatches advance in groups of `stages`: a group passes chunk 0, then chunk 1, ...; backward visits the
    chunks in reverse.  Warm-up = (stages - stage - 1) * 2 + (chunks - 1) * stages forward units, then one forward
    and one input-gradient unit alternate, then the remaining input gradients.  The weight gradient of a unit
    follows its input gradient once more than `defer` of them are waiting (defer = 0: full backward).
    M must be a multiple of `stages`.
    """
    if M % stages:
        raise ValueError("M must be a multiple of the number of stages")
    total = M * chunks

    def unit(k: int, backward: bool) -> Tuple[int, int]:
        group, r = divmod(k, stages * chunks)
        c, j = divmod(r, stages)
        return group * stages + j, (chunks - 1 - c) if backward else c

    out: List[ChunkAction] = []
    warm = min((stages - stage - 1) * 2 + (chunks - 1) * stages, total)
    f = b = w = 0
    for _ in range(warm):
        out.append(("F",) + unit(f, False))
        f += 1
    while b < total:
        if f < total:
            out.append(("F",) + unit(f, False))
            f += 1
        out.append(("dI",) + unit(b, True))
        b += 1
        if b - w > defer:
            out.append(("dW",) + unit(w, True))
            w += 1
    while w < total:
        out.append(("dW",) + unit(w, True))
        w += 1
    return out


def zb_v(M: int, stages: int, stage: int, max_live: int = 0) -> List[ChunkAction]:
    """Order seen by `stage` under a V-shaped zero-bubble placement: device d holds chunk 0 = model part d and
    chunk 1 = model part 2*stages-1-d, so a microbatch runs down the devices and back up.

    The order comes from a unit-time simulation of all stages (F, dI and dW cost one slot each): in every slot a
    stage runs the ready input gradient of the oldest microbatch if there is one, else a ready forward (while fewer
    than `max_live` tapes are alive on it; default 2 * stages), else a pending weight gradient -- weight gradients
    fill the slots that would otherwise idle.  Per chunk the weight gradients stay in microbatch order.
    """
    p = stages
    limit = max_live or 2 * p
    done = {}  # (kind, part, mb) -> slot in which it finished; part = position along the model, 0 .. 2p-1
    dev_of = lambda part: part if part < p else 2 * p - 1 - part
    orders: List[List[ChunkAction]] = [[] for _ in range(p)]
    live = [0] * p
    next_dw = [[0, 0] for _ in range(p)]  # per device and chunk: next microbatch whose dW may run
    t, remaining = 0, 3 * 2 * p * M
    while remaining:
        finished = []
        for d in range(p):
            pick = None
            # input gradients first (critical path), oldest microbatch first, the later model part first
            for m in range(M):
                for part in (2 * p - 1 - d, d):
                    if ("dI", part, m) in done or ("F", part, m) not in done:
                        continue
                    up = ("dI", part + 1, m) if part < 2 * p - 1 else ("F", part, m)
                    if up in done and done[up] < t:
                        pick = ("dI", part, m)
                        break
                if pick:
                    break
            if not pick and live[d] < limit:
                for m in range(M):
                    for part in (2 * p - 1 - d, d):
                        if ("F", part, m) in done:
                            continue
                        if part == 0 or (("F", part - 1, m) in done and done[("F", part - 1, m)] < t):
                            pick = ("F", part, m)
                            break
                    if pick:
                        break
            if not pick:
                for c, part in ((1, 2 * p - 1 - d), (0, d)):
                    m = next_dw[d][c]
                    if m < M and ("dI", part, m) in done and done[("dI", part, m)] < t:
                        pick = ("dW", part, m)
                        break
            if pick:
                finished.append((d, pick))
        for d, (kind, part, m) in finished:
            done[(kind, part, m)] = t
            c = 0 if part < p else 1
            orders[d].append((kind, m, c))
            if kind == "F":
                live[d] += 1
            elif kind == "dW":
                live[d] -= 1
                next_dw[d][c] += 1
            remaining -= 1
        t += 1
        if t > 64 * p * M:
            raise RuntimeError("schedule simulation did not finish")
    return orders[stage]


def peak_live_per_chunk(schedule: List[ChunkAction], chunks: int = 2) -> List[int]:
    """Largest number of tapes alive at once in each chunk's pool."""
    live, peak = [0] * chunks, [0] * chunks
    for a, _, c in schedule:
        if a == "F":
            live[c] += 1
            peak[c] = max(peak[c], live[c])
        elif a == "dW":
            live[c] -= 1
    return peak


def full_backward_chunks(schedule: List[ChunkAction]) -> List[ChunkAction]:
    """Same F and dI order, every dW directly after its dI."""
    out: List[ChunkAction] = []
    for a, m, c in schedule:
        if a == "dW":
            continue
        out.append((a, m, c))
        if a == "dI":
            out.append(("dW", m, c))
    return out


# ------------------------------------------------------------------------------------------------ issue plan
# A unit of the schedule ("F" | "dI" | "dW", microbatch) stands for one action per linear of the stage.  Units whose
# inputs are at hand at the same time are independent of each other, so their per-linear actions may share launches.
LayerAction = Tuple[str, int, int]  # (kind, linear, microbatch)


def plan_rounds(schedule: List[Action], n_linears: int, slots: int, max_group: int = 4, window: int = 3) -> List[List[LayerAction]]:
    """Cuts a schedule into rounds of at most `max_group` per-linear actions that may be issued together.

    Looking at most `window` units ahead of the earliest unfinished one, a round takes every action whose
    predecessors were issued in EARLIER rounds: the previous linear of its own unit (F walks the linears up, dI
    down; dW has no order among linears), the same linear of the previous unit of its kind (each linear sees the
    microbatches in schedule order), F before dI before dW of a (linear, microbatch), and a free tape slot for a
    forward (slots are released by rounds before this one).  At most one action of a kind per linear in a round,
    and never two actions of the same (linear, microbatch).  The one-action-per-round plan is the schedule itself.
    """
    units = list(schedule)
    prev_of_kind = {}
    last = {}
    for idx, (a, m) in enumerate(units):
        prev_of_kind[idx] = last.get(a)
        last[a] = idx
    todo = []  # per unit: linears still to issue, in chain order
    for a, _ in units:
        todo.append(list(range(n_linears)) if a == "F" else list(range(n_linears - 1, -1, -1)))
    issued = set()
    live = [0] * n_linears
    rounds: List[List[LayerAction]] = []
    first = 0
    while first < len(units):
        group: List[LayerAction] = []
        for idx in range(first, min(first + window, len(units))):
            a, m = units[idx]
            cands = todo[idx][:1] if a != "dW" else list(todo[idx])
            for l in cands:
                if len(group) == max_group:
                    break
                if any((a2 == a and l2 == l) or (l2 == l and m2 == m) for a2, l2, m2 in group):
                    continue
                p = prev_of_kind[idx]
                if p is not None and (a, l, units[p][1]) not in issued:
                    continue
                if a == "F" and live[l] >= slots:
                    continue
                if a == "dI" and ("F", l, m) not in issued:
                    continue
                if a == "dW" and ("dI", l, m) not in issued:
                    continue
                group.append((a, l, m))
        if not group:
            raise RuntimeError("no action is ready: the schedule is not legal for this pool size")
        for a, l, m in group:
            issued.add((a, l, m))
            idx = next(i for i in range(first, len(units)) if units[i] == (a, m))
            todo[idx].remove(l)
            if a == "F":
                live[l] += 1
            elif a == "dW":
                live[l] -= 1
        rounds.append(group)
        while first < len(units) and not todo[first]:
            first += 1
    return rounds
