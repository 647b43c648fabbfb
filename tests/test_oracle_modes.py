"""Pins for the oracle's test-speed switches (CPU only).

The full-size parity tests drive the oracle with `light=True` (bookkeeping, amax and scale updates only) or with
`rows=[...]` (a few GEMM rows) and compare the GPU's class-(i) state with it.  That is sound only if neither switch
changes the state trajectory: Eqs. 3-5 make the scaling state and the token a function of the action sequence and of
the tensors' amax alone, and Invariant 1 (Sec. 3.2) forbids it to depend on whether payload bytes were produced.  These
tests run one layer three ways on the same inputs and compare everything but the payload after EVERY action; a run
whose light mode is deliberately broken must fail the same comparison.
"""
import numpy as np
import pytest

from harness import c1_inputs
from oracle import bf16
from oracle.layer import OracleLinear
from paper_2609_23536_b200 import inputs
from paper_2609_23536_b200.schedules import peak_live, sched

T, K, N = 64, 64, 96
CFG = "C1m"


def _weights(n):
    ws = [inputs.weights(CFG, 0, 0, N, K)]
    for e in range(1, n):
        ws.append(inputs.optimizer_perturbation(ws[-1], CFG, e, 0, 0))
    return [inputs.bits(w) for w in ws]


def _u32(x):
    return int(np.float32(x).view(np.uint32))


def _record(L: OracleLinear, with_Y: bool):
    """Everything of the layer but the payload bytes, as plain integers (floats by bit pattern)."""
    classes = ("X", "W", "G", "Y") if with_Y else ("X", "W", "G")
    rec = {
        "classes": {
            c: (
                tuple(int(v) for v in L.S[c].window().view(np.uint32)),
                _u32(L.S[c].scale),
                _u32(L.S[c].scale_inv),
                L.S[c].count,
            )
            for c in classes
        },
        "token": L.token,
        "e_W": L.e_W,
        "e_C": L.e_C,
        "fwd_in_epoch": L.fwd_in_epoch,
        "write_mask": L.write_mask,
        "cache_sinv_W": _u32(L.cache_sinv_W),
        "slots": tuple(
            (s.gen, s.live, s.bits, tuple(s.key) if s.live else None, _u32(s.sinv_X), _u32(s.sinv_G)) for s in L.slots
        ),
    }
    return rec


def _run(schedule, steps, M, H, mode, layer_cls=OracleLinear, heavy_at=()):
    """mode: 'heavy' | 'light' | 'rows'.  Returns the list of per-action records (and the layer).
    heavy_at: (step, kind, mb) actions that run heavy although the mode is light."""
    W = _weights(steps)
    L = layer_cls(T, K, N, H, 0, peak_live(schedule))
    buf = np.zeros(N * K, np.float32)
    trace = []
    for step in range(steps):
        L.set_weight(W[step])
        tapes = {}
        for a, m in schedule:
            X, dY = c1_inputs(step, m, T, K, N, CFG)
            light = mode == "light" and (step, a, m) not in heavy_at
            rows = [0] if mode == "rows" else None
            if a == "F":
                tapes[m], _ = L.forward(m, L.e_W, X, rows=rows, light=light)
            elif a == "dI":
                L.backward_dI(tapes[m], dY, rows=rows, light=light)
            else:
                L.backward_dW(tapes[m], buf, 0, rows=rows)
            trace.append(((step, a, m), _record(L, with_Y=(mode == "heavy"))))
        L.optimizer_boundary(M)
        trace.append(((step, "boundary", -1), _record(L, with_Y=(mode == "heavy"))))
    return trace, L, buf


def _assert_same_trajectory(ref, other):
    assert len(ref) == len(other)
    for (what, a), (what2, b) in zip(ref, other):
        assert what == what2
        a = {**a, "classes": {c: v for c, v in a["classes"].items() if c in b["classes"]}}
        assert a == b, what


CASES = [
    pytest.param(sched(4, 1, 0), 3, 4, 4, id="1f1b-4mb-3steps-H4"),
    pytest.param(sched(8, 3, 3), 1, 8, 1024, id="zb-8mb-1step-H1024"),
]


@pytest.mark.parametrize("schedule,steps,M,H", CASES)
def test_light_and_row_sampled_modes_leave_the_state_trajectory_unchanged(schedule, steps, M, H):
    heavy, Lh, _ = _run(schedule, steps, M, H, "heavy")
    light, _, _ = _run(schedule, steps, M, H, "light")
    rows, _, _ = _run(schedule, steps, M, H, "rows")
    _assert_same_trajectory(heavy, light)
    _assert_same_trajectory(heavy, rows)
    # the trajectory is not trivial: scales moved, the short history rolled over, generations advanced
    assert Lh.S["X"].count == steps * M and Lh.S["G"].count == steps * M and Lh.S["W"].count == steps
    assert Lh.S["X"].scale != 1.0 and Lh.S["G"].scale != 1.0 and Lh.S["W"].scale != 1.0
    assert Lh.token == 2 * steps * M
    assert max(s.gen for s in Lh.slots) >= 2 or steps * M <= len(Lh.slots)


def test_row_sampled_mode_writes_the_sampled_rows_of_the_heavy_results():
    s = sched(4, 1, 0)
    W = _weights(1)
    outs = []
    for rows in (None, [0, 5, 63]):
        L = OracleLinear(T, K, N, 4, 0, peak_live(s))
        L.set_weight(W[0])
        buf = np.zeros(N * K, np.float32)
        got = {}
        tapes = {}
        for a, m in s:
            X, dY = c1_inputs(0, m, T, K, N, CFG)
            if a == "F":
                tapes[m], got[("Y", m)] = L.forward(m, 0, X, rows=rows)
            elif a == "dI":
                got[("dX", m)] = L.backward_dI(tapes[m], dY, rows=rows)
            else:
                L.backward_dW(tapes[m], buf, 0, rows=rows)
        got["mg"] = buf.reshape(N, K).copy()
        outs.append(got)
    full, part = outs
    sel = [0, 5, 63]
    for k in full:
        assert np.array_equal(full[k][sel].view(np.uint8), part[k][sel].view(np.uint8) if k == "mg" else part[k].view(np.uint8)), k
    assert not part["mg"][1].any()  # an unsampled row stays untouched


@pytest.mark.parametrize("schedule,steps,M,H", CASES)
def test_heavy_action_after_a_light_refresh_uses_the_refresh_time_weight_scale(schedule, steps, M, H):
    """The lazily produced weight cache: a refresh done in light mode remembers the scale the cache is cast with;
    the first heavy action of that epoch must produce the bytes an all-heavy run holds, although the W class has
    been committed (and its scale changed) in between."""
    last = steps - 1
    # the last forward of the last step and everything of its microbatch run heavy, all else light
    m_heavy = M - 1
    heavy_at = {(last, "F", m_heavy), (last, "dI", m_heavy)}
    W = _weights(steps)

    def run(mode):
        L = OracleLinear(T, K, N, H, 0, peak_live(schedule))
        buf = np.zeros(N * K, np.float32)
        seen = {}
        for step in range(steps):
            L.set_weight(W[step])
            tapes = {}
            for a, m in schedule:
                X, dY = c1_inputs(step, m, T, K, N, CFG)
                light = mode == "light" and (step, a, m) not in heavy_at
                if a == "F":
                    tapes[m], Y = L.forward(m, L.e_W, X, light=light)
                    if (step, a, m) in heavy_at:
                        seen["Y"], seen["Wq"] = Y.copy(), L.Wq.copy()
                        seen["Xq"] = L.slots[tapes[m].ref.slot].Xq.copy()
                elif a == "dI":
                    dX = L.backward_dI(tapes[m], dY, light=light)
                    if (step, a, m) in heavy_at:
                        seen["dX"] = dX.copy()
                        seen["Gq"] = L.slots[tapes[m].ref.slot].Gq.copy()
                else:
                    if step == last and m == m_heavy:
                        # what the deferred dW is about to consume (the buffers themselves differ: the light run
                        # accumulated nothing for the earlier microbatches)
                        D = L.slots[tapes[m].ref.slot]
                        seen["dW_operands"] = (D.Xq.copy(), D.Gq.copy(), _u32(D.sinv_X), _u32(D.sinv_G))
                    L.backward_dW(tapes[m], buf, 0)
            L.optimizer_boundary(M)
        return seen

    a, b = run("heavy"), run("light")
    assert a.keys() == b.keys() and {"Y", "Wq", "Xq", "dX", "Gq", "dW_operands"} <= a.keys()
    for k in ("Y", "Wq", "Xq", "dX", "Gq"):
        assert np.array_equal(a[k], b[k]), k
    assert np.array_equal(a["dW_operands"][0], b["dW_operands"][0])
    assert np.array_equal(a["dW_operands"][1], b["dW_operands"][1])
    assert a["dW_operands"][2:] == b["dW_operands"][2:]
    # the weight scale did move between the refresh and the heavy action's epoch start (else the pin is vacuous)
    L = OracleLinear(T, K, N, H, 0, 1)
    L.set_weight(W[0])
    X, _ = c1_inputs(0, 0, T, K, N, CFG)
    before = _u32(L.S["W"].scale)
    L.forward(0, 0, X, light=True)
    assert _u32(L.S["W"].scale) != before and _u32(L._refresh_scale_W) == before


class _LightForwardDropsTheXCommit(OracleLinear):
    """A deliberately broken oracle: in light mode the forward of microbatch 2 forgets to commit the X class."""

    def forward(self, mb, gen, X_bits, rows=None, light=False):
        if light and mb == 2:
            keep = (self.S["X"].hist.copy(), self.S["X"].count, self.S["X"].scale, self.S["X"].scale_inv)
            out = super().forward(mb, gen, X_bits, rows=rows, light=light)
            self.S["X"].hist, self.S["X"].count, self.S["X"].scale, self.S["X"].scale_inv = keep
            return out
        return super().forward(mb, gen, X_bits, rows=rows, light=light)


class _LightDIKeepsAStaleSnapshot(OracleLinear):
    """A deliberately broken oracle: in light mode dI stores the inverse scale AFTER its commit in the tape."""

    def backward_dI(self, tape, dY_bits, rows=None, light=False):
        out = super().backward_dI(tape, dY_bits, rows=rows, light=light)
        if light:
            self.slots[tape.ref.slot].sinv_G = np.float32(self.S["G"].scale_inv)
        return out


@pytest.mark.parametrize("broken", [_LightForwardDropsTheXCommit, _LightDIKeepsAStaleSnapshot])
def test_a_broken_light_mode_fails_the_trajectory_comparison(broken):
    s = sched(4, 1, 0)
    heavy, _, _ = _run(s, 3, 4, 4, "heavy")
    bad, _, _ = _run(s, 3, 4, 4, "light", layer_cls=broken)
    with pytest.raises(AssertionError):
        _assert_same_trajectory(heavy, bad)


# ------------------------------------------------------------------------------------------ bf16.ulp
def test_bf16_ulp_hand_values():
    """bfloat16 has 8 significant bits: the spacing in [2^e, 2^(e+1)) is 2^(e-7); below the smallest normal 2^-126
    the spacing is the subnormal step 2^-133.  This function sets the width of every elementwise tolerance."""
    cases = [
        (1.0, 2.0**-7),
        (1.99, 2.0**-7),
        (2.0, 2.0**-6),
        (-2.0, 2.0**-6),
        (3.999, 2.0**-6),
        (0.5, 2.0**-8),
        (0.75, 2.0**-8),
        (256.0, 2.0),
        (2.0**-126, 2.0**-133),
        (2.0**-127, 2.0**-133),
        (2.0**-133, 2.0**-133),
        (0.0, 2.0**-133),
        (2.0**-125, 2.0**-132),
        (2.0**127, 2.0**120),
    ]
    v = np.array([c[0] for c in cases])
    want = np.array([c[1] for c in cases])
    assert np.array_equal(bf16.ulp(v), want)


def test_bf16_ulp_is_the_gap_between_adjacent_bit_patterns():
    """Independent of the formula: for every positive finite bfloat16 pattern b, ulp(value(b)) is
    value(b + 1) - value(b) (taken in float64, where the difference is exact)."""
    b = np.arange(0, 0x7F7F, dtype=np.uint16)  # up to the second largest finite value
    lo = bf16.decode(b).astype(np.float64)
    hi = bf16.decode((b + 1).astype(np.uint16)).astype(np.float64)
    assert np.array_equal(bf16.ulp(lo), hi - lo)
