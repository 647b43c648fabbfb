"""Pins for the oracle's delayed-scaling rule (CPU only)."""
import os

import numpy as np
import pytest

from oracle import fp8
from oracle.scaling import ScaleState, amax_bf16

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _cases():
    cases, cur = [], None
    for line in open(os.path.join(GOLD, "scale_rollover.txt")):
        body = line.split("#")[0].strip()
        if not body:
            continue
        p = body.split()
        if p[0] == "case":
            cur = dict(name=p[1], fp8_max=float(p[2]), H=int(p[3]), margin=int(p[4]), steps=[])
            cases.append(cur)
        else:
            extra = dict(kv.split("=") for kv in p[2:])
            cur["steps"].append((float(p[0]), float(p[1]), extra))
    return cases


@pytest.mark.parametrize("case", _cases(), ids=lambda c: c["name"])
def test_hand_worked_rollover(case):
    fmt = fp8.E4M3 if case["fp8_max"] == 448 else fp8.E5M2
    assert fmt.max_finite == case["fp8_max"]
    s = ScaleState(fmt, case["H"], case["margin"])
    assert s.scale == 1.0 and s.scale_inv == 1.0
    for amax, want, extra in case["steps"]:
        s.commit(np.float32(amax))
        assert s.scale == np.float32(want) or abs(float(s.scale) - want) < 1e-4 * want
        if "bits" in extra:
            assert int(np.float32(s.scale).view(np.uint32)) == int(extra["bits"], 16)
            assert int(np.float32(s.scale_inv).view(np.uint32)) == int(extra["inv_bits"], 16)


def test_known_bit_patterns():
    s = ScaleState(fp8.E4M3, 4, 0)
    s.commit(np.float32(1.0))
    assert int(s.scale.view(np.uint32)) == 0x43E00000  # 448
    assert int(s.scale_inv.view(np.uint32)) == 0x3B124925  # fp32(1/448)
    s.commit(np.float32(8.0))
    assert int(s.scale.view(np.uint32)) == 0x42600000  # 56


@pytest.mark.parametrize("H,margin", [(1, 0), (4, 0), (16, 1), (1024, 2)])
def test_closed_form_over_random_sequences(H, margin):
    rng = np.random.default_rng(H * 10 + margin)
    a = np.exp2(rng.uniform(-12, 12, size=3 * H + 7)).astype(np.float32)
    a[rng.random(a.size) < 0.1] = 0.0
    s = ScaleState(fp8.E5M2, H, margin)
    prev = np.float32(1.0)
    for t in range(a.size):
        s.commit(a[t])
        m = a[max(0, t - H + 1) : t + 1].max()
        if m > 0:
            want = np.float32(np.float32(np.float32(57344.0) / m) * np.float32(2.0**-margin))
            assert s.scale == want
            # against real arithmetic: within one fp32 rounding of 57344 / m / 2^margin
            assert abs(float(s.scale) - 57344.0 / float(m) / 2**margin) <= 2**-23 * float(s.scale)
        else:
            assert s.scale == prev
        assert s.scale_inv == np.float32(np.float32(1.0) / s.scale)
        prev = s.scale
        # logical window is newest first
        w = s.window()
        assert w[0] == a[t] and (t == 0 or H == 1 or w[1] == a[t - 1])


def test_scale_used_at_an_action_never_depends_on_its_own_amax():
    s = ScaleState(fp8.E4M3, 4, 0)
    used = []
    for amax in [2.0, 100.0, 1.0]:
        used.append(float(s.scale))  # what a quantise at this action would read
        s.commit(np.float32(amax))
    assert used == [1.0, 224.0, float(np.float32(448.0) / np.float32(100.0))]


def test_tiny_amax_clamps_scale_to_flt_max_and_nonfinite_leaves_scale():
    s = ScaleState(fp8.E5M2, 2, 0)
    s.commit(np.float32(2.0**-133))  # bf16 subnormal: 57344 / 2^-133 overflows
    assert s.scale == np.finfo(np.float32).max
    assert s.scale_inv == np.float32(np.float32(1.0) / np.finfo(np.float32).max)
    t = ScaleState(fp8.E4M3, 2, 0)
    t.commit(np.float32(4.0))
    before = (t.scale, t.scale_inv)
    t.commit(np.float32(np.inf))
    assert (t.scale, t.scale_inv) == before


def test_amax_is_max_abs():
    x = np.array([[0.5, -3.0], [2.0, -0.0]], np.float32)
    assert amax_bf16(x) == np.float32(3.0)
    assert amax_bf16(np.zeros((0,), np.float32)) == 0.0
