"""Shared test driver: runs a schedule through any backend that has the layer interface
(forward / backward_dI / backward_dW / optimizer_boundary / state), oracle or CUDA binding."""
from __future__ import annotations

import numpy as np

from paper_2609_23536_b200 import inputs
from paper_2609_23536_b200.schedules import sched


def c1_inputs(step, mb, T=256, K=256, N=256, cfg="C1"):
    X = inputs.bits(inputs.activations(cfg, step, 0, 0, mb, T, K))
    dY = inputs.bits(inputs.upstream_grads(cfg, step, 0, 0, mb, T, N))
    return X, dY


def run_oracle_steps(layer, schedule, steps, M, buf, off, get_inputs, weight_for_step, on_action=None):
    """Drive an OracleLinear through `steps` optimizer steps of `schedule`."""
    outs = {}
    for step in range(steps):
        layer.set_weight(weight_for_step(step))
        tapes = {}
        for a, m in schedule:
            X, dY = get_inputs(step, m)
            if a == "F":
                tapes[m], Y = layer.forward(m, layer.e_W, X)
                outs[(step, "Y", m)] = Y
            elif a == "dI":
                outs[(step, "dX", m)] = layer.backward_dI(tapes[m], dY)
            else:
                slot = layer.slots[tapes[m].ref.slot]
                if layer.write_mask == 0:
                    absp = np.zeros(layer.N * layer.K)
                absp += dW_abs_products(slot, np.arange(layer.N)).reshape(-1)
                layer.backward_dW(tapes[m], buf, off)
            if on_action:
                on_action(step, a, m, layer)
        outs[(step, "mg")] = buf.copy()
        # what the FP32 error of this step's gradient slice scales with (see assert_grad_close), slice only
        outs[(step, "mg_abs")] = absp
        layer.optimizer_boundary(M)
    return outs


def state_equal(a: dict, b: dict) -> bool:
    """Bitwise comparison of two oracle-style state dicts."""
    for c in a["classes"]:
        x, y = a["classes"][c], b["classes"][c]
        if not np.array_equal(x["window"].view(np.uint32), y["window"].view(np.uint32)):
            return False
        for k in ("scale", "scale_inv"):
            if np.float32(x[k]).view(np.uint32) != np.float32(y[k]).view(np.uint32):
                return False
        if x["count"] != y["count"]:
            return False
    keys = ("token", "e_W", "e_C", "write_mask", "fwd_in_epoch", "aborted", "slots")
    return all(a[k] == b[k] for k in keys)


# ----------------------------------------------------------------------------------------- GPU side
def run_gpu_steps(qe, layer, schedule, steps, M, grad_buf, off, get_inputs, weight_for_step, on_action=None,
                  staged_temp=None, stream=None):
    """Drive a binding.Layer through `steps` optimizer steps; returns outputs keyed like run_oracle_steps
    (as numpy: bf16 bits for Y/dX, float32 for the gradient buffer)."""
    import torch

    dev = layer.weight.device
    outs = {}
    for step in range(steps):
        layer.weight.copy_(inputs.from_bits(weight_for_step(step)).to(dev))
        tapes = {}
        for a, m in schedule:
            X, dY = get_inputs(step, m)
            if a == "F":
                x = inputs.from_bits(X).to(dev)
                y = torch.empty((layer.T, layer.N), dtype=torch.bfloat16, device=dev)
                gen = layer.state()["e_W"]  # the caller's view of the weight version
                tapes[m] = layer.forward(m, gen, x, y, stream)
                outs[(step, "Y", m)] = y
            elif a == "dI":
                dy = inputs.from_bits(dY).to(dev)
                dx = torch.empty((layer.T, layer.K), dtype=torch.bfloat16, device=dev)
                layer.backward_dI(tapes[m], dy, dx, stream)
                outs[(step, "dX", m)] = dx
            elif staged_temp is not None:
                layer.backward_dW_staged(tapes[m], grad_buf, off, staged_temp, stream)
            else:
                layer.backward_dW(tapes[m], grad_buf, off, stream)
            if on_action:
                on_action(step, a, m, layer, tapes[m])
        torch.cuda.synchronize()
        layer.optimizer_boundary(M)  # with overlapped dW the gradient buffer is complete only after the boundary
        outs[(step, "mg")] = grad_buf.clone()
    res = {}
    for k, v in outs.items():
        res[k] = v.cpu().numpy() if k[1] == "mg" else inputs.bits(v.cpu())
    return res


FLOOR_ONLY = {"elements": 0, "floor_only": 0}  # running count over a test session (see assert_gemm_close)


def assert_gemm_close(got_bits, want_bits, what=""):
    """bf16 outputs: relative Frobenius <= 1e-3 and <= 4 bf16 ulp elementwise.  The ulp is taken at the oracle's
    magnitude, except that it is never taken below 2^-6 of the tensor's rms: an output that is small because large
    products cancelled carries the FP32 accumulation error of those products (which scales with the sum of their
    magnitudes, not with the result), so 4 ulp of its own tiny magnitude is not a bound the arithmetic can meet.
    Elements that pass only thanks to that floor are counted; they must stay under 0.5 % of the tensor (for Gaussian
    outputs 1.2 % of the elements lie below the floor at all, and few of those need it)."""
    from oracle import bf16

    g = bf16.decode(got_bits).astype(np.float64)
    w = bf16.decode(want_bits).astype(np.float64)
    denom = np.linalg.norm(w)
    rel = np.linalg.norm(g - w) / denom if denom > 0 else np.abs(g).max()
    assert rel <= 1e-3, (what, rel)
    floor = 2.0**-6 * np.sqrt(np.mean(w**2))
    err = np.abs(g - w)
    ok = err <= 4 * bf16.ulp(np.maximum(np.abs(w), floor))
    assert ok.all(), (what, int((~ok).sum()), err.max())
    floor_only = int((err > 4 * bf16.ulp(np.abs(w))).sum())
    FLOOR_ONLY["elements"] += g.size
    FLOOR_ONLY["floor_only"] += floor_only
    assert floor_only <= max(2, 0.005 * g.size), (what, "elements within 4 ulp only at the floored magnitude", floor_only, g.size)
    return rel


def dW_abs_products(slot, rows):
    """sum_t |dec(Gq[t,n])| |dec(Xq[t,k])| * sinv_G * sinv_X for the rows n of one oracle tape slot (float64 [len(rows), K]):
    the quantity the rounding error of an FP32-accumulated weight gradient scales with.  Call before the oracle's dW
    releases the slot."""
    from oracle import fp8

    G = np.abs(fp8.decode(slot.Gq[:, np.asarray(rows)], fp8.E5M2))
    X = np.abs(fp8.decode(slot.Xq, fp8.E4M3))
    return (G.T @ X) * float(slot.sinv_G) * float(slot.sinv_X)


GRAD_ULPS = 8.0  # per-element FP32 bound for ordinary data, in units of 2^-24 * sum |products| (see assert_grad_close)


def assert_grad_close(got, want, what="", abs_products=None, rel_tol=1e-3, contraction=None):
    """FP32 gradient against the oracle's (exact products, one rounding per microbatch): relative Frobenius error, and
    -- given abs_products = sum over the microbatches written so far of dW_abs_products, and the contraction length T --
    an elementwise bound in units of u = 2^-24 * abs_products:

      * no element beyond (2 * T / 32 + 8) u.  The tensor cores add the products of 32 contraction indices to the FP32
        accumulator per instruction; each such step, the multiply by alpha and the addition to the buffer lose at most
        one unit in the last place (2^-23, chopping allowed for) of a magnitude that never exceeds the sum of the
        absolute products.  This is what FP32 accumulation guarantees whatever the data.
      * at most 1 % of the elements beyond GRAD_ULPS u.  On data without a dominating product the partial sums stay far
        below sum|p| and the errors add up like a random walk; only where one huge product sits in the accumulator for
        the rest of the contraction (the 1000x outliers of the rollover stress) does an element approach the first bound.

    A wrong, missing or doubled product of typical size is sum|p| / T = 2^-11..2^-12 of sum|p|, far outside both."""
    g, w = got.astype(np.float64), want.astype(np.float64)
    denom = np.linalg.norm(w)
    rel = np.linalg.norm(g - w) / denom if denom > 0 else np.abs(g).max()
    assert rel <= rel_tol, (what, rel)
    if abs_products is not None:
        assert contraction is not None
        u = 2.0**-24 * abs_products + 2.0**-149
        err = np.abs(g - w) / u
        hard = 2.0 * contraction / 32 + 8
        assert (err <= hard).all(), (what, "beyond the FP32 accumulation bound", int((err > hard).sum()), float(err.max()), hard)
        frac = float((err > GRAD_ULPS).mean())
        assert frac <= 0.01, (what, "share of elements beyond GRAD_ULPS", frac, float(err.max()))
    return rel


def state_equal_except_Y(gpu: dict, orc: dict) -> bool:
    """Class (i) state: bit-exact.  The Y class hangs off a GEMM result (tolerance class) and is
    checked separately."""
    for c in ("X", "W", "G"):
        x, y = gpu["classes"][c], orc["classes"][c]
        if not np.array_equal(x["window"].view(np.uint32), y["window"].view(np.uint32)):
            return False
        for k in ("scale", "scale_inv"):
            if np.float32(x[k]).view(np.uint32) != np.float32(y[k]).view(np.uint32):
                return False
        if x["count"] != y["count"]:
            return False
    keys = ("token", "e_W", "e_C", "write_mask", "fwd_in_epoch", "aborted", "slots")
    return all(gpu[k] == orc[k] for k in keys)


def transposed_or_none(layer, which, slot=0):
    """A layer's transposed FP8 copy (which = 1, 3, 5), or None when the layer keeps none because its GEMMs read the
    row-major tensor as an MN-major operand."""
    from paper_2609_23536_b200 import binding as qe

    try:
        return layer.read_fp8(which, slot)
    except qe.QEError as e:
        assert e.code == "UNSUPPORTED"
        return None


def state_diff(gpu: dict, orc: dict, classes=("X", "W", "G")) -> list:
    """Names of the fields in which two state dicts differ (for assertion messages)."""
    out = []
    for c in classes:
        x, y = gpu["classes"][c], orc["classes"][c]
        a, b = x["window"].view(np.uint32), y["window"].view(np.uint32)
        if not np.array_equal(a, b):
            i = int(np.argmax(a != b))
            out.append(f"{c}.window[{i}]: {x['window'][i]!r} != {y['window'][i]!r} ({int((a != b).sum())} entries differ)")
        for k in ("scale", "scale_inv"):
            if np.float32(x[k]).view(np.uint32) != np.float32(y[k]).view(np.uint32):
                out.append(f"{c}.{k}: {x[k]!r} != {y[k]!r}")
        if x["count"] != y["count"]:
            out.append(f"{c}.count: {x['count']} != {y['count']}")
    for k in ("token", "e_W", "e_C", "write_mask", "fwd_in_epoch", "aborted", "slots"):
        if gpu[k] != orc[k]:
            out.append(f"{k}: {gpu[k]!r} != {orc[k]!r}")
    return out
