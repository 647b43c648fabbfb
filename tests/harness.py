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
                layer.backward_dW(tapes[m], buf, off)
            if on_action:
                on_action(step, a, m, layer)
        outs[(step, "mg")] = buf.copy()
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
