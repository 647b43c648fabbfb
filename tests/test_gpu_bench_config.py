"""The launch configuration bench.py times (config 2 at full size: graph mode, forward + input-gradient (+ deferred
weight-gradient) units issued together in shared launches, the other weight gradients grouped on the second stream)
against plain one-action-per-call eager execution, bit for bit, and against the oracle on one linear's state and
sampled gradient rows."""
import os
import sys

import numpy as np
import pytest
import torch

from harness import assert_grad_close, dW_abs_products, state_diff, state_equal, state_equal_except_Y
from oracle.layer import OracleLinear
from paper_2609_23536_b200 import inputs
from paper_2609_23536_b200.schedules import peak_live

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def qe():
    from paper_2609_23536_b200 import build

    build.build()
    from paper_2609_23536_b200 import binding

    return binding


def test_bench_launch_configuration_equals_single_calls_and_oracle(qe):
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench

    cfg = inputs.CONFIGS["C2"]
    M, T, steps = cfg["M"], cfg["T"], 2
    device = torch.device("cuda", 0)
    with torch.cuda.stream(torch.cuda.Stream(device)):
        stage = bench.Stage(qe, "C2", cfg, "graph", device, same_stream=True, overlap_dw=True,
                            plan_window=cfg["sched"][0] + cfg["sched"][1])  # bench.py's defaults
        for _ in range(steps):
            stage.step()
        torch.cuda.synchronize()
        st = stage.ctx.stats()
        assert st["paired_f_di"] > 0 and st["grouped_dw"] > 0 and len(stage.rounds) < 40  # the shared launches were really used
        n = len(stage.layers)

        # the same tensors through one call per action, eager, no second stream
        ctx = qe.Context(qe.EAGER)
        ref = [qe.Layer(ctx, T, L.K, L.N, cfg["H"], cfg["margin"], peak_live(stage.schedule), L.weight.clone(), unit=i)
               for i, L in enumerate(stage.layers)]
        grad = torch.zeros_like(stage.grad)
        Y = [[torch.empty_like(t) for t in row] for row in stage.Y]
        dX = [[torch.empty_like(t) for t in row] for row in stage.dX]
        for step in range(steps):
            tapes = {}
            for a, m in stage.schedule:
                for i in (range(n) if a == "F" else range(n - 1, -1, -1)):
                    if a == "F":
                        tapes[(m, i)] = ref[i].forward(m, step, stage.X[m][i], Y[m][i])
                    elif a == "dI":
                        ref[i].backward_dI(tapes[(m, i)], stage.dY[m][i], dX[m][i])
                    else:
                        ref[i].backward_dW(tapes[(m, i)], grad, stage.offsets[i])
            for L in ref:
                L.optimizer_boundary(M)
        torch.cuda.synchronize()
        for m in range(M):
            for i in range(n):
                assert torch.equal(stage.Y[m][i].view(torch.int16), Y[m][i].view(torch.int16)), ("Y", m, i)
                assert torch.equal(stage.dX[m][i].view(torch.int16), dX[m][i].view(torch.int16)), ("dX", m, i)
        assert torch.equal(stage.grad.view(torch.int32), grad.view(torch.int32))
        for a, b in zip(stage.layers, ref):
            sa, sb = a.state(), b.state()
            assert state_equal({**sa, "slots": []}, {**sb, "slots": []}) and sa["device_token"] == sb["device_token"] and sa["device_status"] == 0

        # the oracle on every linear of the block: state after two steps (bit-exact) and sampled gradient rows of the
        # second step, element by element.  The attention output projection runs its casts in both steps; the
        # others (qkv, the 92 MB gate_up slice, down) advance through step 1 on amax values alone and cast in step 2
        for u in (1, 0, 2, 3):
            L = stage.layers[u]
            O = OracleLinear(T, L.K, L.N, cfg["H"], cfg["margin"], peak_live(stage.schedule), unit=u)
            O.set_weight(inputs.bits(L.weight.cpu()))
            rows = [0, 1, 777, L.N - 1] if u == 1 else [0, 255, 256, 1531, L.N - 129, L.N - 1]
            obuf = np.zeros(L.N * L.K, np.float32)
            for step in range(steps):
                light = u != 1 and step < steps - 1
                tapes, absp = {}, 0.0
                for a, m in stage.schedule:
                    if a == "F":
                        tapes[m], _ = O.forward(m, step, inputs.bits(stage.X[m][u].cpu()), rows=[0], light=light)
                    elif a == "dI":
                        O.backward_dI(tapes[m], inputs.bits(stage.dY[m][u].cpu()), rows=[0], light=light)
                    else:
                        if not light:
                            absp = absp + dW_abs_products(O.slots[tapes[m].ref.slot], rows)
                        O.backward_dW(tapes[m], obuf, 0, rows=rows)
                O.optimizer_boundary(M)
            # (slot generations are identities of this process and follow the issue order: the planned rounds reuse slots in
            # another order than the schedule the oracle walks)
            gs, os_ = {**L.state(), "slots": []}, {**O.state(), "slots": []}
            assert state_equal_except_Y(gs, os_), (u, state_diff(gs, os_))
            got = stage.grad[stage.offsets[u]: stage.offsets[u] + L.N * L.K].view(L.N, L.K)[rows].cpu().numpy()
            assert_grad_close(got, obuf.reshape(L.N, L.K)[rows], ("bench issue order, linear", u), abs_products=absp, rel_tol=1e-5, contraction=T)
