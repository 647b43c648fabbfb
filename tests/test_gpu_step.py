"""qe_step_run (whole action list in one call; one graph per list in graph mode) against the per-action calls."""
import numpy as np
import pytest
import torch

from harness import state_equal
from paper_2609_23536_b200 import inputs
from paper_2609_23536_b200.schedules import peak_live, sched

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def qe():
    from paper_2609_23536_b200 import build

    build.build()
    from paper_2609_23536_b200 import binding

    return binding


SHAPES = [(256, 512), (512, 256), (384, 384)]  # (K, N) of three linears; T = 256


def _setup(qe, mode, M, s, staged=False):
    T = 256
    ctx = qe.Context(mode)
    P = peak_live(s)
    layers = [qe.Layer(ctx, T, K, N, 4, 0, P, inputs.weights("ST", 0, j, N, K).to(DEV), unit=j) for j, (K, N) in enumerate(SHAPES)]
    offs, total = inputs.grad_offsets([("l", K, N) for K, N in SHAPES])
    X = [[inputs.activations("ST", 0, 0, j, m, T, K).to(DEV) for j, (K, N) in enumerate(SHAPES)] for m in range(M)]
    dY = [[inputs.upstream_grads("ST", 0, 0, j, m, T, N).to(DEV) for j, (K, N) in enumerate(SHAPES)] for m in range(M)]
    Y = [[torch.zeros((T, N), dtype=torch.bfloat16, device=DEV) for K, N in SHAPES] for m in range(M)]
    dX = [[torch.zeros((T, K), dtype=torch.bfloat16, device=DEV) for K, N in SHAPES] for m in range(M)]
    grad = torch.full((total,), 5.0, device=DEV)
    temp = torch.empty(max(K * N for K, N in SHAPES), device=DEV) if staged else None
    return ctx, layers, offs, X, Y, dY, dX, grad, temp


def _actions(s, n):
    out = []
    for a, m in s:
        for l in (range(n) if a == "F" else range(n - 1, -1, -1)):
            out.append((a, l, m))
    return out


def _snapshot(layers, Y, dX, grad):
    torch.cuda.synchronize()
    return ([inputs.bits(t.cpu()) for row in Y for t in row], [inputs.bits(t.cpu()) for row in dX for t in row],
            grad.cpu().numpy().copy(), [{**L.state(), "slot_sinv_X": 0, "slot_sinv_G": 0} for L in layers])


@pytest.mark.parametrize("mode", [0, 1], ids=["eager", "graph"])
@pytest.mark.parametrize("staged", [False, True])
def test_step_call_equals_per_action_calls_bitwise(qe, mode, staged):
    M = 4
    s = sched(M, 2, 1)
    acts = _actions(s, len(SHAPES))
    # reference: the single calls
    ctx, layers, offs, X, Y, dY, dX, grad, temp = _setup(qe, mode, M, s, staged)
    for step in range(3):
        tapes = {}
        for a, l, m in acts:
            L = layers[l]
            if a == "F":
                tapes[(l, m)] = L.forward(m, step, X[m][l], Y[m][l])
            elif a == "dI":
                L.backward_dI(tapes[(l, m)], dY[m][l], dX[m][l])
            elif staged:
                L.backward_dW_staged(tapes[(l, m)], grad, offs[l], temp)
            else:
                L.backward_dW(tapes[(l, m)], grad, offs[l])
        for L in layers:
            L.optimizer_boundary(M)
    want = _snapshot(layers, Y, dX, grad)
    # the whole list in one call per step
    ctx2, layers2, offs2, X2, Y2, dY2, dX2, grad2, temp2 = _setup(qe, mode, M, s, staged)
    plan = qe.StepPlan(ctx2, layers2, acts, M, X2, Y2, dY2, dX2, grad2, offs2, temp2)
    for step in range(3):
        plan.run()
        for L in layers2:
            L.optimizer_boundary(M)
    got = _snapshot(layers2, Y2, dX2, grad2)
    for a, b in zip(want[0] + want[1], got[0] + got[1]):
        assert np.array_equal(a, b)
    assert np.array_equal(want[2].view(np.uint32), got[2].view(np.uint32))
    for a, b in zip(want[3], got[3]):
        assert state_equal(a, b) and a["device_token"] == b["device_token"]
    st = ctx2.stats()
    assert st["handoffs"] == 2 * 3  # one handshake pair per step instead of per action
    n_kernels = 3 * len(SHAPES) * (M * ((2 + 2 + 2) if staged else 5) + 1)
    assert st["kernels_launched"] == n_kernels
    if mode == 1:
        assert st["graphs_built"] == 1 and st["graph_replays"] == 3


def test_step_call_failure_aborts_at_the_failing_action(qe):
    M = 2
    s = sched(M, 2, 0)
    ctx, layers, offs, X, Y, dY, dX, grad, temp = _setup(qe, 0, M, s)
    acts = _actions(s, len(SHAPES))
    bad = acts[: len(acts) // 2] + [("dI", 0, 0), ("dI", 0, 0)] + acts[len(acts) // 2:]  # a repeated dI somewhere
    plan = qe.StepPlan(ctx, layers, bad, M, X, Y, dY, dX, grad, offs)
    with pytest.raises(qe.QEError) as e:
        plan.run()
    assert e.value.code in ("DUP_CONSUME", "STALE_REF") and "step aborted at action" in str(e.value)
    for L in layers:
        st = L.state()
        assert st["aborted"] and st["device_token"] == st["token"]  # the valid prefix ran: host and device agree
        assert all(not sl["live"] for sl in st["slots"])
        L.arena_rebuild()
    # after the rebuild the epoch restarts cleanly
    plan2 = qe.StepPlan(ctx, layers, acts, M, X, Y, dY, dX, grad, offs)
    plan2.run()
    for L in layers:
        L.optimizer_boundary(M)
        assert L.state()["e_W"] == 1
