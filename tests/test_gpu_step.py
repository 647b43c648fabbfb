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
        # (which slot a tape gets depends on the order of allocations and releases, which grouping changes; all else is equal)
        assert state_equal({**a, "slots": []}, {**b, "slots": []}) and a["device_token"] == b["device_token"]
    st = ctx2.stats()
    assert st["handoffs"] == 2 * 3  # one handshake pair per step instead of per action
    per_action = 3 * len(SHAPES) * (M * ((2 + 2 + 2) if staged else 5) + 1)  # kernels of the one-call-per-action run
    if staged:
        assert st["kernels_launched"] == per_action and st["grouped_dw"] == 0 and st["paired_f_di"] == 0
    else:
        # forward units directly followed by input-gradient (and weight-gradient) units went out together, and
        # weight gradients of layers that can pair shared launches: fewer kernels, same bits
        assert st["paired_f_di"] > 0 and st["grouped_dw"] > 0 and st["kernels_launched"] < per_action - 3 * M
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


MULTI_SHAPES = [(256, 512), (512, 256), (384, 384), (256, 768), (512, 512), (256, 256)]  # five of six can pair


@pytest.mark.parametrize("mode", [0, 1], ids=["eager", "graph"])
@pytest.mark.parametrize("overlap", [False, True], ids=["inline", "overlapped"])
def test_dW_multi_equals_per_layer_calls_bitwise(qe, mode, overlap):
    """One call for a microbatch's weight gradients of all layers (shared launches) against one call per layer."""
    T, M = 256, 3
    n = len(MULTI_SHAPES)
    offs, total = inputs.grad_offsets([("l", K, N) for K, N in MULTI_SHAPES])
    results = []
    for multi in (False, True):
        ctx = qe.Context(mode, overlap_dw=overlap)
        layers = [qe.Layer(ctx, T, K, N, 4, 0, M, inputs.weights("MU", 0, j, N, K).to(DEV), unit=j) for j, (K, N) in enumerate(MULTI_SHAPES)]
        grad = torch.full((total,), -3.0, device=DEV)
        Y = [torch.zeros((T, N), dtype=torch.bfloat16, device=DEV) for K, N in MULTI_SHAPES]
        dX = [torch.zeros((T, K), dtype=torch.bfloat16, device=DEV) for K, N in MULTI_SHAPES]
        for step in range(2):
            tapes = {}
            for m in range(M):
                for j, (K, N) in enumerate(MULTI_SHAPES):
                    tapes[(j, m)] = layers[j].forward(m, step, inputs.activations("MU", 0, step, j, m, T, K).to(DEV), Y[j])
            for m in range(M):
                for j, (K, N) in enumerate(MULTI_SHAPES):
                    layers[j].backward_dI(tapes[(j, m)], inputs.upstream_grads("MU", 0, step, j, m, T, N).to(DEV), dX[j])
                if multi:
                    qe.backward_dW_multi(layers, [tapes[(j, m)] for j in range(n)], grad, offs)
                else:
                    for j in range(n):
                        layers[j].backward_dW(tapes[(j, m)], grad, offs[j])
            for L in layers:
                L.optimizer_boundary(M)
        torch.cuda.synchronize()
        results.append((grad.cpu().numpy().copy(), [L.state() for L in layers], ctx.stats()))
    (g0, s0, st0), (g1, s1, st1) = results
    assert np.array_equal(g0.view(np.uint32), g1.view(np.uint32))
    assert not np.any(g1 == -3.0)  # every slice was overwritten by its first microbatch
    for a, b in zip(s0, s1):
        assert state_equal(a, b)
    assert st0["grouped_dw"] == 0 and st1["grouped_dw"] == 2 * M * 5
    # per microbatch: 4 + 1 GEMMs share two launches, the layer with N = 384 runs alone
    assert st0["kernels_launched"] - st1["kernels_launched"] == 2 * M * (n - 3)


def test_dW_multi_checks_every_layer_before_anything_runs(qe):
    T = 256
    ctx = qe.Context(0)
    shapes = MULTI_SHAPES[:3]
    layers = [qe.Layer(ctx, T, K, N, 4, 0, 2, inputs.weights("MV", 0, j, N, K).to(DEV), unit=j) for j, (K, N) in enumerate(shapes)]
    offs, total = inputs.grad_offsets([("l", K, N) for K, N in shapes])
    grad = torch.full((total,), 7.0, device=DEV)
    tapes = []
    for j, (K, N) in enumerate(shapes):
        y = torch.zeros((T, N), dtype=torch.bfloat16, device=DEV)
        dx = torch.zeros((T, K), dtype=torch.bfloat16, device=DEV)
        tapes.append(layers[j].forward(0, 0, inputs.activations("MV", 0, 0, j, 0, T, K).to(DEV), y))
        if j != 2:  # the last layer's tape has not had its dI yet
            layers[j].backward_dI(tapes[j], inputs.upstream_grads("MV", 0, 0, j, 0, T, N).to(DEV), dx)
    before = [L.state() for L in layers]
    with pytest.raises(qe.QEError) as e:
        qe.backward_dW_multi(layers, tapes, grad, offs)
    assert e.value.code == "ORDER"
    torch.cuda.synchronize()
    assert torch.all(grad == 7.0).item()
    for a, L in zip(before, layers):
        assert state_equal(a, L.state())
    with pytest.raises(qe.QEError):
        qe.backward_dW_multi([layers[0], layers[0]], [tapes[0], tapes[0]], grad, [offs[0], offs[0]])
    # the first two layers are still consumable
    qe.backward_dW_multi(layers[:2], tapes[:2], grad, offs[:2])
    torch.cuda.synchronize()
    assert not torch.any(grad[: offs[2]] == 7.0).item() and torch.all(grad[offs[2]:] == 7.0).item()


# ------------------------------------------------------------------------------------------ two local chunks
CHUNK_SHAPES = [[(256, 512), (512, 256)], [(256, 256), (256, 384)]]  # chunk -> its linears (K, N)


def _chunk_actions(s, chunk_layers):
    """(kind, mb, chunk) -> one action per linear of the chunk: forward in order, backward in reverse."""
    out = []
    for a, m, c in s:
        ls = chunk_layers[c]
        for l in (ls if a == "F" else reversed(ls)):
            out.append((a, l, m))
    return out


@pytest.mark.parametrize("gen", ["interleaved", "zb_v"])
@pytest.mark.parametrize("mode", [0, 1], ids=["eager", "graph"])
def test_two_chunk_schedules_split_equals_full_and_match_the_oracle(qe, gen, mode):
    """Two model chunks on the device, each with its own tape pools (Sec. 4.2): the interleaved and V-shaped orders
    through the whole-step call, against the same F/dI order with immediate dW (bitwise) and against the oracle."""
    from oracle.layer import OracleLinear
    from harness import assert_gemm_close, assert_grad_close, state_equal_except_Y
    from paper_2609_23536_b200.schedules import full_backward_chunks, interleaved_1f1b, peak_live_per_chunk, zb_v

    T, M, steps = 256, 4, 2
    s = interleaved_1f1b(M, 2, 0, 2, defer=2) if gen == "interleaved" else zb_v(M, 2, 0)
    flat = [kn for ch in CHUNK_SHAPES for kn in ch]
    chunk_layers, i = [], 0
    for ch in CHUNK_SHAPES:
        chunk_layers.append(list(range(i, i + len(ch))))
        i += len(ch)
    chunk_of = [c for c, ls in enumerate(chunk_layers) for _ in ls]
    offs, total = inputs.grad_offsets([("l", K, N) for K, N in flat])
    P = peak_live_per_chunk(s)

    def tensors(step):
        X = [[inputs.activations("CK", step, 0, j, m, T, K) for j, (K, N) in enumerate(flat)] for m in range(M)]
        dY = [[inputs.upstream_grads("CK", step, 0, j, m, T, N) for j, (K, N) in enumerate(flat)] for m in range(M)]
        return X, dY

    def run_gpu(schedule):
        ctx = qe.Context(mode)
        layers = [qe.Layer(ctx, T, K, N, 4, 0, P[chunk_of[j]], inputs.weights("CK", 0, j, N, K).to(DEV), unit=j)
                  for j, (K, N) in enumerate(flat)]
        grad = torch.full((total,), 2.0, device=DEV)
        outs = []
        for step in range(steps):
            Xh, dYh = tensors(step)
            X = [[t.to(DEV) for t in row] for row in Xh]
            dY = [[t.to(DEV) for t in row] for row in dYh]
            Y = [[torch.zeros((T, N), dtype=torch.bfloat16, device=DEV) for K, N in flat] for m in range(M)]
            dX = [[torch.zeros((T, K), dtype=torch.bfloat16, device=DEV) for K, N in flat] for m in range(M)]
            qe.StepPlan(ctx, layers, _chunk_actions(schedule, chunk_layers), M, X, Y, dY, dX, grad, offs).run()
            for L in layers:
                L.optimizer_boundary(M)
            torch.cuda.synchronize()
            outs.append(([[inputs.bits(t.cpu()) for t in row] for row in Y], [[inputs.bits(t.cpu()) for t in row] for row in dX],
                         grad.cpu().numpy().copy()))
        return outs, [L.state() for L in layers]

    got, st = run_gpu(s)
    full, st_full = run_gpu(full_backward_chunks(s))
    for (Y, dX, g), (Y2, dX2, g2) in zip(got, full):
        for m in range(M):
            for j in range(len(flat)):
                assert np.array_equal(Y[m][j], Y2[m][j]) and np.array_equal(dX[m][j], dX2[m][j])
        assert np.array_equal(g.view(np.uint32), g2.view(np.uint32))
    for a, b in zip(st, st_full):
        assert state_equal({**a, "slots": []}, {**b, "slots": []})

    # the oracle, driven by the same two-chunk order
    orc = [OracleLinear(T, K, N, 4, 0, P[chunk_of[j]], stage=0, unit=j) for j, (K, N) in enumerate(flat)]
    for j, (K, N) in enumerate(flat):
        orc[j].set_weight(inputs.bits(inputs.weights("CK", 0, j, N, K)))
    buf = np.full(total, 2.0, np.float32)
    for step in range(steps):
        Xh, dYh = tensors(step)
        tapes = {}
        for a, l, m in _chunk_actions(s, chunk_layers):
            L = orc[l]
            if a == "F":
                tapes[(l, m)], Yo = L.forward(m, L.e_W, inputs.bits(Xh[m][l]))
                assert_gemm_close(got[step][0][m][l], Yo, f"Y step {step} linear {l} mb {m}")
            elif a == "dI":
                dXo = L.backward_dI(tapes[(l, m)], inputs.bits(dYh[m][l]))
                assert_gemm_close(got[step][1][m][l], dXo, f"dX step {step} linear {l} mb {m}")
            else:
                L.backward_dW(tapes[(l, m)], buf, offs[l])
        assert_grad_close(got[step][2], buf, f"main_grad step {step}")
        for L in orc:
            L.optimizer_boundary(M)
    for a, L in zip(st, orc):
        # (the whole-step call issues adjacent independent units together, which changes the order of slot allocations
        # and releases and with it the slot a tape gets; everything else is equal)
        assert state_equal_except_Y({**a, "slots": []}, {**L.state(), "slots": []})


# ------------------------------------------------------------------------------------------ F and dI in one call
@pytest.mark.parametrize("mode", [0, 1], ids=["eager", "graph"])
@pytest.mark.parametrize("overlap", [False, True], ids=["inline", "overlapped-dW"])
def test_forward_dI_pair_equals_separate_calls_bitwise(qe, mode, overlap):
    """Steady state of a split-backward schedule: F(m + 2) of linear i together with dI(m) of linear n-1-i."""
    T, M = 256, 5
    shapes = [(256, 512), (512, 256), (384, 384), (256, 768)]  # F and dI GEMMs have M = T = 256: all take the paired variant
    n = len(shapes)
    offs, total = inputs.grad_offsets([("l", K, N) for K, N in shapes])
    s = sched(M, 2, 2)
    results = []
    for paired in (False, True):
        ctx = qe.Context(mode, overlap_dw=overlap)
        layers = [qe.Layer(ctx, T, K, N, 4, 0, peak_live(s), inputs.weights("PR", 0, j, N, K).to(DEV), unit=j) for j, (K, N) in enumerate(shapes)]
        grad = torch.full((total,), 1.5, device=DEV)
        Y = [[torch.zeros((T, N), dtype=torch.bfloat16, device=DEV) for K, N in shapes] for m in range(M)]
        dX = [[torch.zeros((T, K), dtype=torch.bfloat16, device=DEV) for K, N in shapes] for m in range(M)]
        for step in range(2):
            X = [[inputs.activations("PR", step, 0, j, m, T, K).to(DEV) for j, (K, N) in enumerate(shapes)] for m in range(M)]
            dY = [[inputs.upstream_grads("PR", step, 0, j, m, T, N).to(DEV) for j, (K, N) in enumerate(shapes)] for m in range(M)]
            tapes, skip = {}, False
            for k, (a, m) in enumerate(s):
                if skip:
                    skip = False
                    continue
                if paired and a == "F" and k + 1 < len(s) and s[k + 1][0] == "dI":
                    mb = s[k + 1][1]
                    for i in range(n):
                        j = n - 1 - i
                        tapes[(m, i)] = qe.forward_dI_pair(layers[i], m, step, X[m][i], Y[m][i], layers[j], tapes[(mb, j)], dY[mb][j], dX[mb][j])
                    skip = True
                elif a == "F":
                    for i in range(n):
                        tapes[(m, i)] = layers[i].forward(m, step, X[m][i], Y[m][i])
                elif a == "dI":
                    for j in range(n - 1, -1, -1):
                        layers[j].backward_dI(tapes[(m, j)], dY[m][j], dX[m][j])
                else:
                    qe.backward_dW_multi(layers, [tapes[(m, j)] for j in range(n)], grad, offs)
            for L in layers:
                L.optimizer_boundary(M)
        torch.cuda.synchronize()
        results.append(([inputs.bits(t.cpu()) for row in Y for t in row], [inputs.bits(t.cpu()) for row in dX for t in row],
                        grad.cpu().numpy().copy(), [L.state() for L in layers], ctx.stats()))
    a, b = results
    for u, v in zip(a[0] + a[1], b[0] + b[1]):
        assert np.array_equal(u, v)
    assert np.array_equal(a[2].view(np.uint32), b[2].view(np.uint32))
    for u, v in zip(a[3], b[3]):
        assert state_equal(u, v) and u["device_token"] == v["device_token"]
    n_pairs = sum(1 for k, (x, m) in enumerate(s) if x == "F" and k + 1 < len(s) and s[k + 1][0] == "dI")
    assert n_pairs == 3
    # every (i, n-1-i) pair shares a launch: one GEMM launch less per pair
    assert b[4]["paired_f_di"] == 2 * n_pairs * n and a[4]["paired_f_di"] == 0
    assert a[4]["kernels_launched"] - b[4]["kernels_launched"] == 2 * n_pairs * n * 2  # one GEMM and one cast launch less per pair


def test_forward_dI_pair_checks_both_before_anything_runs(qe):
    T = 256
    ctx = qe.Context(0)
    A = qe.Layer(ctx, T, 256, 512, 4, 0, 2, inputs.weights("PR", 0, 0, 512, 256).to(DEV), unit=0)
    B = qe.Layer(ctx, T, 512, 256, 4, 0, 2, inputs.weights("PR", 0, 1, 256, 512).to(DEV), unit=1)
    xa, ya = torch.zeros((T, 256), dtype=torch.bfloat16, device=DEV), torch.zeros((T, 512), dtype=torch.bfloat16, device=DEV)
    xb, yb = torch.zeros((T, 512), dtype=torch.bfloat16, device=DEV), torch.zeros((T, 256), dtype=torch.bfloat16, device=DEV)
    tb = B.forward(0, 0, xb, yb)
    B.backward_dI(tb, yb, xb)
    before = (A.state(), B.state())
    with pytest.raises(qe.QEError) as e:  # B's tape already had its dI: A's forward must not run either
        qe.forward_dI_pair(A, 0, 0, xa, ya, B, tb, yb, xb)
    assert e.value.code == "DUP_CONSUME"
    assert state_equal(before[0], A.state()) and state_equal(before[1], B.state())
    with pytest.raises(qe.QEError) as e:
        qe.forward_dI_pair(A, 0, 0, xa, ya, A, tb, yb, xb)
    assert e.value.code == "BAD_ARG"
    tb1 = B.forward(1, 0, xb, yb)
    ta = qe.forward_dI_pair(A, 0, 0, xa, ya, B, tb1, yb, xb)
    assert A.state()["token"] == 1 and B.state()["token"] == 4 and ta.key.mb == 0


# ------------------------------------------------------------------------------------------ independent actions together
@pytest.mark.parametrize("mode", [0, 1], ids=["eager", "graph"])
def test_run_together_equals_one_action_after_the_other_bitwise(qe, mode):
    """F(m + 2) of linear i, dI(m) of linear n-1-i and the deferred dW(m - 1) of linear i in one call each."""
    T, M = 256, 6
    shapes = [(256, 512), (512, 256), (384, 384), (256, 768)]
    n = len(shapes)
    offs, total = inputs.grad_offsets([("l", K, N) for K, N in shapes])
    s = sched(M, 2, 1)  # F0 F1 | F2 dI0 | F3 dI1 dW0 | ... : triples from the third round on
    results = []
    for together in (False, True):
        ctx = qe.Context(mode)
        layers = [qe.Layer(ctx, T, K, N, 4, 0, peak_live(s), inputs.weights("TG", 0, j, N, K).to(DEV), unit=j) for j, (K, N) in enumerate(shapes)]
        grad = torch.full((total,), -2.5, device=DEV)
        Y = [[torch.zeros((T, N), dtype=torch.bfloat16, device=DEV) for K, N in shapes] for m in range(M)]
        dX = [[torch.zeros((T, K), dtype=torch.bfloat16, device=DEV) for K, N in shapes] for m in range(M)]
        for step in range(2):
            X = [[inputs.activations("TG", step, 0, j, m, T, K).to(DEV) for j, (K, N) in enumerate(shapes)] for m in range(M)]
            dY = [[inputs.upstream_grads("TG", step, 0, j, m, T, N).to(DEV) for j, (K, N) in enumerate(shapes)] for m in range(M)]
            tapes, skip, k = {}, 0, 0
            while k < len(s):
                a, m = s[k]
                triple = together and a == "F" and k + 2 < len(s) and s[k + 1][0] == "dI" and s[k + 2][0] == "dW"
                if triple:
                    mb, mw = s[k + 1][1], s[k + 2][1]
                    for i in range(n):
                        j = n - 1 - i
                        acts = [("F", layers[i], m, step, X[m][i], Y[m][i]), ("dI", layers[j], tapes[(mb, j)], dY[mb][j], dX[mb][j]),
                                ("dW", layers[i], tapes[(mw, i)], offs[i])]
                        tapes[(m, i)] = qe.run_together(ctx, acts, grad)[0]
                    k += 3
                    continue
                if a == "F":
                    for i in range(n):
                        tapes[(m, i)] = layers[i].forward(m, step, X[m][i], Y[m][i])
                elif a == "dI":
                    for j in range(n - 1, -1, -1):
                        layers[j].backward_dI(tapes[(m, j)], dY[m][j], dX[m][j])
                else:
                    for i in range(n):
                        layers[i].backward_dW(tapes[(m, i)], grad, offs[i])
                k += 1
            for L in layers:
                L.optimizer_boundary(M)
        torch.cuda.synchronize()
        results.append(([inputs.bits(t.cpu()) for row in Y for t in row], [inputs.bits(t.cpu()) for row in dX for t in row],
                        grad.cpu().numpy().copy(), [L.state() for L in layers], ctx.stats()))
    a, b = results
    for u, v in zip(a[0] + a[1], b[0] + b[1]):
        assert np.array_equal(u, v)
    assert np.array_equal(a[2].view(np.uint32), b[2].view(np.uint32))
    assert not np.any(b[2] == -2.5)
    for u, v in zip(a[3], b[3]):
        assert state_equal({**u, "slots": []}, {**v, "slots": []}) and u["device_token"] == v["device_token"]
    n_triples = sum(1 for k in range(len(s) - 2) if s[k][0] == "F" and s[k + 1][0] == "dI" and s[k + 2][0] == "dW")
    assert n_triples == 3
    # per triple call three GEMM launches became one, except for the 384-wide linear whose dW takes the single-CTA variant
    assert a[4]["kernels_launched"] - b[4]["kernels_launched"] == 2 * n_triples * (2 * n - 1 + n)  # ... and the two casts became one
    assert b[4]["grouped_dw"] == 2 * n_triples * (n - 1)


def test_run_together_is_all_or_nothing(qe):
    T = 256
    ctx = qe.Context(0)
    A = qe.Layer(ctx, T, 256, 512, 4, 0, 2, inputs.weights("TG", 0, 0, 512, 256).to(DEV), unit=0)
    B = qe.Layer(ctx, T, 512, 256, 4, 0, 2, inputs.weights("TG", 0, 1, 256, 512).to(DEV), unit=1)
    grad = torch.full((2 * 512 * 256,), float("nan"), device=DEV)
    xa, ya = torch.ones((T, 256), dtype=torch.bfloat16, device=DEV), torch.zeros((T, 512), dtype=torch.bfloat16, device=DEV)
    xb, yb = torch.ones((T, 512), dtype=torch.bfloat16, device=DEV), torch.zeros((T, 256), dtype=torch.bfloat16, device=DEV)
    tb = B.forward(0, 0, xb, yb)
    before = (A.state(), B.state())
    # B's dW in the same call as its dI: ORDER, and A's forward must not have run
    with pytest.raises(qe.QEError) as e:
        qe.run_together(ctx, [("F", A, 0, 0, xa, ya), ("dI", B, tb, yb, xb), ("dW", B, tb, 512 * 256)], grad)
    assert e.value.code == "ORDER"
    torch.cuda.synchronize()
    assert state_equal(before[0], A.state()) and state_equal(before[1], B.state()) and torch.all(torch.isnan(grad)).item()
    with pytest.raises(qe.QEError) as e:
        qe.run_together(ctx, [("F", A, 0, 0, xa, ya), ("F", A, 1, 0, xa, ya)], grad)
    assert e.value.code == "BAD_ARG"
    (ta,) = qe.run_together(ctx, [("F", A, 0, 0, xa, ya), ("dI", B, tb, yb, xb)])
    qe.run_together(ctx, [("dI", A, ta, ya, xa), ("dW", B, tb, 512 * 256)], grad)
    torch.cuda.synchronize()
    assert not torch.any(torch.isnan(grad[512 * 256:])).item() and torch.all(torch.isnan(grad[: 512 * 256])).item()


@pytest.mark.parametrize("seed", [1, 2, 3, 4, 5, 6, 7, 8])
def test_run_together_random_groupings_equal_sequential_bitwise(qe, seed):
    """Random legal action orders over three linears and four microbatches, cut at random into groups of independent
    neighbours (at most one action of a kind per layer, a dW never in the group of its own dI): every grouping must
    give the bits of the plain one-by-one order."""
    rng = np.random.default_rng(seed)
    T, M = 256, 4
    shapes = [(256, 512), (512, 256), (256, 256)]
    n = len(shapes)
    offs, total = inputs.grad_offsets([("l", K, N) for K, N in shapes])
    # a random legal order: per (layer, mb) F < dI < dW; per layer F, dI and dW each in microbatch order
    nxt = {(k, l): 0 for k in ("F", "dI", "dW") for l in range(n)}
    order = []
    while len(order) < 3 * n * M:
        cand = []
        for l in range(n):
            if nxt[("F", l)] < M and nxt[("F", l)] - nxt[("dW", l)] < 3:  # at most three live tapes per layer
                cand.append(("F", l, nxt[("F", l)]))
            if nxt[("dI", l)] < nxt[("F", l)]:
                cand.append(("dI", l, nxt[("dI", l)]))
            if nxt[("dW", l)] < nxt[("dI", l)]:
                cand.append(("dW", l, nxt[("dW", l)]))
        k, l, m = cand[rng.integers(len(cand))]
        order.append((k, l, m))
        nxt[(k, l)] += 1
    # random grouping of neighbours
    groups, cur = [], []
    for act in order:
        k, l, m = act
        clash = any((k2 == k and l2 == l) or (l2 == l and m2 == m) for k2, l2, m2 in cur)  # same kind+layer, or same unit
        if cur and (clash or len(cur) == 4 or rng.random() < 0.3):
            groups.append(cur)
            cur = []
        cur.append(act)
    groups.append(cur)
    assert any(len(g) >= 3 for g in groups)
    results = []
    for grouped in (False, True):
        ctx = qe.Context(int(seed % 2))
        # four slots for at most three live tapes: a forward is checked against the pool as it stands before the call, so a
        # slot released by a dW of the same group is not yet available to it
        layers = [qe.Layer(ctx, T, K, N, 4, 0, 4, inputs.weights("RG", 0, j, N, K).to(DEV), unit=j) for j, (K, N) in enumerate(shapes)]
        grad = torch.full((total,), float("nan"), device=DEV)
        X = [[inputs.activations("RG", 0, 0, j, m, T, K).to(DEV) for j, (K, N) in enumerate(shapes)] for m in range(M)]
        dY = [[inputs.upstream_grads("RG", 0, 0, j, m, T, N).to(DEV) for j, (K, N) in enumerate(shapes)] for m in range(M)]
        Y = [[torch.zeros((T, N), dtype=torch.bfloat16, device=DEV) for K, N in shapes] for m in range(M)]
        dX = [[torch.zeros((T, K), dtype=torch.bfloat16, device=DEV) for K, N in shapes] for m in range(M)]
        tapes = {}
        for g in (groups if grouped else [[a] for a in order]):
            acts, fkeys = [], []
            for k, l, m in g:
                if k == "F":
                    acts.append(("F", layers[l], m, 0, X[m][l], Y[m][l]))
                    fkeys.append((l, m))
                elif k == "dI":
                    acts.append(("dI", layers[l], tapes[(l, m)], dY[m][l], dX[m][l]))
                else:
                    acts.append(("dW", layers[l], tapes[(l, m)], offs[l]))
            for key, t in zip(fkeys, qe.run_together(ctx, acts, grad)):
                tapes[key] = t
        for L in layers:
            L.optimizer_boundary(M)
        torch.cuda.synchronize()
        results.append(([inputs.bits(t.cpu()) for row in Y for t in row], [inputs.bits(t.cpu()) for row in dX for t in row],
                        grad.cpu().numpy().copy(), [L.state() for L in layers]))
    a, b = results
    for u, v in zip(a[0] + a[1], b[0] + b[1]):
        assert np.array_equal(u, v)
    assert np.array_equal(a[2].view(np.uint32), b[2].view(np.uint32)) and not np.any(np.isnan(b[2]))
    for u, v in zip(a[3], b[3]):
        assert state_equal({**u, "slots": []}, {**v, "slots": []}) and u["device_token"] == v["device_token"]


@pytest.mark.parametrize("M,w,d,window,group", [(4, 1, 0, 2, 4), (6, 3, 3, 4, 4), (5, 2, 1, 3, 8), (6, 3, 3, 6, 8)])
@pytest.mark.parametrize("mode", [0, 1], ids=["eager", "graph"])
def test_planned_rounds_equal_the_schedule_issued_action_by_action_bitwise(qe, mode, M, w, d, window, group):
    """schedules.plan_rounds regroups the schedule into rounds of independent per-linear actions; issuing a round per
    qe_run_together call must give the bits of issuing the schedule one action at a time."""
    from paper_2609_23536_b200.schedules import plan_rounds

    T = 256
    shapes = [(256, 512), (512, 256), (256, 256), (256, 768)]
    n = len(shapes)
    offs, total = inputs.grad_offsets([("l", K, N) for K, N in shapes])
    s = sched(M, w, d)
    P = peak_live(s)
    rounds = plan_rounds(s, n, P, group, window)
    assert group == 4 or any(len(g) > 4 for g in rounds)
    plain = [[(a, l, m)] for a, m in s for l in (range(n) if a == "F" else range(n - 1, -1, -1))]
    results = []
    for plan in (plain, rounds):
        ctx = qe.Context(mode)
        layers = [qe.Layer(ctx, T, K, N, 4, 0, P, inputs.weights("PL", 0, j, N, K).to(DEV), unit=j) for j, (K, N) in enumerate(shapes)]
        grad = torch.full((total,), float("nan"), device=DEV)
        Y = [[torch.zeros((T, N), dtype=torch.bfloat16, device=DEV) for K, N in shapes] for m in range(M)]
        dX = [[torch.zeros((T, K), dtype=torch.bfloat16, device=DEV) for K, N in shapes] for m in range(M)]
        for step in range(2):
            X = [[inputs.activations("PL", step, 0, j, m, T, K).to(DEV) for j, (K, N) in enumerate(shapes)] for m in range(M)]
            dY = [[inputs.upstream_grads("PL", step, 0, j, m, T, N).to(DEV) for j, (K, N) in enumerate(shapes)] for m in range(M)]
            tapes = {}
            for g in plan:
                acts, keys = [], []
                for a, l, m in g:
                    if a == "F":
                        acts.append(("F", layers[l], m, step, X[m][l], Y[m][l]))
                        keys.append((l, m))
                    elif a == "dI":
                        acts.append(("dI", layers[l], tapes[(l, m)], dY[m][l], dX[m][l]))
                    else:
                        acts.append(("dW", layers[l], tapes[(l, m)], offs[l]))
                for key, t in zip(keys, qe.run_together(ctx, acts, grad)):
                    tapes[key] = t
            for L in layers:
                L.optimizer_boundary(M)
        torch.cuda.synchronize()
        results.append(([inputs.bits(t.cpu()) for row in Y for t in row], [inputs.bits(t.cpu()) for row in dX for t in row],
                        grad.cpu().numpy().copy(), [L.state() for L in layers]))
    a, b = results
    for u, v in zip(a[0] + a[1], b[0] + b[1]):
        assert np.array_equal(u, v)
    assert np.array_equal(a[2].view(np.uint32), b[2].view(np.uint32)) and not np.any(np.isnan(b[2]))
    for u, v in zip(a[3], b[3]):
        assert state_equal({**u, "slots": []}, {**v, "slots": []}) and u["device_token"] == v["device_token"]
    assert len(rounds) < len(plain)


def test_run_together_host_equals_device_buffers_bitwise(qe):
    """Rounds with pinned HOST tensors (qe_run_together_host) against the same rounds with device tensors."""
    from paper_2609_23536_b200.schedules import plan_rounds

    T, M = 256, 4
    shapes = [(256, 512), (512, 256), (256, 256)]
    n = len(shapes)
    offs, total = inputs.grad_offsets([("l", K, N) for K, N in shapes])
    s = sched(M, 2, 1)
    P = peak_live(s)
    rounds = plan_rounds(s, n, P, 8, 4)
    results = []
    for host in (False, True):
        ctx = qe.Context(1)
        layers = [qe.Layer(ctx, T, K, N, 4, 0, P, inputs.weights("HR", 0, j, N, K).to(DEV), unit=j, host_io=host) for j, (K, N) in enumerate(shapes)]
        grad = torch.full((total,), float("nan"), device=DEV)
        place = (lambda t: t.pin_memory()) if host else (lambda t: t.to(DEV))
        X = [[place(inputs.activations("HR", 0, 0, j, m, T, K)) for j, (K, N) in enumerate(shapes)] for m in range(M)]
        dY = [[place(inputs.upstream_grads("HR", 0, 0, j, m, T, N)) for j, (K, N) in enumerate(shapes)] for m in range(M)]
        Y = [[place(torch.zeros((T, N), dtype=torch.bfloat16)) for K, N in shapes] for m in range(M)]
        dX = [[place(torch.zeros((T, K), dtype=torch.bfloat16)) for K, N in shapes] for m in range(M)]
        tapes = {}
        for g in rounds:
            acts, keys = [], []
            for a, l, m in g:
                if a == "F":
                    acts.append(("F", layers[l], m, 0, X[m][l], Y[m][l]))
                    keys.append((l, m))
                elif a == "dI":
                    acts.append(("dI", layers[l], tapes[(l, m)], dY[m][l], dX[m][l]))
                else:
                    acts.append(("dW", layers[l], tapes[(l, m)], offs[l]))
            for key, t in zip(keys, qe.run_together(ctx, acts, grad, host=host)):
                tapes[key] = t
        for L in layers:
            L.optimizer_boundary(M)
        torch.cuda.synchronize()
        results.append(([inputs.bits(t.cpu()) for row in Y for t in row], [inputs.bits(t.cpu()) for row in dX for t in row],
                        grad.cpu().numpy().copy(), [L.state() for L in layers]))
    a, b = results
    for u, v in zip(a[0] + a[1], b[0] + b[1]):
        assert np.array_equal(u, v)
    assert np.array_equal(a[2].view(np.uint32), b[2].view(np.uint32)) and not np.any(np.isnan(b[2]))
    for u, v in zip(a[3], b[3]):
        assert state_equal(u, v) and u["device_token"] == v["device_token"]
    ctx = qe.Context(0)
    L = qe.Layer(ctx, T, 256, 256, 4, 0, 2, inputs.weights("HR", 0, 0, 256, 256).to(DEV))  # no staging buffers
    with pytest.raises(qe.QEError) as e:
        qe.run_together(ctx, [("F", L, 0, 0, torch.zeros((T, 256), dtype=torch.bfloat16).pin_memory(), None)], host=True)
    assert e.value.code == "BAD_ARG"
