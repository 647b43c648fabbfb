"""GPU parity of the layer (F / dI / dW through the C-ABI) against the oracle, action by action."""
import numpy as np
import pytest
import torch

from harness import (assert_gemm_close, assert_grad_close, c1_inputs, run_gpu_steps, run_oracle_steps, state_equal,
                     state_equal_except_Y, transposed_or_none)
from oracle import bf16, fp8
from oracle.layer import ContractError, OracleLinear
from paper_2609_23536_b200 import inputs
from paper_2609_23536_b200.schedules import full_backward, peak_live, sched

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def qe():
    from paper_2609_23536_b200 import build

    build.build()
    from paper_2609_23536_b200 import binding

    return binding


def _weights(cfg, N, K, steps):
    ws = [inputs.weights(cfg, 0, 0, N, K)]
    for e in range(1, steps):
        ws.append(inputs.optimizer_perturbation(ws[-1], cfg, e, 0, 0))
    return [inputs.bits(w) for w in ws]


def _mk_layer(qe, mode, T, K, N, H, margin, P, overlap=False):
    ctx = qe.Context(mode, overlap_dw=overlap)
    w = torch.zeros((N, K), dtype=torch.bfloat16, device=DEV)
    return ctx, qe.Layer(ctx, T, K, N, H, margin, P, w)


def _scale_from_window(window, fp8_max, margin, prev):
    m = np.float32(window.max())
    if not (np.isfinite(m) and m > 0):
        return prev
    return np.float32(np.float32(np.float32(fp8_max) / m) * np.float32(2.0**-margin))


@pytest.mark.parametrize("mode", [0, 1], ids=["eager", "graph"])
def test_config1_every_action_against_oracle(qe, mode):
    # Single linear 256^3, history 4, margin 0, 4 microbatches x 3 steps in 1F1B order: the history rolls over.
    T = K = N = 256
    M, steps, H = 4, 3, 4
    s = sched(M, 1, 0)
    P = peak_live(s)
    W = _weights("C1", N, K, steps)
    get = lambda step, mb: c1_inputs(step, mb, T, K, N, "C1")
    O = OracleLinear(T, K, N, H, 0, P)
    obuf = np.zeros(N * K + 64, np.float32)
    otrace = []
    oouts = run_oracle_steps(O, s, steps, M, obuf, 64, get, lambda e: W[e],
                             on_action=lambda st, a, m, L: otrace.append((st, a, m, L.state(),
                                       {p: (sl.Xq, sl.Gq, sl.sinv_X, sl.sinv_G) for p, sl in enumerate(L.slots) if sl.live},
                                       L.Wq.copy(), L.cache_sinv_W)))
    ctx, L = _mk_layer(qe, mode, T, K, N, H, 0, P)
    gbuf = torch.full((N * K + 64,), 7.0, device=DEV)  # garbage: the first write of an epoch must overwrite
    it = iter(otrace)
    prevY = [np.float32(1.0)]

    def check(step, a, m, layer, tape):
        ost, oa, om, ostate, oslots, oWq, osinvW = next(it)
        assert (ost, oa, om) == (step, a, m)
        g = layer.state()
        assert g["device_status"] == 0 and g["device_token"] == g["token"]
        assert state_equal_except_Y(g, ostate), (step, a, m)
        assert np.float32(g["cache_sinv_W"]).view(np.uint32) == np.float32(osinvW).view(np.uint32)
        assert np.array_equal(layer.read_fp8(4), oWq)
        assert transposed_or_none(layer, 5) is None  # 256-multiples: the dI GEMM reads Wq itself, MN-major
        for p, (Xq, Gq, sX, sG) in oslots.items():
            assert np.array_equal(layer.read_fp8(0, p), Xq) and transposed_or_none(layer, 1, p) is None
            assert g["slot_sinv_X"][p].view(np.uint32) == np.float32(sX).view(np.uint32)
            if Gq is not None:
                assert np.array_equal(layer.read_fp8(2, p), Gq) and transposed_or_none(layer, 3, p) is None
                assert g["slot_sinv_G"][p].view(np.uint32) == np.float32(sG).view(np.uint32)
        # class Y: newest entry is max|Y_gpu| exactly; its scale is the closed form of the GPU's own window
        gy = g["classes"]["Y"]
        assert gy["count"] == ostate["classes"]["Y"]["count"]
        want = _scale_from_window(gy["window"], 448.0, 0, prevY[0])
        assert gy["scale"].view(np.uint32) == want.view(np.uint32)
        assert gy["scale_inv"].view(np.uint32) == np.float32(np.float32(1.0) / want).view(np.uint32)
        prevY[0] = want
        oy = ostate["classes"]["Y"]["window"]
        assert np.all(np.abs(gy["window"].astype(np.float64) - oy) <= 4 * bf16.ulp(oy))

    gouts = run_gpu_steps(qe, L, s, steps, M, gbuf, 64, get, lambda e: W[e], on_action=check)
    assert set(gouts) == {k for k in oouts if k[1] != "mg_abs"}
    for k in gouts:
        if k[1] == "mg":
            assert np.array_equal(gouts[k][:64], np.full(64, 7.0, np.float32))  # nothing outside the slice
            rel = assert_grad_close(gouts[k][64:], oouts[k][64:], k, abs_products=oouts[(k[0], "mg_abs")], contraction=T)
            assert rel < 1e-5, rel
        else:
            assert_gemm_close(gouts[k], oouts[k], k)
    # newest Y amax equals max|Y| of the last forward, exactly
    lastY = bf16.decode(gouts[(steps - 1, "Y", M - 1)])
    assert L.state()["classes"]["Y"]["window"][0] == np.abs(lastY).max()
    st = ctx.stats()
    n_actions = steps * 3 * M
    assert st["handoffs"] == 2 * n_actions
    if mode == 1:
        assert st["graphs_built"] == 3 * P + 1  # one F/dI/dW triple per slot + the cache refresh
        assert st["graph_replays"] == n_actions + steps and st["eager_launches"] == 0
    else:
        assert st["graphs_built"] == 0 and st["eager_launches"] == st["kernels_launched"]
    assert st["kernels_launched"] == steps * (M * (2 + 2 + 1) + 1)  # quantise+GEMM, quantise+GEMM, GEMM; + weight refresh


def _run_variant(qe, mode, schedule, staged=False, T=256, K=384, N=512, M=4, steps=2, H=4, overlap=False):
    P = max(peak_live(schedule), 2)
    W = _weights("V", N, K, steps)
    get = lambda step, mb: c1_inputs(step, mb, T, K, N, "V")
    ctx, L = _mk_layer(qe, mode, T, K, N, H, 1, P, overlap)
    gbuf = torch.zeros(N * K, device=DEV)
    temp = torch.empty(N * K, device=DEV) if staged else None
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        outs = run_gpu_steps(qe, L, schedule, steps, M, gbuf, 0, get, lambda e: W[e], staged_temp=temp)
    st = L.state()
    return outs, {**st, "slots": [], "slot_sinv_X": 0, "slot_sinv_G": 0}


def _same(a, b):
    (oa, sa), (ob, sb) = a, b
    assert oa.keys() == ob.keys()
    for k in oa:
        assert np.array_equal(oa[k].view(np.uint8), ob[k].view(np.uint8)), k
    assert state_equal(sa, sb) and sa["device_token"] == sb["device_token"]


def test_split_equals_full_backward_bitwise(qe):
    s = sched(4, 2, 1)
    _same(_run_variant(qe, 0, s), _run_variant(qe, 0, full_backward(s)))


def test_graph_replay_equals_eager_bitwise(qe):
    s = sched(4, 2, 1)
    _same(_run_variant(qe, 0, s), _run_variant(qe, 1, s))
    _same(_run_variant(qe, 0, full_backward(s)), _run_variant(qe, 1, s))


@pytest.mark.parametrize("mode", [0, 1])
def test_staged_copy_path_equals_direct_placement_bitwise(qe, mode):
    s = sched(4, 2, 1)
    _same(_run_variant(qe, mode, s), _run_variant(qe, mode, s, staged=True))


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("staged", [False, True])
def test_overlapped_dW_stream_gives_the_same_bits(qe, mode, staged):
    # dW on the context's second stream (joined at the optimizer boundary): same outputs, same state
    s = sched(8, 3, 3)
    kw = dict(M=8, T=512, K=512, N=768, steps=3)
    _same(_run_variant(qe, mode, s, staged=staged, **kw), _run_variant(qe, mode, s, staged=staged, overlap=True, **kw))


@pytest.mark.parametrize("mode", [0, 1], ids=["eager", "graph"])
def test_shapes_that_take_the_single_cta_gemm_against_oracle(qe, mode):
    # T and N multiples of 128 but not of 256: F, dI and dW all run the 128 x 256-tile variant, with ragged last tiles
    T, K, N, M, H = 384, 640, 896, 3, 4
    s = sched(M, 2, 1)
    P = peak_live(s)
    W = _weights("S", N, K, 2)
    get = lambda step, mb: c1_inputs(step, mb, T, K, N, "S")
    O = OracleLinear(T, K, N, H, 0, P)
    obuf = np.zeros(N * K, np.float32)
    want = run_oracle_steps(O, s, 2, M, obuf, 0, get, lambda e: W[e])
    ctx, L = _mk_layer(qe, mode, T, K, N, H, 0, P)
    gbuf = torch.full((N * K,), -1.0, device=DEV)
    got = run_gpu_steps(qe, L, s, 2, M, gbuf, 0, get, lambda e: W[e])
    for k in got:
        if k[1] == "mg":
            assert assert_grad_close(got[k], want[k], k, abs_products=want[(k[0], "mg_abs")], contraction=T) < 1e-5
        else:
            assert_gemm_close(got[k], want[k], k)
    assert state_equal_except_Y(L.state(), O.state())
    # these shapes keep transposed copies (their dI / dW GEMMs take contraction-major operands only)
    assert np.array_equal(L.read_fp8(5), O.Wq.T) and np.array_equal(L.read_fp8(4), O.Wq)
    assert L.read_fp8(1, 0).shape == (K, T) and L.read_fp8(3, 0).shape == (N, T)


def test_scale_commit_standalone_matches_hand_worked_rollover(qe):
    ctx, L = _mk_layer(qe, 0, 256, 256, 256, 4, 0, 1)
    seq = [1, 8, 2, 2, 2, 2, 0.5, 0, 0, 0, 0, 3]
    want = [448, 56, 56, 56, 56, 224, 224, 224, 224, 896, 896, None]
    for a, w in zip(seq, want):
        L.scale_commit(qe.CLASS_X, torch.tensor([a], dtype=torch.float32, device=DEV))
        s = L.state()["classes"]["X"]
        if w is not None:
            assert s["scale"] == np.float32(w)
    assert s["scale"].view(np.uint32) == 0x43155555 and s["scale_inv"].view(np.uint32) == 0x3BDB6DB7
    assert list(s["window"]) == [3.0, 0.0, 0.0, 0.0] and s["count"] == 12
    assert L.state()["device_token"] == 0  # a standalone commit does not advance the effect token
    # E5M2 class with margin handled by the same kernel
    ctx2, L2 = _mk_layer(qe, 1, 256, 256, 256, 4, 1, 1)
    for a, w in zip([1, 8, 2, 2, 2, 2], [28672, 3584, 3584, 3584, 3584, 14336]):
        L2.scale_commit(qe.CLASS_G, torch.tensor([a], dtype=torch.float32, device=DEV))
        assert L2.state()["classes"]["G"]["scale"] == np.float32(w)


def _bits(x):
    return int(np.float32(x).view(np.uint32))


@pytest.mark.parametrize("cls,fmt,margin", [("X", fp8.E4M3, 0), ("G", fp8.E5M2, 1), ("W", fp8.E4M3, -2)])
def test_scale_commit_edge_cases_against_the_oracle(qe, cls, fmt, margin):
    # What the scale rule does at the edges of its domain, compared with the oracle's ScaleState bit for bit after
    # every commit: an amax so small that fp8_max / amax overflows (scale clamps to the largest finite binary32 and its
    # inverse is a subnormal), +Inf and NaN entries (stored in the window, scale and inverse left alone until they
    # have rolled out), and a window that becomes all zero (scale left alone again).
    from oracle.scaling import ScaleState

    H = 4
    ctx, L = _mk_layer(qe, 0, 256, 256, 256, H, margin, 1)
    O = ScaleState(fmt, H, margin)
    seq = [2.0**-133, 0.0, float("inf"), 1.0, float("nan"), 2.0, 0.5, 0.25, 0.125, 0.0, 0.0, 0.0, 0.0, 0.0, 3.0, 2.0**-126, 3.3895314e38]
    kinds = set()
    for i, a in enumerate(seq):
        before = _bits(O.scale)
        L.scale_commit(getattr(qe, "CLASS_" + cls), torch.tensor([a], dtype=torch.float32, device=DEV))
        O.commit(np.float32(a))
        g = L.state()["classes"][cls]
        assert _bits(g["scale"]) == _bits(O.scale), (i, a, g["scale"], O.scale)
        assert _bits(g["scale_inv"]) == _bits(O.scale_inv), (i, a)
        assert np.array_equal(g["window"].view(np.uint32), O.window().view(np.uint32)), (i, a)
        assert g["count"] == O.count == i + 1
        if _bits(O.scale) == before:
            kinds.add("unchanged")
        if O.scale == np.finfo(np.float32).max:
            kinds.add("clamped")
            assert 0 < float(O.scale_inv) < 2.0**-126  # the inverse of the clamp is a subnormal, kept as such
    assert {"unchanged", "clamped"} <= kinds
    st = L.state()
    assert st["device_status"] == 0 and st["device_token"] == 0
    for other in "XWGY":
        if other != cls:
            assert st["classes"][other]["count"] == 0 and st["classes"][other]["scale"] == 1.0


@pytest.mark.parametrize("fmt_id,fmt", [(0, fp8.E4M3), (1, fp8.E5M2)])
def test_cast_of_a_tensor_holding_one_nan_and_the_commit_that_follows(qe, fmt_id, fmt):
    # One NaN among ordinary values: every other byte as the oracle casts it, the NaN's byte the format's NaN code
    # whatever its sign, the tensor's amax not finite -- and committing that amax leaves the scale where it was.
    from oracle.scaling import ScaleState, amax_bf16

    rows, cols = 256, 384
    x = inputs.normal_bf16((rows, cols), 1.0, "nan-cast", fmt_id)
    x[17, 101] = float("nan")
    scale = np.float32(37.25)
    q = torch.empty((rows, cols), dtype=torch.uint8, device=DEV)
    amax = torch.zeros(1, dtype=torch.float32, device=DEV)
    qe.qe_quantize(x.to(DEV), torch.tensor([scale], device=DEV), fmt_id, q, None, amax)
    got = q.cpu().numpy()
    want = fp8.quantize(bf16.decode(inputs.bits(x)), scale, fmt)
    assert want[17, 101] & 0x7F == fmt.nan_code
    assert np.array_equal(got & 0x7F, want & 0x7F) and np.array_equal(np.delete(got.reshape(-1), 17 * cols + 101), np.delete(want.reshape(-1), 17 * cols + 101))
    a = amax.cpu().numpy()[0]
    assert not np.isfinite(a) and not np.isfinite(amax_bf16(bf16.decode(inputs.bits(x))))
    cls = "X" if fmt_id == 0 else "G"
    ctx, L = _mk_layer(qe, 0, 256, 256, 256, 4, 0, 1)
    O = ScaleState(fmt, 4, 0)
    for v in (2.5, a, 0.75):  # an ordinary commit, the non-finite one, an ordinary one while the NaN is still in the window
        L.scale_commit(getattr(qe, "CLASS_" + cls), torch.tensor([v], dtype=torch.float32, device=DEV))
        O.commit(np.float32(v))
        g = L.state()["classes"][cls]
        assert _bits(g["scale"]) == _bits(O.scale) == _bits(np.float32(fmt.max_finite) / np.float32(2.5))
        assert _bits(g["scale_inv"]) == _bits(O.scale_inv)
        assert np.array_equal(g["window"].view(np.uint32) & 0x7FFFFFFF, O.window().view(np.uint32) & 0x7FFFFFFF)


def test_boundary_of_many_layers_in_one_call(qe):
    # 70 small layers of one context (more than one 64-entry gather launch): a step each, then ONE boundary call.
    # While one layer still lacks a microbatch the call fails and bumps NO layer; afterwards all move together.
    T = K = N = 256
    M, nl = 2, 70
    ctx = qe.Context(qe.EAGER)
    Ls = [qe.Layer(ctx, T, K, N, 4, 0, 2, inputs.weights("B", 0, u % 3, N, K).to(DEV), unit=u) for u in range(nl)]
    x = inputs.activations("B", 0, 0, 0, 0, T, K).to(DEV)
    dy = inputs.upstream_grads("B", 0, 0, 0, 0, T, N).to(DEV)
    y, dx = torch.empty((T, N), dtype=torch.bfloat16, device=DEV), torch.empty((T, K), dtype=torch.bfloat16, device=DEV)
    grad = torch.zeros(nl * N * K, device=DEV)
    held = None
    for u, L in enumerate(Ls):
        for m in range(M):
            t = L.forward(m, 0, x, y)
            L.backward_dI(t, dy, dx)
            if u == 67 and m == 1:
                held = t  # layer 67 keeps its last weight gradient back
            else:
                L.backward_dW(t, grad, u * N * K)
    with pytest.raises(qe.QEError) as e:
        qe.optimizer_boundary_all(Ls, M)
    assert e.value.code == "PENDING"
    assert all(L.state()["e_W"] == 0 for L in Ls)
    Ls[67].backward_dW(held, grad, 67 * N * K)
    with pytest.raises(qe.QEError) as e:
        qe.optimizer_boundary_all(Ls, M + 1)
    assert e.value.code == "INCOMPLETE" and all(L.state()["e_W"] == 0 for L in Ls)
    k0 = ctx.stats()["kernels_launched"]
    qe.optimizer_boundary_all(Ls, M)
    assert ctx.stats()["kernels_launched"] - k0 == 2  # two gather launches for 70 status words
    for L in Ls:
        s_ = L.state()
        assert s_["e_W"] == 1 and s_["write_mask"] == 0 and s_["fwd_in_epoch"] == 0 and s_["device_status"] == 0
    # the boundary touches no data: every layer saw the same X and dY, so every slice holds the same gradient
    g = grad.view(nl, N * K)
    assert torch.equal(g[0], g[67]) and torch.equal(g[1], g[69]) and torch.count_nonzero(g[0]).item() > 0
    other = qe.Context(qe.EAGER)
    alien = qe.Layer(other, T, K, N, 4, 0, 2, torch.zeros((N, K), dtype=torch.bfloat16, device=DEV))
    with pytest.raises(qe.QEError) as e:
        qe.optimizer_boundary_all([Ls[0], alien], M)
    assert e.value.code == "BAD_ARG"


def test_contract_violations_through_the_layer_leave_state_untouched(qe):
    T = K = N = 256
    ctx, L = _mk_layer(qe, 0, T, K, N, 4, 0, 2)
    L.weight.copy_(inputs.weights("E", 0, 0, N, K).to(DEV))
    x = inputs.activations("E", 0, 0, 0, 0, T, K).to(DEV)
    dy = inputs.upstream_grads("E", 0, 0, 0, 0, T, N).to(DEV)
    y, dx = torch.empty((T, N), dtype=torch.bfloat16, device=DEV), torch.empty((T, K), dtype=torch.bfloat16, device=DEV)
    buf = torch.zeros(N * K + 4, device=DEV)

    def expect(code, fn, *a):
        before = L.state()
        with pytest.raises(qe.QEError) as e:
            fn(*a)
        assert e.value.code == code, e.value
        after = L.state()
        assert state_equal(before, after) and before["device_token"] == after["device_token"]

    expect("EPOCH", L.forward, 0, 3, x, y)
    t0 = L.forward(0, 0, x, y)
    expect("KEY_LIVE", L.forward, 0, 0, x, y)
    expect("ORDER", L.backward_dW, t0, buf, 0)
    L.backward_dI(t0, dy, dx)
    expect("DUP_CONSUME", L.backward_dI, t0, dy, dx)
    expect("DEST", L.backward_dW, t0, buf, 2)
    expect("DEST", L.backward_dW, t0, buf, 8)
    L.backward_dW(t0, buf, 0)
    expect("STALE_REF", L.backward_dW, t0, buf, 0)
    t1 = L.forward(1, 0, x, y)
    assert (t1.ref.slot, t1.ref.gen) == (0, 2)
    expect("STALE_REF", L.backward_dI, t0, dy, dx)
    expect("PENDING", L.optimizer_boundary, 2)
    L.invalidate_cache()
    expect("STALE_CACHE", L.forward, 2, 0, x, y)
    L.abort_step()
    expect("ABORTED", L.backward_dI, t1, dy, dx)
    L.arena_rebuild()
    t = L.forward(0, 0, x, y)
    L.backward_dI(t, dy, dx)
    L.backward_dW(t, buf, 4)
    expect("INCOMPLETE", L.optimizer_boundary, 2)
    L.optimizer_boundary(1)
    assert L.state()["e_W"] == 1


def test_bad_configs_are_rejected(qe):
    ctx = qe.Context(0)
    w = torch.zeros((256, 256), dtype=torch.bfloat16, device=DEV)
    for T, K, N, code in [(200, 256, 256, "SHAPE"), (256, 0, 256, "SHAPE"), (256, 256, 128, "SHAPE")]:
        with pytest.raises(qe.QEError) as e:
            qe.Layer(ctx, T, K, N, 4, 0, 2, torch.zeros((N, max(K, 1)), dtype=torch.bfloat16, device=DEV)) if K else \
                qe.lib.qe_layer_workspace_bytes and qe._check(qe.lib.qe_layer_workspace_bytes(
                    __import__("ctypes").byref(qe.qe_layer_config(T=T, K=K, N=N, history_len=4, slots=2)),
                    __import__("ctypes").byref(__import__("ctypes").c_uint64())))
        assert e.value.code == code
    with pytest.raises(qe.QEError) as e:
        qe.Layer(ctx, 256, 256, 256, 0, 0, 2, w)
    assert e.value.code == "BAD_ARG"


@pytest.mark.parametrize("mode", [0, 1], ids=["eager", "graph"])
def test_resume_from_checkpoint_equals_uninterrupted_run(qe, mode):
    # save at step 3 into a fresh context and layer ("fresh process"), continue through step 8
    T, K, N, M, H = 256, 256, 384, 4, 4
    s = sched(M, 2, 1)
    P = peak_live(s)
    W = _weights("R", N, K, 8)
    get = lambda step, mb: c1_inputs(step, mb, T, K, N, "R")

    def run(L, buf, steps, first_epoch):
        L._e = first_epoch
        outs = {}
        for step in steps:
            o = run_gpu_steps(qe, L, s, 1, M, buf, 0, lambda _s, mb: get(step, mb), lambda _e: W[step])
            outs.update({(step,) + k[1:]: v for k, v in o.items()})
        return outs

    ctxA, A = _mk_layer(qe, mode, T, K, N, H, 0, P)
    bufA = torch.zeros(N * K, device=DEV)
    full = run(A, bufA, range(8), 0)

    ctxB, B = _mk_layer(qe, mode, T, K, N, H, 0, P)
    bufB = torch.zeros(N * K, device=DEV)
    run(B, bufB, range(3), 0)
    B.weight.copy_(inputs.from_bits(W[3]).to(DEV))
    x = inputs.from_bits(get(3, 0)[0]).to(DEV)
    y = torch.empty((T, N), dtype=torch.bfloat16, device=DEV)
    t = B.forward(0, 3, x, y)
    with pytest.raises(qe.QEError) as e:
        B.state_save()
    assert e.value.code == "PENDING"  # checkpoint withheld while a tape is live
    B.abort_step()
    B.arena_rebuild()
    # (the abandoned forward advanced the X and Y histories; save a clean boundary state from another run instead)
    ctxD, D = _mk_layer(qe, mode, T, K, N, H, 0, P)
    bufD = torch.zeros(N * K, device=DEV)
    run(D, bufD, range(3), 0)
    payload = D.state_save()
    assert len(payload) == 88 + 4 * H * 4  # persistent state only: a few hundred bytes here, ~16 KB at H = 1024
    del D, ctxD

    ctxE, E = _mk_layer(qe, mode, T, K, N, H, 0, P)
    E.state_load(payload)
    st = E.state()
    assert st["e_W"] == 3 and st["e_C"] == qe.QE_INVALID_EPOCH and st["token"] == 0
    bufE = torch.zeros(N * K, device=DEV)
    got = run(E, bufE, range(3, 8), 3)
    for k in got:
        assert np.array_equal(full[k].view(np.uint8), got[k].view(np.uint8)), k
    sa, se = A.state(), E.state()
    assert state_equal({**sa, "slots": [], "token": 0}, {**se, "slots": [], "token": 0})
    # wrong configuration is rejected
    ctxF, F = _mk_layer(qe, mode, T, K, N, H + 1, 0, P)
    with pytest.raises(qe.QEError):
        F.state_load(payload)


_RESUME_CHILD = r"""
import sys, numpy as np, torch
sys.path.insert(0, {root!r}); sys.path.insert(0, {root!r} + "/tests")
from harness import c1_inputs, run_gpu_steps
from paper_2609_23536_b200 import binding as qe, inputs
from paper_2609_23536_b200.schedules import peak_live, sched
T, K, N, M, H, mode = 256, 256, 384, 4, 4, {mode}
s = sched(M, 2, 1)
W = [inputs.weights("R", 0, 0, N, K)]
for e in range(1, 8):
    W.append(inputs.optimizer_perturbation(W[-1], "R", e, 0, 0))
ctx = qe.Context(mode)
L = qe.Layer(ctx, T, K, N, H, 0, peak_live(s), torch.zeros((N, K), dtype=torch.bfloat16, device="cuda:0"))
L.state_load(open({ckpt!r}, "rb").read())
assert L.state()["e_W"] == 3 and L.state()["token"] == 0
buf = torch.zeros(N * K, device="cuda:0")
out = {{}}
for step in range(3, 8):
    o = run_gpu_steps(qe, L, s, 1, M, buf, 0, lambda _s, mb: c1_inputs(step, mb, T, K, N, "R"), lambda _e: inputs.bits(W[step]))
    out.update({{"%d_%s_%s" % ((step,) + (k[1], k[2] if len(k) > 2 else "")): v for k, v in o.items()}})
st = L.state()
out["final_scales"] = np.array([st["classes"][c]["scale"] for c in "XWGY"], np.float32)
out["final_windows"] = np.stack([st["classes"][c]["window"] for c in "XWGY"])
np.savez({result!r}, **out)
"""


@pytest.mark.parametrize("mode", [0, 1], ids=["eager", "graph"])
def test_resume_in_a_fresh_process_equals_the_uninterrupted_run(qe, mode, tmp_path):
    # Sec. 5.2's restart check as the paper runs it: the persistent state saved at the boundary after step 3 goes to a
    # file; a NEW process (new CUDA context, new layer, new graphs, new tape generations) loads it and runs steps 4-8;
    # its outputs, gradients and final scaling state equal the uninterrupted run's bit for bit.
    import os
    import subprocess
    import sys

    T, K, N, M, H = 256, 256, 384, 4, 4
    s = sched(M, 2, 1)
    P = peak_live(s)
    W = _weights("R", N, K, 8)
    get = lambda step, mb: c1_inputs(step, mb, T, K, N, "R")
    ctx, A = _mk_layer(qe, mode, T, K, N, H, 0, P)
    buf = torch.zeros(N * K, device=DEV)
    full = {}
    for step in range(8):
        o = run_gpu_steps(qe, A, s, 1, M, buf, 0, lambda _s, mb: get(step, mb), lambda _e: W[step])
        full.update({"%d_%s_%s" % ((step,) + (k[1], k[2] if len(k) > 2 else "")): v for k, v in o.items()})
        if step == 2:
            ckpt = tmp_path / "state_after_step_3.bin"
            ckpt.write_bytes(A.state_save())
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    result = str(tmp_path / "resumed.npz")
    code = _RESUME_CHILD.format(root=root, mode=mode, ckpt=str(ckpt), result=result)
    r = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    got = np.load(result)
    keys = [k for k in got.files if not k.startswith("final")]
    assert len(keys) == 5 * (2 * M + 1)
    for k in keys:
        assert np.array_equal(full[k].view(np.uint8), got[k].view(np.uint8)), k
    st = A.state()
    assert np.array_equal(got["final_scales"].view(np.uint32), np.array([st["classes"][c]["scale"] for c in "XWGY"], np.float32).view(np.uint32))
    assert np.array_equal(got["final_windows"].view(np.uint32), np.stack([st["classes"][c]["window"] for c in "XWGY"]).view(np.uint32))


@pytest.mark.parametrize("mode", [0, 1], ids=["eager", "graph"])
def test_one_way_handoff_reads_stale_outputs_two_way_never_does(qe, mode):
    # Sec. 2.3: fixed producer/consumer pairs, 200 checks per protocol.  The producer is a forward on the context's
    # own stream; the consumer, on the caller's stream, copies Y right after the call returns.  With the one-way
    # handoff the copy runs before the forward has finished and sees the sentinel the buffer held; with the two-way
    # handshake it never does.  (A stale read is wrong data, not a fault.)
    T, K, N = 2048, 4096, 4096
    stale = {}
    for one_way in (True, False):
        ctx = qe.Context(mode, unsafe_one_way=one_way)
        w = inputs.weights("H", 0, 0, N, K).to(DEV)
        L = qe.Layer(ctx, T, K, N, 4, 0, 1, w)
        x = inputs.activations("H", 0, 0, 0, 0, T, K).to(DEV)
        dy = inputs.upstream_grads("H", 0, 0, 0, 0, T, N).to(DEV)
        y = torch.empty((T, N), dtype=torch.bfloat16, device=DEV)
        seen = torch.empty_like(y)
        dx = torch.empty((T, K), dtype=torch.bfloat16, device=DEV)
        buf = torch.zeros(N * K, device=DEV)
        caller = torch.cuda.Stream()
        n_stale = 0
        with torch.cuda.stream(caller):
            for i in range(200):
                y.fill_(-7.0)  # sentinel, on the caller's stream (the forward waits for it: caller -> exec edge)
                t = L.forward(0, i, x, y)
                seen.copy_(y)  # the consumer
                torch.cuda.synchronize()
                n_stale += int((seen == -7.0).any().item())
                assert not (y == -7.0).any().item()  # the producer itself always completes
                L.backward_dI(t, dy, dx)
                L.backward_dW(t, buf, 0)
                torch.cuda.synchronize()
                L.optimizer_boundary(1)
        stale[one_way] = n_stale
    assert stale[False] == 0
    assert stale[True] >= 190, stale


@pytest.mark.parametrize("mode", [0, 1], ids=["eager", "graph"])
def test_host_buffer_entry_points_equal_the_device_ones_bitwise(qe, mode):
    T, K, N, M = 256, 384, 512, 3
    s = sched(M, 2, 1)
    P = peak_live(s)
    w = inputs.weights("HB", 0, 0, N, K).to(DEV)
    res = []
    for host in (False, True):
        ctx = qe.Context(mode)
        L = qe.Layer(ctx, T, K, N, 4, 0, P, w.clone(), host_io=host)
        buf = torch.zeros(N * K, device=DEV)
        outs, tapes = {}, {}
        for a, m in s:
            X, dY = c1_inputs(0, m, T, K, N, "HB")
            if a == "F":
                x = inputs.from_bits(X)
                if host:
                    y = torch.empty((T, N), dtype=torch.bfloat16).pin_memory()
                    tapes[m] = L.forward_host(m, 0, x.pin_memory(), y)
                else:
                    y = torch.empty((T, N), dtype=torch.bfloat16, device=DEV)
                    tapes[m] = L.forward(m, 0, x.to(DEV), y)
                outs[("Y", m)] = y
            elif a == "dI":
                g = inputs.from_bits(dY)
                if host:
                    dx = torch.empty((T, K), dtype=torch.bfloat16).pin_memory()
                    L.backward_dI_host(tapes[m], g.pin_memory(), dx)
                else:
                    dx = torch.empty((T, K), dtype=torch.bfloat16, device=DEV)
                    L.backward_dI(tapes[m], g.to(DEV), dx)
                outs[("dX", m)] = dx
            else:
                L.backward_dW(tapes[m], buf, 0)
        torch.cuda.synchronize()
        L.optimizer_boundary(M)
        res.append(({k: inputs.bits(v.cpu()) for k, v in outs.items()}, buf.cpu().numpy(), L.state()))
    (oa, ga, sa), (ob, gb, sb) = res
    for k in oa:
        assert np.array_equal(oa[k], ob[k]), k
    assert np.array_equal(ga.view(np.uint32), gb.view(np.uint32))
    assert state_equal(sa, sb)
    # a layer created without staging refuses the host entry points
    ctx = qe.Context(mode)
    L = qe.Layer(ctx, T, K, N, 4, 0, P, w.clone())
    with pytest.raises(qe.QEError) as e:
        L.forward_host(0, 0, torch.zeros((T, K), dtype=torch.bfloat16), None)
    assert e.value.code == "BAD_ARG"


def test_limits_longest_history_most_slots_and_microbatches(qe):
    # H = 4096 (longest history), 64 slots and 64 microbatches (the write mask's width): all forwards first, then all
    # input-grads, then all weight-grads, against the oracle's state; a 65th microbatch index is rejected.
    T = K = N = 256
    M = 64
    ctx, L = _mk_layer(qe, 1, T, K, N, 4096, 2, 64)
    O = OracleLinear(T, K, N, 4096, 2, 64)
    w = inputs.weights("LIM", 0, 0, N, K)
    L.weight.copy_(w.to(DEV))
    O.set_weight(inputs.bits(w))
    buf = torch.zeros(N * K, device=DEV)
    obuf = np.zeros(N * K, np.float32)
    y = torch.empty((T, N), dtype=torch.bfloat16, device=DEV)
    dx = torch.empty((T, K), dtype=torch.bfloat16, device=DEV)
    gt, ot = {}, {}
    for m in range(M):
        X, _ = c1_inputs(0, m % 4, T, K, N, "LIM")
        gt[m] = L.forward(m, 0, inputs.from_bits(X).to(DEV), y)
        ot[m], _ = O.forward(m, 0, X, rows=[0])
        assert gt[m].astuple() == (tuple(ot[m].key), tuple(ot[m].ref))
    with pytest.raises(qe.QEError) as e:
        L.forward(64, 0, inputs.from_bits(X).to(DEV), y)
    assert e.value.code == "BAD_ARG"
    with pytest.raises(qe.QEError) as e:
        L.forward(0, 0, inputs.from_bits(X).to(DEV), y)
    assert e.value.code == "KEY_LIVE"
    for m in range(M):
        _, dY = c1_inputs(0, m % 4, T, K, N, "LIM")
        L.backward_dI(gt[m], inputs.from_bits(dY).to(DEV), dx)
        O.backward_dI(ot[m], dY, rows=[0])
    for m in range(M):
        L.backward_dW(gt[m], buf, 0)
        O.backward_dW(ot[m], obuf, 0)
    assert state_equal_except_Y(L.state(), O.state())
    assert assert_grad_close(buf.cpu().numpy(), obuf, "64 microbatches") < 1e-5
    L.optimizer_boundary(64)
    O.optimizer_boundary(64)
    assert L.state()["e_W"] == 1 and L.state()["write_mask"] == 0


# ------------------------------------------------------------------------------------------ per-microbatch arena
@pytest.mark.parametrize("mode", [0, 1], ids=["eager", "graph"])
@pytest.mark.parametrize("overlap", [False, True], ids=["inline", "overlapped"])
def test_arena_variant_against_oracle_and_flat_path(qe, mode, overlap):
    """One bf16 view per microbatch, summed at finalisation (the arena as the paper sizes it) against the oracle's
    arena functions; and against the flat accumulate, which it must stay close to (bf16 rounding per microbatch)."""
    T, K, N, M, H = 256, 256, 512, 4, 4
    s = sched(M, 2, 1)
    P = peak_live(s)
    W = _weights("AR", N, K, 2)
    get = lambda step, mb: c1_inputs(step, mb, T, K, N, "AR")
    n = N * K
    # oracle
    O = OracleLinear(T, K, N, H, 0, P)
    o_arena = np.zeros(8 + M * n, np.uint16)
    o_buf = np.zeros(4 + n, np.float32)
    # GPU
    ctx = qe.Context(mode, overlap_dw=overlap)
    L = qe.Layer(ctx, T, K, N, H, 0, P, inputs.from_bits(W[0]).to(DEV))
    arena = torch.full((8 + M * n,), float("nan"), dtype=torch.bfloat16, device=DEV)
    grad = torch.full((4 + n,), -1.0, device=DEV)
    flat = torch.zeros(n, device=DEV)
    ctx2 = qe.Context(mode)
    L2 = qe.Layer(ctx2, T, K, N, H, 0, P, inputs.from_bits(W[0]).to(DEV))
    for step in range(2):
        O.set_weight(W[step])
        for lay in (L, L2):
            lay.weight.copy_(inputs.from_bits(W[step]).to(DEV))
        tapes, otapes, tapes2 = {}, {}, {}
        for a, m in s:
            X, dY = get(step, m)
            x, dy = inputs.from_bits(X).to(DEV), inputs.from_bits(dY).to(DEV)
            if a == "F":
                otapes[m], _ = O.forward(m, O.e_W, X)
                tapes[m] = L.forward(m, step, x, torch.empty((T, N), dtype=torch.bfloat16, device=DEV))
                tapes2[m] = L2.forward(m, step, x, torch.empty((T, N), dtype=torch.bfloat16, device=DEV))
            elif a == "dI":
                O.backward_dI(otapes[m], dY)
                L.backward_dI(tapes[m], dy, torch.empty((T, K), dtype=torch.bfloat16, device=DEV))
                L2.backward_dI(tapes2[m], dy, torch.empty((T, K), dtype=torch.bfloat16, device=DEV))
            else:
                O.backward_dW_arena(otapes[m], o_arena, 8, M)
                L.backward_dW_arena(tapes[m], arena, 8, M)
                L2.backward_dW(tapes2[m], flat, 0)
        O.arena_finalize(o_arena, 8, M, o_buf, 4)
        L.arena_finalize(arena, 8, M, grad, 4)
        torch.cuda.synchronize()
        got_views = inputs.bits(arena.cpu())
        for m in range(M):
            assert_gemm_close(got_views[8 + m * n: 8 + (m + 1) * n].reshape(N, K), o_arena[8 + m * n: 8 + (m + 1) * n].reshape(N, K),
                              f"view step {step} mb {m}")
        assert np.all(np.isnan(bf16.decode(got_views[:8])))  # nothing before the region
        g = grad.cpu().numpy()
        assert np.all(g[:4] == -1.0)
        assert assert_grad_close(g[4:], o_buf[4:], f"finalised gradient step {step}") < 1e-3
        # the GPU's own views summed by the oracle's rule give the GPU's gradient bit for bit
        want = bf16.decode(got_views[8: 8 + n]).astype(np.float32)
        for m in range(1, M):
            want = (want + bf16.decode(got_views[8 + m * n: 8 + (m + 1) * n]).astype(np.float32)).astype(np.float32)
        assert np.array_equal(g[4:].view(np.uint32), want.view(np.uint32))
        L2.optimizer_boundary(M)
        # against the flat FP32 accumulate the views lose what bf16 rounding loses: up to 2^-9 relative per view
        f = flat.cpu().numpy().astype(np.float64)
        assert np.linalg.norm(g[4:] - f) / np.linalg.norm(f) < 2.0**-8
        O.optimizer_boundary(M)
        L.optimizer_boundary(M)
        assert state_equal_except_Y(L.state(), O.state())


def test_arena_variant_contract_errors(qe):
    T, K, N, M = 256, 256, 256, 2
    ctx, L = _mk_layer(qe, 0, T, K, N, 4, 0, 2)
    n = N * K
    arena = torch.zeros(M * n + 8, dtype=torch.bfloat16, device=DEV)
    grad = torch.zeros(n, device=DEV)
    x = torch.ones((T, K), dtype=torch.bfloat16, device=DEV)
    dy = torch.ones((T, N), dtype=torch.bfloat16, device=DEV)
    y, dx = torch.empty((T, N), dtype=torch.bfloat16, device=DEV), torch.empty((T, K), dtype=torch.bfloat16, device=DEV)
    t0, t1 = L.forward(0, 0, x, y), L.forward(1, 0, x, y)
    L.backward_dI(t0, dy, dx)
    L.backward_dI(t1, dy, dx)
    for args, code in (((t1, arena, 8, M), "ORDER"), ((t0, arena, 4, M), "DEST"), ((t0, arena[: n + 8], 8, M), "DEST"),
                       ((t0, arena, 8, 0), "BAD_ARG")):
        with pytest.raises(qe.QEError) as e:
            L.backward_dW_arena(*args)
        assert e.value.code == code
    L.backward_dW_arena(t0, arena, 8, M)
    with pytest.raises(qe.QEError) as e:
        L.arena_finalize(arena, 8, M, grad, 0)
    assert e.value.code == "INCOMPLETE"
    with pytest.raises(qe.QEError) as e:
        L.backward_dW_arena(t1, arena, 0, M)  # another region than the one bound this epoch
    assert e.value.code == "DEST"
    L.backward_dW_arena(t1, arena, 8, M)
    with pytest.raises(qe.QEError) as e:
        L.arena_finalize(arena, 0, M, grad, 0)
    assert e.value.code == "DEST"
    L.arena_finalize(arena, 8, M, grad, 0)
    torch.cuda.synchronize()
    L.optimizer_boundary(M)
    assert L.state()["e_W"] == 1
