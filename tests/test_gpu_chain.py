"""FP8 hand-off between directly chained linears (qe_forward_chain / qe_backward_dI_chain): bit for bit the result of
running the layers one by one through bf16 tensors, and within tolerance of the oracle's composition."""
import numpy as np
import pytest
import torch

from harness import assert_gemm_close, assert_grad_close, dW_abs_products, state_equal, state_equal_except_Y
from oracle import bf16
from oracle.layer import OracleLinear
from paper_2609_23536_b200 import inputs
from paper_2609_23536_b200.schedules import peak_live, sched

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
T = 256
CHAIN = [(256, 512), (512, 256), (256, 768)]  # (K, N): each layer consumes the one before


@pytest.fixture(scope="module")
def qe():
    from paper_2609_23536_b200 import build

    build.build()
    from paper_2609_23536_b200 import binding

    return binding


def _layers(qe, mode, P, overlap=False):
    ctx = qe.Context(mode, overlap_dw=overlap)
    return ctx, [qe.Layer(ctx, T, K, N, 4, 0, P, inputs.weights("CN", 0, j, N, K).to(DEV), unit=j) for j, (K, N) in enumerate(CHAIN)]


def _run(qe, mode, chained, steps=2, M=3, overlap=False):
    s = sched(M, 2, 1)
    ctx, layers = _layers(qe, mode, peak_live(s), overlap)
    n = len(layers)
    offs, total = inputs.grad_offsets([("l", K, N) for K, N in CHAIN])
    grad = torch.full((total,), 3.0, device=DEV)
    rec = {"Y": [], "dX": [], "Xq": [], "Gq": [], "mg": [], "state": [], "Yall": [], "dXall": [], "state_F": [], "state_dI": []}
    for step in range(steps):
        tapes = {}
        for a, m in s:
            if a == "F":
                x = inputs.activations("CN", step, 0, 0, m, T, CHAIN[0][0]).to(DEV)
                y = torch.empty((T, CHAIN[-1][1]), dtype=torch.bfloat16, device=DEV)
                if chained:
                    tapes[m] = qe.forward_chain(layers, m, step, x, y)
                else:
                    tapes[m], cur, outs = [], x, []
                    for j, L in enumerate(layers):
                        out = y if j == n - 1 else torch.empty((T, CHAIN[j][1]), dtype=torch.bfloat16, device=DEV)
                        tapes[m].append(L.forward(m, step, cur, out))
                        cur = out
                        outs.append(out)
                    rec["Yall"].append([inputs.bits(o.cpu()) for o in outs])  # every layer's bf16 output
                torch.cuda.synchronize()
                rec["state_F"].append([L.state() for L in layers])
                rec["Y"].append(inputs.bits(y.cpu()))
                rec["Xq"].append([L.read_fp8(0, tapes[m][j].ref.slot).copy() for j, L in enumerate(layers)])
            elif a == "dI":
                dy = inputs.upstream_grads("CN", step, 0, n - 1, m, T, CHAIN[-1][1]).to(DEV)
                dx = torch.empty((T, CHAIN[0][0]), dtype=torch.bfloat16, device=DEV)
                if chained:
                    qe.backward_dI_chain(layers, tapes[m], dy, dx)
                else:
                    cur, outs = dy, [None] * n
                    for j in range(n - 1, -1, -1):
                        out = dx if j == 0 else torch.empty((T, CHAIN[j][0]), dtype=torch.bfloat16, device=DEV)
                        layers[j].backward_dI(tapes[m][j], cur, out)
                        cur = out
                        outs[j] = out
                    rec["dXall"].append([inputs.bits(o.cpu()) for o in outs])  # every layer's bf16 input gradient
                torch.cuda.synchronize()
                rec["state_dI"].append([L.state() for L in layers])
                rec["dX"].append(inputs.bits(dx.cpu()))
                rec["Gq"].append([L.read_fp8(2, tapes[m][j].ref.slot).copy() for j, L in enumerate(layers)])
            else:
                qe.backward_dW_multi(layers, tapes[m], grad, offs)
        for L in layers:
            L.optimizer_boundary(M)
        torch.cuda.synchronize()
        rec["mg"].append(grad.cpu().numpy().copy())
        rec["state"].append([L.state() for L in layers])
    rec["stats"] = ctx.stats()
    return rec


@pytest.mark.parametrize("mode", [0, 1], ids=["eager", "graph"])
@pytest.mark.parametrize("overlap", [False, True], ids=["inline", "overlapped-dW"])
def test_chained_equals_layer_by_layer_bitwise(qe, mode, overlap):
    a = _run(qe, mode, chained=False, overlap=overlap)
    b = _run(qe, mode, chained=True, overlap=overlap)
    for key in ("Y", "dX", "mg"):
        for u, v in zip(a[key], b[key]):
            assert np.array_equal(u.view(np.uint8), v.view(np.uint8)), key
    for key in ("Xq", "Gq"):  # the deposited FP8 tensors are the bytes the consumer's own cast would have written
        for u, v in zip(a[key], b[key]):
            for x, y in zip(u, v):
                assert np.array_equal(x, y), key
    for u, v in zip(a["state"], b["state"]):
        for x, y in zip(u, v):
            assert state_equal(x, y) and x["device_token"] == y["device_token"]
    # two cast kernels per microbatch and direction are gone
    steps, M, n = 2, 3, len(CHAIN)
    assert a["stats"]["kernels_launched"] - b["stats"]["kernels_launched"] == steps * M * 2 * (n - 1)


def test_chain_against_the_oracle_composition(qe):
    M, steps = 3, 2
    s = sched(M, 2, 1)
    got = _run(qe, 0, chained=True, steps=steps, M=M)
    orc = [OracleLinear(T, K, N, 4, 0, peak_live(s), unit=j) for j, (K, N) in enumerate(CHAIN)]
    for j, (K, N) in enumerate(CHAIN):
        orc[j].set_weight(inputs.bits(inputs.weights("CN", 0, j, N, K)))
    offs, total = inputs.grad_offsets([("l", K, N) for K, N in CHAIN])
    buf = np.full(total, 3.0, np.float32)
    n = len(CHAIN)
    iy = idx = 0

    def rel(g, w):
        g, w = g.astype(np.float64), w.astype(np.float64)
        return np.linalg.norm(g - w) / np.linalg.norm(w)

    for step in range(steps):
        tapes = {}
        for a, m in s:
            if a == "F":
                cur = inputs.bits(inputs.activations("CN", step, 0, 0, m, T, CHAIN[0][0]))
                tapes[m] = []
                for L in orc:
                    t, cur = L.forward(m, L.e_W, cur)
                    tapes[m].append(t)
                # a one-ulp difference in an intermediate bf16 value can move an FP8 code of the next layer's input by
                # a whole step (2^-3 relative) on isolated elements, so the end-to-end bound is looser than one GEMM's
                assert rel(bf16.decode(got["Y"][iy]), bf16.decode(cur)) < 5e-3
                assert np.array_equal(got["Xq"][iy][0], orc[0].slots[tapes[m][0].ref.slot].Xq)  # first layer: seeded input
                iy += 1
            elif a == "dI":
                cur = inputs.bits(inputs.upstream_grads("CN", step, 0, n - 1, m, T, CHAIN[-1][1]))
                for j in range(n - 1, -1, -1):
                    if j == n - 1:
                        pass
                    cur = orc[j].backward_dI(tapes[m][j], cur)
                assert rel(bf16.decode(got["dX"][idx]), bf16.decode(cur)) < 5e-3
                assert np.array_equal(got["Gq"][idx][n - 1], orc[n - 1].slots[tapes[m][n - 1].ref.slot].Gq)
                idx += 1
            else:
                for j, L in enumerate(orc):
                    L.backward_dW(tapes[m][j], buf, offs[j])
        for L in orc:
            L.optimizer_boundary(M)
        assert rel(got["mg"][step], buf) < 5e-3
    # class-(i) state of the classes fed by seeded tensors only: first layer's X, every layer's W, last layer's G
    for j, L in enumerate(orc):
        gs, os_ = got["state"][-1][j], L.state()
        for c in (["W"] + (["X"] if j == 0 else []) + (["G"] if j == n - 1 else [])):
            assert np.array_equal(gs["classes"][c]["window"].view(np.uint32), os_["classes"][c]["window"].view(np.uint32)), (j, c)
            assert np.float32(gs["classes"][c]["scale"]).view(np.uint32) == np.float32(os_["classes"][c]["scale"]).view(np.uint32)
        assert gs["token"] == os_["token"] and gs["e_W"] == os_["e_W"] and gs["slots"] == os_["slots"]


@pytest.mark.parametrize("mode", [0, 1], ids=["eager", "graph"])
def test_chain_layer_by_layer_against_a_teacher_forced_oracle(qe, mode):
    """Every layer of the chain against the oracle at the single-GEMM tolerance.  The free-running comparison above
    lets a one-ulp difference in an interior bf16 value move an FP8 code downstream, so it cannot be tight.  Here the
    oracle layer j+1 is fed the bf16 tensor the GPU's layer j produced (taken from the layer-by-layer run, which the
    chained run equals bit for bit): what the hand-off deposits in the consumer -- FP8 bytes, amax, inverse-scale
    snapshot, the consumer's X / G scale state -- is then fixed exactly by the delayed-scaling recipe (Sec. 2.1) and
    must match bit for bit, and each GEMM output must lie within 1e-3 (Frobenius) and 4 bf16 ulp of the oracle's."""
    M, steps = 3, 2
    s = sched(M, 2, 1)
    P = peak_live(s)
    plain = _run(qe, mode, chained=False, steps=steps, M=M)
    chain = _run(qe, mode, chained=True, steps=steps, M=M)
    n = len(CHAIN)
    orc = [OracleLinear(T, K, N, 4, 0, P, unit=j) for j, (K, N) in enumerate(CHAIN)]
    for j, (K, N) in enumerate(CHAIN):
        orc[j].set_weight(inputs.bits(inputs.weights("CN", 0, j, N, K)))
    offs, total = inputs.grad_offsets([("l", K, N) for K, N in CHAIN])
    buf = np.full(total, 3.0, np.float32)
    iy = idx = 0
    for step in range(steps):
        tapes, absp = {}, [0.0] * n
        for a, m in s:
            if a == "F":
                tapes[m] = []
                for j, L in enumerate(orc):
                    x = inputs.bits(inputs.activations("CN", step, 0, 0, m, T, CHAIN[0][0])) if j == 0 else plain["Yall"][iy][j - 1]
                    t, y = L.forward(m, L.e_W, x)
                    tapes[m].append(t)
                    assert_gemm_close(plain["Yall"][iy][j], y, ("Y", step, m, j))
                    slot = L.slots[t.ref.slot]
                    assert np.array_equal(chain["Xq"][iy][j], slot.Xq), ("deposited Xq", step, m, j)
                    g = chain["state_F"][iy][j]
                    assert state_equal_except_Y(g, L.state()), ("state after F", step, m, j)
                    assert g["slot_sinv_X"][t.ref.slot].view(np.uint32) == np.float32(slot.sinv_X).view(np.uint32)
                    # the consumer's newest X amax is the magnitude of the bf16 tensor it was handed
                    assert g["classes"]["X"]["window"][0] == np.abs(bf16.decode(x)).max()
                iy += 1
            elif a == "dI":
                for j in range(n - 1, -1, -1):
                    dy = inputs.bits(inputs.upstream_grads("CN", step, 0, n - 1, m, T, CHAIN[-1][1])) if j == n - 1 else plain["dXall"][idx][j + 1]
                    dx = orc[j].backward_dI(tapes[m][j], dy)
                    assert_gemm_close(plain["dXall"][idx][j], dx, ("dX", step, m, j))
                    slot = orc[j].slots[tapes[m][j].ref.slot]
                    assert np.array_equal(chain["Gq"][idx][j], slot.Gq), ("deposited Gq", step, m, j)
                    g = chain["state_dI"][idx][j]
                    assert state_equal_except_Y(g, orc[j].state()), ("state after dI", step, m, j)
                    assert g["slot_sinv_G"][tapes[m][j].ref.slot].view(np.uint32) == np.float32(slot.sinv_G).view(np.uint32)
                    assert g["classes"]["G"]["window"][0] == np.abs(bf16.decode(dy)).max()
                idx += 1
            else:
                for j, L in enumerate(orc):
                    if m == 0:
                        absp[j] = 0.0
                    absp[j] = absp[j] + dW_abs_products(L.slots[tapes[m][j].ref.slot], np.arange(L.N))
                    L.backward_dW(tapes[m][j], buf, offs[j])
        for L in orc:
            L.optimizer_boundary(M)
        # the gradients: the oracle's tapes hold the same FP8 bytes and snapshots as the GPU's, so this is one GEMM's error
        for j, (K, N) in enumerate(CHAIN):
            assert_grad_close(chain["mg"][step][offs[j]: offs[j] + N * K], buf[offs[j]: offs[j] + N * K], ("mg", step, j),
                              abs_products=absp[j].reshape(-1), rel_tol=1e-5, contraction=T)
        for j, L in enumerate(orc):
            assert state_equal_except_Y(chain["state"][step][j], L.state()), ("state after the boundary", step, j)


def test_chain_argument_checks(qe):
    ctx, layers = _layers(qe, 0, 2)
    x = torch.zeros((T, 256), dtype=torch.bfloat16, device=DEV)
    y = torch.zeros((T, 768), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(qe.QEError) as e:
        qe.forward_chain([layers[0], layers[2]], 0, 0, x, y)  # 512 outputs into a 256-input layer
    assert e.value.code == "SHAPE"
    with pytest.raises(qe.QEError) as e:
        qe.forward_chain([layers[0], layers[0]], 0, 0, x, y)
    assert e.value.code == "BAD_ARG"
    odd = qe.Layer(ctx, T, 768, 384, 4, 0, 2, inputs.weights("CN", 0, 9, 384, 768).to(DEV), unit=9)  # N = 384 keeps transposed copies
    tail = qe.Layer(ctx, T, 384, 256, 4, 0, 2, inputs.weights("CN", 0, 10, 256, 384).to(DEV), unit=10)
    with pytest.raises(qe.QEError) as e:
        qe.forward_chain(layers + [odd, tail], 0, 0, x, torch.zeros((T, 256), dtype=torch.bfloat16, device=DEV))
    assert e.value.code == "UNSUPPORTED"
    before = [L.state() for L in layers]
    tapes = qe.forward_chain(layers, 0, 0, x, y)
    with pytest.raises(qe.QEError) as e:
        qe.forward_chain(layers, 0, 0, x, y)  # key live in every layer: nothing ran
    assert e.value.code == "KEY_LIVE"
    assert all(L.state()["token"] == b["token"] + 1 for L, b in zip(layers, before))
    dy, dx = torch.zeros((T, 768), dtype=torch.bfloat16, device=DEV), torch.zeros((T, 256), dtype=torch.bfloat16, device=DEV)
    qe.backward_dI_chain(layers, tapes, dy, dx)
    with pytest.raises(qe.QEError) as e:
        qe.backward_dI_chain(layers, tapes, dy, dx)
    assert e.value.code == "DUP_CONSUME"
