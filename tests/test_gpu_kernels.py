"""GPU parity of the standalone kernels against the oracle (through the C-ABI)."""
import numpy as np
import pytest
import torch

from oracle import bf16, fp8
from oracle.layer import gemm_dI, gemm_dW, gemm_fwd
from oracle.scaling import amax_bf16
from paper_2609_23536_b200 import inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
FMT = {0: fp8.E4M3, 1: fp8.E5M2}


@pytest.fixture(scope="module")
def qe():
    from paper_2609_23536_b200 import build

    build.build()
    from paper_2609_23536_b200 import binding

    return binding


def _dev(bits_np):
    return inputs.from_bits(bits_np).to(DEV)


def _special_values(n):
    """bf16 patterns that exercise saturation, subnormals, ties, signed zero and infinities."""
    vals = [0.0, -0.0, 1.0, -1.0, 448.0, 464.0, -480.0, 57344.0, 61440.0, 1e30, -1e30, float("inf"), -float("inf"),
            2.0**-9, 2.0**-10, 1.5 * 2.0**-10, 2.0**-16, 2.0**-17, 1.0625, 1.1875, 1.125, 1.375, 2.0**-126, 2.0**-133]
    t = torch.tensor(vals, dtype=torch.float32).to(torch.bfloat16)
    return t.repeat((n + len(vals) - 1) // len(vals))[:n]


@pytest.mark.parametrize("rows,cols", [(64, 64), (320, 192), (2048, 1024), (4096 + 64, 2048 + 64)])
@pytest.mark.parametrize("fmt", [0, 1])
@pytest.mark.parametrize("scale", [1.0, 448.0 / 3.3, 2.0**-3, 3.1e4])
def test_quantize_bytes_transposed_copy_and_amax_bit_exact(qe, rows, cols, fmt, scale):
    if rows > 4096 and scale != 1.0:
        pytest.skip("large case once per format")
    x = inputs.normal_bf16((rows, cols), 1.0 if fmt == 0 else 1e-3, "q", rows, cols, fmt)
    x.view(-1)[: min(4096, x.numel())] = _special_values(min(4096, x.numel()))
    xb = inputs.bits(x)
    xd = x.to(DEV)
    s = torch.tensor([scale], dtype=torch.float32, device=DEV)
    q = torch.empty((rows, cols), dtype=torch.uint8, device=DEV)
    qT = torch.empty((cols, rows), dtype=torch.uint8, device=DEV)
    amax = torch.zeros(1, dtype=torch.float32, device=DEV)
    qe.qe_quantize(xd, s, fmt, q, qT, amax)
    torch.cuda.synchronize()
    want = fp8.quantize(bf16.decode(xb), np.float32(s.item()), FMT[fmt])
    got = q.cpu().numpy()
    assert np.array_equal(got, want), np.argwhere(got != want)[:5]
    assert np.array_equal(qT.cpu().numpy(), want.T)
    a = amax_bf16(bf16.decode(xb))
    assert amax.cpu().numpy().view(np.uint32)[0] == np.float32(a).view(np.uint32)
    # without the optional outputs
    q2 = torch.zeros_like(q)
    qe.qe_quantize(xd, s, fmt, q2)
    assert torch.equal(q2, q)


def test_quantize_rejects_bad_shapes(qe):
    x = torch.zeros((64, 96), dtype=torch.bfloat16, device=DEV)
    s = torch.ones(1, device=DEV)
    q = torch.empty((64, 96), dtype=torch.uint8, device=DEV)
    with pytest.raises(qe.QEError) as e:
        qe.qe_quantize(x, s, 0, q)
    assert e.value.code == "SHAPE"
    with pytest.raises(qe.QEError) as e:
        qe.qe_quantize(x[:, :64].contiguous(), s, 7, q)
    assert e.value.code == "BAD_ARG"


@pytest.mark.parametrize("n", [8, 8 * 1000 + 8, 1 << 20, (1 << 24) + 4096])
def test_standalone_amax(qe, n):
    x = inputs.normal_bf16((n,), 3.0, "amax", n)
    x[n // 3] = 1234.0
    x[-1] = -4321.0 if n > 8 else x[-1]
    xd = x.to(DEV)
    part = torch.full((qe.qe_amax_partials(),), 7e9, dtype=torch.float32, device=DEV)  # stale contents must not matter
    out = torch.zeros(1, dtype=torch.float32, device=DEV)
    for _ in range(2):
        qe.qe_amax(xd, part, out)
    assert out.item() == float(amax_bf16(bf16.decode(inputs.bits(x))))


@pytest.mark.parametrize("n", [4, 4 * 257, 1 << 22])
def test_accumulate(qe, n):
    a = torch.randn(n, device=DEV)
    b = torch.randn(n, device=DEV) * 1e-3
    d = a.clone()
    qe.qe_accumulate(d, b, True)
    assert torch.equal(d, a + b)  # one IEEE add per element
    qe.qe_accumulate(d, b, False)
    assert torch.equal(d, b)


# ------------------------------------------------------------------------------------------ GEMM
def _run_gemm(qe, A, afmt, B, bfmt, sa, sb, kind, init=None):
    M, Nn = A.shape[0], B.shape[0]
    Ad, Bd = torch.from_numpy(A).to(DEV), torch.from_numpy(B).to(DEV)
    sad = torch.tensor([sa], dtype=torch.float32, device=DEV)
    sbd = torch.tensor([sb], dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    amax = torch.zeros(1, dtype=torch.float32, device=DEV)
    if kind == 0:
        D = torch.empty((M, Nn), dtype=torch.bfloat16, device=DEV)
    else:
        D = init.clone().to(DEV) if init is not None else torch.full((M, Nn), float("nan"), device=DEV)
    qe.qe_gemm_fp8(Ad, afmt, Bd, bfmt, sad, sbd, D, kind, amax if kind == 0 else None, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    return D.cpu(), amax.item()


def _int_codes(rng, shape, lim, fmt):
    v = rng.integers(-lim, lim + 1, shape).astype(np.float32)
    q = fp8.encode(v, fmt)
    assert np.array_equal(fp8.decode(q, fmt), v)
    return q, v


@pytest.mark.parametrize("M,Nn,Kc", [(128, 256, 128), (256, 256, 256), (384, 384, 512), (128 * 5, 256 * 3, 4096), (128 * 30, 256 * 11, 256)])
def test_gemm_integer_inputs_are_bit_exact(qe, M, Nn, Kc):
    # every partial sum is an integer below 2^24: exact in FP32 in any order, so layout or descriptor
    # mistakes cannot hide behind a tolerance
    rng = np.random.default_rng(M + Nn + Kc)
    A, Av = _int_codes(rng, (M, Kc), 8, fp8.E4M3)
    B, Bv = _int_codes(rng, (Nn, Kc), 4, fp8.E4M3)
    want = Av.astype(np.float64) @ Bv.astype(np.float64).T
    assert np.abs(want).max() < 2**24
    D32, _ = _run_gemm(qe, A, 0, B, 0, 1.0, 1.0, 1)
    assert np.array_equal(D32.numpy(), want.astype(np.float32))
    Dbf, amax = _run_gemm(qe, A, 0, B, 0, 1.0, 1.0, 0)
    wb = bf16.round_from_f64(want)
    assert np.array_equal(inputs.bits(Dbf), wb)
    assert amax == float(np.abs(bf16.decode(wb)).max())
    init = torch.randint(-1000, 1000, (M, Nn)).float()
    Dacc, _ = _run_gemm(qe, A, 0, B, 0, 1.0, 1.0, 2, init)
    assert np.array_equal(Dacc.numpy(), init.numpy() + want.astype(np.float32))


def test_gemm_accumulate_keeps_subnormals(qe):
    # the in-place accumulate is a plain round-to-nearest FP32 addition like the oracle's: subnormal destination
    # values and subnormal addends are kept, not flushed to zero
    M, Nn, Kc = 256, 256, 128
    ones = np.full((M, Kc), 0x38, dtype=np.uint8)  # E4M3 1.0: every dot product is 128
    init = torch.full((M, Nn), 1e-40)
    init[0, 0], init[0, 1], init[0, 2] = -1e-40, 1.5, 2e-38
    tiny = 1e-21  # alpha = 1e-42 in FP32 (subnormal), D = 128 * alpha (subnormal)
    alpha = np.float32(np.float32(tiny) * np.float32(tiny))
    want = init.numpy() + np.float32(128.0) * alpha
    assert 0 < abs(want[1, 1]) < 1.2e-38
    got, _ = _run_gemm(qe, ones, 0, np.full((Nn, Kc), 0x38, dtype=np.uint8), 0, tiny, tiny, 2, init)
    assert np.array_equal(got.numpy().view(np.uint32), want.view(np.uint32))
    zero, _ = _run_gemm(qe, np.zeros((M, Kc), dtype=np.uint8), 0, np.zeros((Nn, Kc), dtype=np.uint8), 0, 1.0, 1.0, 2, init)
    assert np.array_equal(zero.numpy().view(np.uint32), init.numpy().view(np.uint32))


def test_gemm_permutation_weight_moves_columns(qe):
    rng = np.random.default_rng(1)
    M, K = 256, 512
    A, Av = _int_codes(rng, (M, K), 8, fp8.E4M3)
    perm = rng.permutation(K)
    Bv = np.zeros((K, K), np.float32)
    Bv[np.arange(K), perm] = 1.0
    B = fp8.encode(Bv, fp8.E4M3)
    D, _ = _run_gemm(qe, A, 0, B, 0, 1.0, 1.0, 1)
    assert np.array_equal(D.numpy(), Av[:, perm])


@pytest.mark.parametrize("afmt,bfmt", [(0, 0), (1, 0), (1, 1)])
@pytest.mark.parametrize("M,Nn,Kc", [(256, 256, 256), (512, 640, 1024), (2048, 2048, 2048)])
def test_gemm_random_bytes_within_tolerance(qe, afmt, bfmt, M, Nn, Kc):
    rng = np.random.default_rng(afmt * 7 + bfmt + M)
    A = fp8.quantize(rng.standard_normal((M, Kc)).astype(np.float32), np.float32(20.0), FMT[afmt])
    B = fp8.quantize(rng.standard_normal((Nn, Kc)).astype(np.float32), np.float32(20.0), FMT[bfmt])
    sa, sb = np.float32(1 / 20.0), np.float32(0.049)
    acc = fp8.decode(A, FMT[afmt]) @ fp8.decode(B, FMT[bfmt]).T * np.float64(sa) * np.float64(sb)
    D32, _ = _run_gemm(qe, A, afmt, B, bfmt, float(sa), float(sb), 1)
    rel = np.linalg.norm(D32.numpy().astype(np.float64) - acc) / np.linalg.norm(acc)
    assert rel < 1e-5, rel
    Dbf, amax = _run_gemm(qe, A, afmt, B, bfmt, float(sa), float(sb), 0)
    got = bf16.decode(inputs.bits(Dbf)).astype(np.float64)
    want = bf16.decode(bf16.round_from_f64(acc)).astype(np.float64)
    assert np.linalg.norm(got - acc) / np.linalg.norm(acc) < 1e-3 * 3
    floor = 2.0**-6 * np.sqrt(np.mean(acc**2))
    assert np.all(np.abs(got - want) <= 4 * bf16.ulp(np.maximum(np.abs(want), floor)))
    assert amax == float(np.abs(got).max())  # self-consistent with what was stored


@pytest.mark.parametrize("a_mn,b_mn", [(True, False), (False, True), (True, True)])
@pytest.mark.parametrize("M,Nn,Kc", [(256, 256, 128), (512, 768, 1024), (2048, 1280, 384)])
def test_gemm_mn_major_operands_integer_exact(qe, a_mn, b_mn, M, Nn, Kc):
    # the same product with operands handed over transposed ([Kc, M] / [Kc, Nn]): bit-exact on integer inputs
    rng = np.random.default_rng(M + Nn + Kc + 2 * a_mn + b_mn)
    A, Av = _int_codes(rng, (M, Kc), 8, fp8.E5M2)
    B, Bv = _int_codes(rng, (Nn, Kc), 4, fp8.E4M3)
    want = (Av.astype(np.float64) @ Bv.astype(np.float64).T).astype(np.float32)
    Ad = torch.from_numpy(np.ascontiguousarray(A.T) if a_mn else A).to(DEV)
    Bd = torch.from_numpy(np.ascontiguousarray(B.T) if b_mn else B).to(DEV)
    one = torch.ones(1, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    D = torch.full((M, Nn), float("nan"), device=DEV)
    qe.qe_gemm_fp8_ex(Ad, 1, a_mn, Bd, 0, b_mn, one, one, D, 1, None, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert np.array_equal(D.cpu().numpy(), want)


def test_gemm_mn_major_needs_the_paired_variant(qe):
    one = torch.ones(1, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    A = torch.zeros((128, 384), dtype=torch.uint8, device=DEV)  # [Kc, M] with M = 384
    B = torch.zeros((256, 128), dtype=torch.uint8, device=DEV)
    D = torch.zeros((384, 256), device=DEV)
    with pytest.raises(qe.QEError) as e:
        qe.qe_gemm_fp8_ex(A, 0, True, B, 0, False, one, one, D, 1, None, status)
    assert e.value.code == "UNSUPPORTED"


# ------------------------------------------------------------------------------------------ arena reduction
@pytest.mark.parametrize("M,n", [(1, 8), (2, 8 * 300), (5, 8 * 1031), (8, 1 << 20), (64, 8 * 512)])
def test_arena_reduce_adds_views_in_order(qe, M, n):
    g = torch.Generator().manual_seed(M * 1000 + n)
    views = (torch.randn((M, n), generator=g) * torch.logspace(-3, 3, M).unsqueeze(1)).to(torch.bfloat16)
    want = bf16.decode(inputs.bits(views[0])).astype(np.float32)
    for m in range(1, M):  # sequential FP32 additions, microbatch order (the oracle's arena_finalize)
        want = (want + bf16.decode(inputs.bits(views[m])).astype(np.float32)).astype(np.float32)
    dst = torch.full((n + 4,), 7.0, device=DEV)
    qe.qe_arena_reduce(views.to(DEV), M, dst[:n])
    torch.cuda.synchronize()
    assert np.array_equal(dst[:n].cpu().numpy().view(np.uint32), want.view(np.uint32))
    assert torch.all(dst[n:] == 7.0).item()


def test_arena_reduce_order_is_visible_in_the_result(qe):
    # (1 + 2^-24) + 2^-24 = 1 in FP32 while 2^-24 + 2^-24 + 1 = 1 + 2^-23
    one, tiny = torch.ones(8, dtype=torch.bfloat16), torch.full((8,), 2.0**-24, dtype=torch.bfloat16)
    dst = torch.zeros(8, device=DEV)
    qe.qe_arena_reduce(torch.stack([one, tiny, tiny]).to(DEV), 3, dst)
    assert torch.all(dst == 1.0).item()
    qe.qe_arena_reduce(torch.stack([tiny, tiny, one]).to(DEV), 3, dst)
    assert torch.all(dst == 1.0 + 2.0**-23).item()
    with pytest.raises(qe.QEError):
        qe.qe_arena_reduce(torch.zeros((2, 12), dtype=torch.bfloat16, device=DEV), 2, torch.zeros(12, device=DEV))


# ------------------------------------------------------------------------------------------ several problems per launch
def test_gemm_group_equals_single_launches_bitwise(qe):
    """Four different problems (formats, operand majors, epilogues, ragged N) in one launch against one launch each."""
    rng = np.random.default_rng(77)
    one = torch.ones(1, device=DEV)
    half = torch.full((1,), 0.5, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    specs = [  # (M, N, Kc, a_fmt, a_mn, b_mn, out_kind)
        (256, 640, 512, 0, 0, 0, 0),      # forward-like, bf16 + amax, N not a multiple of 256
        (512, 256, 1280, 1, 0, 1, 0),     # input-gradient-like: E5M2 x E4M3, MN-major B
        (768, 512, 256, 1, 1, 1, 2),      # weight-gradient-like: both MN-major, FP32 accumulate
        (256, 256, 128, 0, 0, 0, 1),      # FP32 overwrite, a single K block
    ]
    probs_single, probs_group, outs = [], [], []
    for M, N, Kc, af, amn, bmn, kind in specs:
        A = torch.from_numpy(rng.integers(0, 120, (Kc, M) if amn else (M, Kc), dtype=np.uint8)).to(DEV)
        B = torch.from_numpy(rng.integers(0, 120, (Kc, N) if bmn else (N, Kc), dtype=np.uint8)).to(DEV)
        init = torch.randn((M, N), device=DEV)
        d1 = init.to(torch.bfloat16) if kind == 0 else init.clone()
        d2 = d1.clone()
        am1, am2 = torch.zeros(1, device=DEV), torch.zeros(1, device=DEV)
        qe.qe_gemm_fp8_ex(A, af, bool(amn), B, 0, bool(bmn), one, half, d1, kind, am1 if kind == 0 else None, status)
        probs_group.append((A, af, amn, B, 0, bmn, one, half, d2, kind, am2 if kind == 0 else None))
        outs.append((d1, d2, am1, am2, kind))
    qe.qe_gemm_fp8_group(probs_group, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    for d1, d2, am1, am2, kind in outs:
        assert torch.equal(d1.view(torch.int16 if kind == 0 else torch.int32), d2.view(torch.int16 if kind == 0 else torch.int32))
        assert am1.item() == am2.item() and (kind != 0 or am1.item() > 0)
    with pytest.raises(qe.QEError) as e:  # a problem that needs the single-CTA variant cannot join
        A = torch.zeros((384, 128), dtype=torch.uint8, device=DEV)
        B = torch.zeros((256, 128), dtype=torch.uint8, device=DEV)
        d = torch.zeros((384, 256), device=DEV)
        qe.qe_gemm_fp8_group([probs_group[0], (A, 0, 0, B, 0, 0, one, one, d, 1, None)], status)
    assert e.value.code == "UNSUPPORTED"
    with pytest.raises(qe.QEError):
        qe.qe_gemm_fp8_group(probs_group[:1], status)


def test_gemm_group_of_eight(qe):
    """The largest group: eight small problems in one launch against eight single launches."""
    rng = np.random.default_rng(8)
    one = torch.ones(1, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    probs, outs = [], []
    for i in range(8):
        M, N, Kc = 256 * (1 + i % 3), 256 + 128 * (i % 4), 128 * (1 + i % 5)
        kind = i % 3
        A = torch.from_numpy(rng.integers(0, 120, (M, Kc), dtype=np.uint8)).to(DEV)
        B = torch.from_numpy(rng.integers(0, 120, (N, Kc), dtype=np.uint8)).to(DEV)
        init = torch.randn((M, N), device=DEV)
        d1 = init.to(torch.bfloat16) if kind == 0 else init.clone()
        d2 = d1.clone()
        qe.qe_gemm_fp8_ex(A, 0, False, B, i % 2, False, one, one, d1, kind, None, status)
        probs.append((A, 0, 0, B, i % 2, 0, one, one, d2, kind, None))
        outs.append((d1, d2, kind))
    qe.qe_gemm_fp8_group(probs, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    for d1, d2, kind in outs:
        assert torch.equal(d1.view(torch.int16 if kind == 0 else torch.int32), d2.view(torch.int16 if kind == 0 else torch.int32))
    with pytest.raises(qe.QEError):
        qe.qe_gemm_fp8_group(probs + probs[:1], status)
