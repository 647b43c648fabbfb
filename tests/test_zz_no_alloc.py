"""The allocation-free copied-gradient entry point against the ordinary one (collected last on purpose).

qe_gemm_fp8_staged_noalloc exists for callers that cannot allocate device memory where they run (inside
another framework's allocator lock, in a no-allocation callback, in a process whose memory was handed
out at start-up); its scratch is an array built into the library.  It must give exactly what the
existing pair qe_gemm_fp8 (FP32 output into caller scratch) + qe_accumulate gives, on consecutive calls
that reuse the shared scratch."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def qe():
    from paper_2609_23536_b200 import build

    build.build()
    from paper_2609_23536_b200 import binding

    return binding


def _operands(seed, M, Nn, Kc):
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    # byte patterns below 0x78: finite in both FP8 formats
    A = torch.randint(0, 0x78, (M, Kc), generator=g, dtype=torch.uint8)
    B = torch.randint(0, 0x78, (Nn, Kc), generator=g, dtype=torch.uint8)
    sign = torch.randint(0, 2, (M, Kc), generator=g, dtype=torch.uint8) * 0x80
    return (A | sign).to(DEV), B.to(DEV)


def test_noalloc_matches_existing_entry_points_on_two_calls_in_a_row(qe):
    assert qe.qe_noalloc_staging_elems() == 1 << 20
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    sa = torch.tensor([2.0**-9], device=DEV)
    sb = torch.tensor([3.0 * 2.0**-11], device=DEV)
    # first call fills a large part of the staging area; the second, smaller, accumulating call must not see it
    calls = [(1024, 1024, 512, False, 1, 0), (256, 768, 256, True, 1, 0), (256, 768, 256, True, 0, 0)]
    dst_new = {}
    dst_old = {}
    for i, (M, Nn, Kc, acc, afmt, bfmt) in enumerate(calls):
        A, B = _operands(100 + i, M, Nn, Kc)
        key = (M, Nn)
        if key not in dst_new:
            init = torch.randn((M, Nn), generator=torch.Generator().manual_seed(7)).to(DEV)
            dst_new[key], dst_old[key] = init.clone(), init.clone()
        if i > 0:  # past the first (warm-up) call on this device: a call must leave the device's free memory as it was
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
        qe.qe_gemm_fp8_staged_noalloc(A, afmt, B, bfmt, sa, sb, dst_new[key], acc, status)
        if i > 0:
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free_before, i
        temp = torch.full((M, Nn), float("nan"), device=DEV)
        qe.qe_gemm_fp8(A, afmt, B, bfmt, sa, sb, temp, 1, None, status)
        qe.qe_accumulate(dst_old[key], temp, acc)
        torch.cuda.synchronize()
        # same kernels, same arithmetic order: identical bits (the suite's GEMM tolerance is trivially met)
        assert torch.equal(dst_new[key], dst_old[key]), i
        assert torch.isfinite(dst_new[key]).all()
    assert status.item() == 0


def test_noalloc_against_the_oracle(qe):
    # the largest case the staging area holds, against the plain definition: exact products of the decoded FP8 values
    # times the two factors, rounded once to FP32, then one FP32 addition to what the destination held
    from oracle import fp8

    M, Nn, Kc = 1024, 1024, 512
    A, B = _operands(300, M, Nn, Kc)
    sa, sb = np.float32(2.0**-9), np.float32(3.0 * 2.0**-11)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    init = torch.randn((M, Nn), generator=torch.Generator().manual_seed(9))
    dst = init.clone().to(DEV)
    qe.qe_gemm_fp8_staged_noalloc(A, 1, B, 0, torch.tensor([sa], device=DEV), torch.tensor([sb], device=DEV), dst, True, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    a, b = fp8.decode(A.cpu().numpy(), fp8.E5M2), fp8.decode(B.cpu().numpy(), fp8.E4M3)
    D = ((a @ b.T) * np.float64(sa) * np.float64(sb)).astype(np.float32)
    want = (init.numpy() + D).astype(np.float32)
    got = dst.cpu().numpy()
    # the suite's FP32 bound: errors scale with the sum of the absolute products (plus the old value, for the addition);
    # these operands are random FP8 bit patterns, i.e. magnitudes spread over 30 binades, where a few huge products
    # dominate a sum -- the case the two-level rule of assert_grad_close is written for
    from harness import assert_grad_close

    absp = (np.abs(a) @ np.abs(b).T) * float(sa) * float(sb) + np.abs(init.numpy())
    assert assert_grad_close(got, want, "allocation-free copy-add against the oracle", abs_products=absp, rel_tol=1e-6, contraction=Kc) < 1e-6


def test_noalloc_rejects_sizes_beyond_its_staging_area(qe):
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    one = torch.ones(1, device=DEV)
    A = torch.zeros((1024, 128), dtype=torch.uint8, device=DEV)
    B = torch.zeros((1280, 128), dtype=torch.uint8, device=DEV)
    dst = torch.zeros((1024, 1280), device=DEV)
    with pytest.raises(qe.QEError) as e:
        qe.qe_gemm_fp8_staged_noalloc(A, 0, B, 0, one, one, dst, False, status)
    assert e.value.code == "UNSUPPORTED" and "staging" in str(e.value)
    assert torch.count_nonzero(dst).item() == 0
