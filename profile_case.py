"""Small single-kernel cases for profiling (ncu) and quick timing.

    python profile_case.py gemm_f|gemm_di|gemm_dw|gemm_microbatch|gemm_microbatch_grouped|gemm_step|quantize|quantize_t|amax|accumulate [--reps N]

Each case holds well under 2 GB on the device, uses operands larger than the 126 MB L2 where DRAM traffic is
the question, does 2 warm-up launches and then `reps` launches, and prints the CUDA-event time per launch.
"""
from __future__ import annotations

import argparse
import json

import torch

import os
import sys

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))

from paper_2609_23536_b200 import build  # noqa: E402

build.build()
from paper_2609_23536_b200 import binding as qe  # noqa: E402


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("case")
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--small", action="store_true", help="Llama-block (hidden 2048) shapes instead of Llama-3-8B ones")
    a = ap.parse_args()
    dev = torch.device("cuda", 0)
    one = torch.ones(1, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    T, H, F = (2048, 2048, 11264) if a.small else (4096, 4096, 28672)
    work = None
    if a.case == "gemm_step":
        # the GEMM launches of one optimizer step as the default issue plan groups them (config 2 with --small)
        from paper_2609_23536_b200 import inputs, step_gemms

        launches, flops, nbytes = step_gemms.build(inputs.CONFIGS["C2" if a.small else "C3"], dev)
        fn = lambda: step_gemms.run(qe, launches, status)
        work = {"flop": flops, "bytes": nbytes, "launches": len(launches)}
    elif a.case == "gemm_microbatch_grouped":
        # the same twelve GEMMs in the five launches of the layer's steady state: F of linear i with dI of linear
        # 3-i (four launches), then the four weight gradients in one launch
        lin = ((H, 6144), (H, H), (H, F), (F // 2, H))

        def prob(M, N, Kc, af, kind, amn, bmn):
            return (torch.randint(0, 120, (Kc, M) if amn else (M, Kc), dtype=torch.uint8, device=dev), af, amn,
                    torch.randint(0, 120, (Kc, N) if bmn else (N, Kc), dtype=torch.uint8, device=dev), 0, bmn, one, one,
                    torch.zeros((M, N), dtype=torch.bfloat16 if kind == 0 else torch.float32, device=dev), kind, None)

        launches = []
        for i in range(4):
            (Ki, Ni), (Kj, Nj) = lin[i], lin[3 - i]
            launches.append([prob(T, Ni, Ki, 0, 0, 0, 0), prob(T, Kj, Nj, 1, 0, 0, 1)])
        launches.append([prob(N, K, T, 1, 2, 1, 1) for K, N in lin])

        def fn():
            for ps in launches:
                qe.qe_gemm_fp8_group(ps, status)

        work = {"flop": sum(6.0 * T * K * N for K, N in lin),
                "bytes": sum(T * K + N * K + 2 * T * N + T * N + N * K + 2 * T * K + T * N + T * K + 8 * N * K for K, N in lin)}
    elif a.case == "gemm_microbatch":
        # the twelve GEMMs (F, dI, dW of four linears) one microbatch of the Llama-style block launches, in order
        shapes = []
        # operand majors as the layer uses them: F both contraction-major; dI takes Wq [N,K] as an MN-major B;
        # dW takes Gq [T,N] and Xq [T,K] as MN-major A and B
        for K, N in ((H, 6144), (H, H), (H, F), (F // 2, H)):
            shapes += [(T, N, K, 0, 0, 0, 0), (T, K, N, 1, 0, 0, 1), (N, K, T, 1, 2, 1, 1)]
        ops = []
        for M, N, Kc, af, kind, amn, bmn in shapes:
            ops.append((torch.randint(0, 120, (Kc, M) if amn else (M, Kc), dtype=torch.uint8, device=dev),
                        torch.randint(0, 120, (Kc, N) if bmn else (N, Kc), dtype=torch.uint8, device=dev),
                        torch.zeros((M, N), dtype=torch.bfloat16 if kind == 0 else torch.float32, device=dev), af, kind, amn, bmn))

        def fn():
            for A, B, D, af, kind, amn, bmn in ops:
                qe.qe_gemm_fp8_ex(A, af, bool(amn), B, 0, bool(bmn), one, one, D, kind, None, status)

        work = {"flop": sum(2.0 * M * N * Kc for M, N, Kc, *_ in shapes),
                "bytes": sum(M * Kc + N * Kc + M * N * (2 if k == 0 else 8) for M, N, Kc, _, k, _, _ in shapes)}
    elif a.case.startswith("gemm"):
        # gate/up projection: F: [T,H]x[F,H]^T ; dI: [T,F]x[H,F]^T ; dW: [F,T]x[H,T]^T (FP32 accumulate)
        M, N, Kc, af, kind, amn, bmn = {"gemm_f": (T, F, H, 0, 0, 0, 0), "gemm_di": (T, H, F, 1, 0, 0, 1),
                                        "gemm_dw": (F, H, T, 1, 2, 1, 1)}[a.case]
        A = torch.randint(0, 120, (Kc, M) if amn else (M, Kc), dtype=torch.uint8, device=dev)
        B = torch.randint(0, 120, (Kc, N) if bmn else (N, Kc), dtype=torch.uint8, device=dev)
        D = torch.zeros((M, N), dtype=torch.bfloat16 if kind == 0 else torch.float32, device=dev)
        fn = lambda: qe.qe_gemm_fp8_ex(A, af, bool(amn), B, 0, bool(bmn), one, one, D, kind, None, status)
        work = {"flop": 2.0 * M * N * Kc, "bytes": M * Kc + N * Kc + M * N * (2 if kind == 0 else 8)}
    else:
        rows, cols = 8192, 16384
        x = torch.randn((rows, cols), device=dev).to(torch.bfloat16)
        n = rows * cols
        if a.case in ("quantize", "quantize_t"):
            q = torch.empty((rows, cols), dtype=torch.uint8, device=dev)
            qT = torch.empty((cols, rows), dtype=torch.uint8, device=dev) if a.case == "quantize_t" else None
            amax = torch.zeros(1, device=dev)
            fn = lambda: qe.qe_quantize(x, one, 0, q, qT, amax)
            work = {"bytes": n * (4 if qT is not None else 3)}
        elif a.case == "amax":
            part = torch.empty(qe.qe_amax_partials(), device=dev)
            out = torch.zeros(1, device=dev)
            fn = lambda: qe.qe_amax(x, part, out)
            work = {"bytes": 2 * n}
        elif a.case == "accumulate":
            g = torch.zeros(n // 2, device=dev)
            t = torch.ones(n // 2, device=dev)
            fn = lambda: qe.qe_accumulate(g, t, True)
            work = {"bytes": 12 * (n // 2)}
        else:
            raise SystemExit("unknown case " + a.case)
    for _ in range(2):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / a.reps
    out = {"case": a.case, "ms": round(ms, 4), "status": int(status.item())}
    if "launches" in work:
        out["launches"] = work["launches"]
    if "flop" in work:
        out["TFLOP/s"] = round(work["flop"] / ms / 1e9, 1)
    out["GB/s_algorithmic"] = round(work["bytes"] / ms / 1e6, 1)
    print(json.dumps(out))


if __name__ == "__main__":
    main()
