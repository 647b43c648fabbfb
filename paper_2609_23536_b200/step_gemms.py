"""The GEMM launches of one optimizer step as the default issue plan groups them (schedules.plan_rounds), with random
FP8 operands of the configuration's shapes: used by bench.py's roofline leg and by the profiling cases to time and
profile the dominant kernel alone.  Holds no arithmetic of the method."""
from __future__ import annotations

import torch

from .schedules import peak_live, plan_rounds, sched


def build(cfg, device, max_group=8):
    """Returns (launches, flops, algorithmic_bytes): launches is a list of lists of qe_gemm_fp8_group problem tuples
    (a, a_format, a_mn, b, b_format, b_mn, alpha_a, alpha_b, d, out_kind, amax); every (linear, microbatch) has
    operands and outputs of its own, every linear one weight and one FP32 gradient slice."""
    T, M = cfg["T"], cfg["M"]
    lin = cfg["linears"] * cfg["layers"]
    schedule = sched(M, *cfg["sched"])
    rounds = plan_rounds(schedule, len(lin), peak_live(schedule), max_group, max(2, cfg["sched"][0] + cfg["sched"][1]))
    one = torch.ones(1, dtype=torch.float32, device=device)
    u8 = lambda *shape: torch.randint(0, 120, shape, dtype=torch.uint8, device=device)
    Wq = [u8(N, K) for _, K, N in lin]
    grad = [torch.zeros((N, K), dtype=torch.float32, device=device) for _, K, N in lin]
    Xq = [[u8(T, K) for _, K, N in lin] for _ in range(M)]
    Gq = [[u8(T, N) for _, K, N in lin] for _ in range(M)]
    Y = [[torch.zeros((T, N), dtype=torch.bfloat16, device=device) for _, K, N in lin] for _ in range(M)]
    dX = [[torch.zeros((T, K), dtype=torch.bfloat16, device=device) for _, K, N in lin] for _ in range(M)]
    launches, flops, nbytes = [], 0.0, 0
    for grp in rounds:
        ps = []
        for a, i, m in grp:
            _, K, N = lin[i]
            flops += 2.0 * T * N * K
            if a == "F":
                ps.append((Xq[m][i], 0, 0, Wq[i], 0, 0, one, one, Y[m][i], 0, None))
                nbytes += T * K + N * K + 2 * T * N
            elif a == "dI":  # Wq [N,K] as an MN-major B operand
                ps.append((Gq[m][i], 1, 0, Wq[i], 0, 1, one, one, dX[m][i], 0, None))
                nbytes += T * N + N * K + 2 * T * K
            else:            # Gq [T,N] and Xq [T,K] as MN-major A and B operands; FP32 accumulate
                ps.append((Gq[m][i], 1, 1, Xq[m][i], 0, 1, one, one, grad[i], 2, None))
                nbytes += T * N + T * K + 8 * N * K
        pairable = [q for q in ps if q[8].shape[0] % 256 == 0]
        launches += [[q] for q in ps if q[8].shape[0] % 256]  # single-CTA variant: a launch of its own, as in the layer
        if len(pairable) >= 2:
            launches.append(pairable)
        else:
            launches += [[q] for q in pairable]
    return launches, flops, nbytes


def run(qe, launches, status):
    for ps in launches:
        if len(ps) == 1:
            a, af, amn, b, bf, bmn, sa, sb, d, kind, am = ps[0]
            qe.qe_gemm_fp8_ex(a, af, bool(amn), b, bf, bool(bmn), sa, sb, d, kind, am, status)
        else:
            qe.qe_gemm_fp8_group(ps, status)
