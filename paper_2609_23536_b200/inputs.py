"""Seeded synthetic tensors for tests and benchmarks (bf16, as torch CPU tensors).

Holds no arithmetic of the method: it only draws random numbers and rounds them to
bfloat16 storage.  Both the CPU oracle's tests and the CUDA path's tests take their
inputs from here, so that they see identical bits.

The paper verifies bit-exact state on synthetic inputs (Sec. 5.1, methodology); the
shapes and distributions here are those of the benchmark configurations:
activations ~ N(0,1) (or Student-t with 3 degrees of freedom for the rollover
stress), weights ~ N(0, 0.02^2), upstream gradients ~ N(0, (1e-3)^2).
"""
from __future__ import annotations

import hashlib

import numpy as np
import torch

BASE_SEED = 23536


def seed_for(*parts) -> int:
    h = hashlib.sha256(repr((BASE_SEED,) + tuple(parts)).encode()).digest()
    return int.from_bytes(h[:8], "little") & ((1 << 63) - 1)


def _gen(*parts) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed_for(*parts))
    return g


def normal_bf16(shape, std: float, *seed_parts, device=None) -> torch.Tensor:
    """device=None: drawn by the CPU generator.  With a CUDA device the same seed feeds that device's generator
    instead (other numbers, equally reproducible): the full-size configurations draw gigabytes per step, which the
    CPU generator would take minutes over; whoever needs the tensor on the host copies it back, so both sides of a
    comparison still see identical bits."""
    if device is None or torch.device(device).type == "cpu":
        x = torch.randn(shape, generator=_gen(*seed_parts), dtype=torch.float32)
    else:
        g = torch.Generator(device=device)
        g.manual_seed(seed_for(*seed_parts))
        x = torch.randn(shape, generator=g, dtype=torch.float32, device=device)
    return (x * std).to(torch.bfloat16)


def student_t3_bf16(shape, *seed_parts) -> torch.Tensor:
    """Student-t with 3 degrees of freedom: Z / sqrt(chi2_3 / 3)."""
    g = _gen(*seed_parts)
    z = torch.randn(shape, generator=g, dtype=torch.float32)
    c = torch.randn((3,) + tuple(shape), generator=g, dtype=torch.float32).square_().sum(0)
    return (z / (c / 3.0).sqrt_()).to(torch.bfloat16)


def spike_mask(shape, fraction: float, *seed_parts) -> torch.Tensor:
    return torch.rand(shape, generator=_gen(*seed_parts)) < fraction


def activations(cfg: str, step: int, layer: int, linear: int, mb: int, T: int, K: int, device=None) -> torch.Tensor:
    return normal_bf16((T, K), 1.0, cfg, step, layer, linear, mb, "X", device=device)


def upstream_grads(cfg: str, step: int, layer: int, linear: int, mb: int, T: int, N: int, device=None) -> torch.Tensor:
    return normal_bf16((T, N), 1e-3, cfg, step, layer, linear, mb, "dY", device=device)


def weights(cfg: str, layer: int, linear: int, N: int, K: int, device=None) -> torch.Tensor:
    return normal_bf16((N, K), 0.02, cfg, 0, layer, linear, "W", device=device)


def optimizer_perturbation(w: torch.Tensor, cfg: str, step: int, layer: int, linear: int) -> torch.Tensor:
    """Stand-in for the optimizer: W <- bf16(W + delta), delta ~ N(0, (2e-5)^2), independent
    of every GEMM output so state trajectories stay comparable bit for bit.  Drawn on w's device."""
    if w.device.type == "cpu":
        d = torch.randn(w.shape, generator=_gen(cfg, step, layer, linear, "dW_opt"), dtype=torch.float32) * 2e-5
    else:
        g = torch.Generator(device=w.device)
        g.manual_seed(seed_for(cfg, step, layer, linear, "dW_opt"))
        d = torch.randn(w.shape, generator=g, dtype=torch.float32, device=w.device) * 2e-5
    return (w.float() + d).to(torch.bfloat16)


def stress_activations(step: int, mb: int, T: int, K: int) -> torch.Tensor:
    """Rollover stress: Student-t(3); x1000 on a seeded 0.1 % of elements at step 5; whole
    tensor x1e-3 at step 9."""
    x = student_t3_bf16((T, K), "C4", step, mb, "X").float()
    if step == 5:
        m = spike_mask((T, K), 1e-3, "C4", step, mb, "spike")
        x = torch.where(m, x * 1000.0, x)
    if step == 9:
        x = x * 1e-3
    return x.to(torch.bfloat16)


def bits(t: torch.Tensor) -> np.ndarray:
    """bf16 torch tensor -> numpy uint16 bit patterns (what the oracle consumes)."""
    assert t.dtype == torch.bfloat16
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def from_bits(b: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(b).view(np.int16)).view(torch.bfloat16)


# Llama-style block linears: (name, K in-features, N out-features)
def block_linears(hidden: int, qkv_out: int, ffn: int):
    return [
        ("qkv", hidden, qkv_out),
        ("o", hidden, hidden),
        ("gate_up", hidden, 2 * ffn),
        ("down", ffn, hidden),
    ]


CONFIGS = {
    # name: tokens, linears, history, margin, microbatches, schedule (warmup, defer), steps
    "C1": dict(T=256, linears=[("lin", 256, 256)], H=4, margin=0, M=4, sched=(1, 0), steps=3, layers=1),
    "C2": dict(T=2048, linears=block_linears(2048, 6144, 5632), H=1024, margin=0, M=8, sched=(3, 3), steps=1, layers=1),
    "C3": dict(T=4096, linears=block_linears(4096, 6144, 14336), H=1024, margin=0, M=16, sched=(3, 3), steps=10, layers=4),
    "C4": dict(T=4096, linears=[("lin", 4096, 4096)], H=16, margin=1, M=8, sched=(1, 2), steps=12, layers=1),
    "C5": dict(T=512, linears=[(f"l{i}", 1024, 1024) for i in range(48)], H=16, margin=0, M=32, sched=(3, 3), steps=1, layers=1),
}


def grad_offsets(linears):
    """Affine element offsets of each linear's [N,K] slice in one flat fp32 buffer."""
    offs, o = [], 0
    for _, K, N in linears:
        offs.append(o)
        o += N * K
    return offs, o
