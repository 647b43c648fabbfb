"""The FP8 delayed-scaling linear layer as a checked F / dI / dW state machine.

TEST INFRASTRUCTURE ONLY; shares no code with the CUDA path.

What is followed, in the paper's order and notation:
  * Eqs. 3-5:  (Y, S1, T) = F(X, W, S0);  (dX, S2, Q) = dI(dY, T, S1);  dW = dW(Q).
    F and dI each advance the effect token once and update scaling state once;
    dW never touches scaling state (Invariant 1).
  * Eqs. 1-2:  TapeKey(e, s, m, u, i) names the stage execution, TapeRef(p, g_p)
    names the slot and its generation.  One live tape per key, an occupied slot
    is never pre-empted, release keeps g_p, a consumer presents key and exact
    generation (Invariant 2).  A per-tape consumer bitmask rejects duplicate
    consumption and frees the slot only after both dI and dW succeeded.
  * Sec. 3.3: weight version e_W and cache version e_C; the first forward after
    an optimizer step refreshes the quantised-weight cache and sets e_C <- e_W,
    later forwards verify it (Invariant 3).
  * Sec. 3.4: direct gradient placement.  The destination is validated, the
    first write of an epoch must be microbatch 0 and overwrites, later writes
    accumulate in place; duplicate / missing / aliased writes fail; every
    configured microbatch writes exactly once before the optimizer commit.
  * Algorithm 1: a check precedes its action; state changes only after the
    action succeeded.  Sec. 4.5: a failure aborts outstanding tapes and marks
    the arena unusable for the epoch.

Numerics (the paper prints none; these are the readings taken):
  amax      max |x| over the bf16 tensor, as fp32
  quantise  fp8_rne_sat(fp32(x) * scale)         X, W -> E4M3, dY -> E5M2
  F         Y  = bf16_rne( sum_k Xq[t,k] Wq[n,k] * sinv_X * sinv_W )     (float64, one rounding)
  dI        dX = bf16_rne( sum_n Gq[t,n] Wq[n,k] * sinv_G * sinv_W )
  dW        D  = fp32_rne( sum_t Gq[t,n] Xq[t,k] * sinv_G * sinv_X ); mg = D or fp32(mg + D)
  The inverse scales a deferred dW uses are the snapshots taken when X_m and
  dY_m were quantised (kept in the tape), never the current state.
  Output amax is taken over the rounded bf16 Y actually produced.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import NamedTuple, Optional

import numpy as np

from . import bf16, fp8
from .scaling import ScaleState, amax_bf16

INVALID_EPOCH = (1 << 64) - 1
DI_BIT, DW_BIT = 1, 2
CLASSES = ("X", "W", "G", "Y")


class ContractError(Exception):
    """A rejected action; .code is the symbolic error name (matches the C-ABI's QE_ERR_<code>)."""

    def __init__(self, code: str, msg: str = ""):
        super().__init__(f"{code}: {msg}" if msg else code)
        self.code = code


class TapeKey(NamedTuple):
    epoch: int
    stage: int
    mb: int
    unit: int
    inv: int


class TapeRef(NamedTuple):
    slot: int
    gen: int


class Tape(NamedTuple):
    key: TapeKey
    ref: TapeRef


@dataclass
class _Slot:
    gen: int = 0
    live: bool = False
    key: Optional[TapeKey] = None
    bits: int = 0
    Xq: Optional[np.ndarray] = None
    Gq: Optional[np.ndarray] = None
    sinv_X: np.float32 = np.float32(0)
    sinv_G: np.float32 = np.float32(0)


class ArenaRegistry:
    """Destinations bound in the current epoch by the layers of one context (alias check)."""

    def __init__(self):
        self.bound = {}  # layer id -> (buffer id, first element, one-past-last element)

    def check_and_bind(self, layer_id, buf, off, n):
        rng = (id(buf), off, off + n)
        for other, (b, lo, hi) in self.bound.items():
            if other != layer_id and b == rng[0] and lo < rng[2] and rng[1] < hi:
                raise ContractError("DEST", "destination aliases another layer's slice")
        self.bound[layer_id] = rng

    def unbind(self, layer_id):
        self.bound.pop(layer_id, None)


class OracleLinear:
    """One linear layer W[N,K]; tokens T; P tape slots; history length H; margin mu."""

    def __init__(self, T, K, N, H, margin, slots, stage=0, unit=0, inv=0, registry=None):
        self.T, self.K, self.N = int(T), int(K), int(N)
        self.P = int(slots)
        self.stage, self.unit, self.inv = stage, unit, inv
        self.S = {
            "X": ScaleState(fp8.E4M3, H, margin),
            "W": ScaleState(fp8.E4M3, H, margin),
            "G": ScaleState(fp8.E5M2, H, margin),
            "Y": ScaleState(fp8.E4M3, H, margin),
        }
        self.e_W = 0
        self.e_C = INVALID_EPOCH
        self.token = 0
        self.fwd_in_epoch = 0
        self.write_mask = 0
        self.aborted = False
        self.slots = [_Slot() for _ in range(self.P)]
        self.W_bits = None  # bf16 bits [N,K], set by the caller ("the parameter")
        self.Wq = None
        self.cache_sinv_W = np.float32(0)
        self.bound_dest = None  # (id(buf), off) for this epoch
        self.registry = registry if registry is not None else ArenaRegistry()

    # ------------------------------------------------------------------ parameters
    def set_weight(self, W_bits: np.ndarray) -> None:
        W_bits = np.asarray(W_bits, dtype=np.uint16)
        assert W_bits.shape == (self.N, self.K)
        self.W_bits = W_bits

    # ------------------------------------------------------------------ pool helpers
    def _resolve(self, tape: Tape) -> _Slot:
        """Retained-work lookup: generation first, then key, then epoch."""
        p, g = tape.ref
        if not (0 <= p < self.P):
            raise ContractError("STALE_REF", "slot out of range")
        s = self.slots[p]
        if not s.live or s.gen != g:
            raise ContractError("STALE_REF", "generation does not name the slot's live tape")
        if s.key != tape.key:
            raise ContractError("KEY_MISMATCH")
        if tape.key.epoch != self.e_W:
            raise ContractError("EPOCH")
        return s

    def live_tapes(self) -> int:
        return sum(1 for s in self.slots if s.live)

    def next_slot(self) -> int:
        for p, s in enumerate(self.slots):
            if not s.live:
                return p
        return -1

    # ------------------------------------------------------------------ F
    def forward(self, mb: int, gen: int, X_bits: np.ndarray, rows=None, light: bool = False):
        """Returns (tape, Y_bits).  With rows=[...] only those rows of Y are computed
        (returned as [len(rows), N]) and the Y scaling class is not advanced.
        light=True (a test-speed switch, no arithmetic of its own): bookkeeping, amax and scale
        updates only -- no FP8 bytes are produced, the tape cannot feed a GEMM, Y_bits is None."""
        if self.aborted:
            raise ContractError("ABORTED")
        if not (0 <= mb < 64):
            raise ContractError("BAD_ARG", "microbatch index out of range")
        if gen != self.e_W:
            raise ContractError("EPOCH", "caller's weight version differs from e_W")
        refresh = self.fwd_in_epoch == 0
        if not refresh and self.e_C != self.e_W:
            raise ContractError("STALE_CACHE", "cache refresh required")
        key = TapeKey(self.e_W, self.stage, mb, self.unit, self.inv)
        if any(s.live and s.key == key for s in self.slots):
            raise ContractError("KEY_LIVE")
        p = self.next_slot()
        if p < 0:
            raise ContractError("POOL_FULL")
        X_bits = np.asarray(X_bits, dtype=np.uint16)
        if X_bits.shape != (self.T, self.K):
            raise ContractError("SHAPE")

        # ---- physical action
        aW = None
        if refresh:
            self._refresh_scale_W = np.float32(self.S["W"].scale)  # the scale this epoch's cache is cast with
            Wf = bf16.decode(self.W_bits)
            aW = amax_bf16(Wf)
            self.Wq = None if light else fp8.quantize(Wf, self.S["W"].scale, fp8.E4M3)
            self.cache_sinv_W = np.float32(self.S["W"].scale_inv)
        Xf = bf16.decode(X_bits)
        aX = amax_bf16(Xf)
        sinv_X = np.float32(self.S["X"].scale_inv)
        Xq = Y_bits = aY = None
        if not light:
            if self.Wq is None:  # the epoch's refresh ran in light mode: produce the cache bytes now, same scale
                self.Wq = fp8.quantize(bf16.decode(self.W_bits), self._refresh_scale_W, fp8.E4M3)
            Xq = fp8.quantize(Xf, self.S["X"].scale, fp8.E4M3)
            Y_bits = gemm_fwd(Xq, self.Wq, sinv_X, self.cache_sinv_W, rows)
            if rows is None:
                aY = amax_bf16(bf16.decode(Y_bits))

        # ---- commit
        s = self.slots[p]
        s.gen += 1
        s.live, s.key, s.bits = True, key, 0
        s.Xq, s.sinv_X, s.Gq, s.sinv_G = Xq, sinv_X, None, np.float32(0)
        if refresh:
            self.S["W"].commit(aW)
            self.e_C = self.e_W
        self.S["X"].commit(aX)
        if aY is not None:
            self.S["Y"].commit(aY)
        self.token += 1
        self.fwd_in_epoch += 1
        return Tape(key, TapeRef(p, s.gen)), Y_bits

    # ------------------------------------------------------------------ dI
    def backward_dI(self, tape: Tape, dY_bits: np.ndarray, rows=None, light: bool = False) -> np.ndarray:
        if self.aborted:
            raise ContractError("ABORTED")
        s = self._resolve(tape)
        if s.bits & DI_BIT:
            raise ContractError("DUP_CONSUME", "dI already consumed this tape")
        dY_bits = np.asarray(dY_bits, dtype=np.uint16)
        if dY_bits.shape != (self.T, self.N):
            raise ContractError("SHAPE")

        Gf = bf16.decode(dY_bits)
        aG = amax_bf16(Gf)
        sinv_G = np.float32(self.S["G"].scale_inv)
        Gq = dX_bits = None
        if not light:
            Gq = fp8.quantize(Gf, self.S["G"].scale, fp8.E5M2)
            dX_bits = gemm_dI(Gq, self.Wq, sinv_G, self.cache_sinv_W, rows)

        s.Gq, s.sinv_G = Gq, sinv_G
        s.bits |= DI_BIT
        self.S["G"].commit(aG)
        self.token += 1
        return dX_bits

    # ------------------------------------------------------------------ dW
    def backward_dW(self, tape: Tape, buf: np.ndarray, off: int, rows=None) -> None:
        """Accumulate into buf[off : off + N*K] viewed as [N,K] (fp32, in place).
        With rows=[...] only those rows n of the slice are computed and written."""
        if self.aborted:
            raise ContractError("ABORTED")
        s = self._resolve(tape)
        if s.bits & DW_BIT:
            raise ContractError("DUP_CONSUME", "dW already consumed this tape")
        if not (s.bits & DI_BIT):
            raise ContractError("ORDER", "dW before dI")
        n = self.N * self.K
        if (
            not isinstance(buf, np.ndarray)
            or buf.dtype != np.float32
            or buf.ndim != 1
            or off < 0
            or off % 4 != 0  # 16-byte alignment of the slice, in fp32 elements
            or off + n > buf.size
        ):
            raise ContractError("DEST")
        if self.bound_dest is not None and self.bound_dest != (id(buf), off):
            raise ContractError("DEST", "differs from the destination bound for this epoch")
        self.registry.check_and_bind(id(self), buf, off, n)
        mb = tape.key.mb
        if self.write_mask >> mb & 1:
            raise ContractError("DUP_WRITE")
        if self.write_mask == 0 and mb != 0:
            raise ContractError("ORDER", "microbatch 0 initialises the accumulation")

        if s.Xq is not None and s.Gq is not None:  # (a tape made in light mode carries no bytes: bookkeeping only)
            D = gemm_dW(s.Gq, s.Xq, s.sinv_G, s.sinv_X, rows)
            view = buf[off : off + n].reshape(self.N, self.K)
            sel = slice(None) if rows is None else np.asarray(rows)
            if self.write_mask == 0:
                view[sel] = D
            else:
                view[sel] = (view[sel] + D).astype(np.float32)  # fp32 + fp32 -> fp32, IEEE RN

        self.bound_dest = (id(buf), off)
        self.write_mask |= 1 << mb
        s.bits |= DW_BIT
        s.live, s.Xq, s.Gq = False, None, None  # both bits set: release, generation kept

    # ------------------------------------------------------------------ per-microbatch arena (Sec. 3.4, Eq. for A_r)
    def backward_dW_arena(self, tape: Tape, arena: np.ndarray, layer_off: int, microbatches: int, rows=None) -> None:
        """The arena as the paper sizes it: one 2-byte view per matrix parameter and configured microbatch
        (capacity M * sizeof(W)).  Microbatch m writes bf16(D_m) into its own view at
        arena[layer_off + m*N*K : +N*K]; nothing is accumulated here.  Same checks and state transitions as
        backward_dW; the bound destination is the layer's whole region of M views."""
        if self.aborted:
            raise ContractError("ABORTED")
        s = self._resolve(tape)
        if s.bits & DW_BIT:
            raise ContractError("DUP_CONSUME", "dW already consumed this tape")
        if not (s.bits & DI_BIT):
            raise ContractError("ORDER", "dW before dI")
        n = self.N * self.K
        mb = tape.key.mb
        if (
            not isinstance(arena, np.ndarray)
            or arena.dtype != np.uint16
            or arena.ndim != 1
            or layer_off < 0
            or layer_off % 8 != 0  # 16-byte alignment, in 2-byte elements
            or not (1 <= microbatches <= 64)
            or mb >= microbatches
            or layer_off + microbatches * n > arena.size
        ):
            raise ContractError("DEST")
        if self.bound_dest is not None and self.bound_dest != (id(arena), layer_off):
            raise ContractError("DEST", "differs from the destination bound for this epoch")
        self.registry.check_and_bind(id(self), arena, layer_off, microbatches * n)
        if self.write_mask >> mb & 1:
            raise ContractError("DUP_WRITE")
        if self.write_mask == 0 and mb != 0:
            raise ContractError("ORDER", "microbatch 0 initialises the accumulation")
        if s.Xq is not None and s.Gq is not None:
            G = fp8.decode(s.Gq, fp8.E5M2)
            if rows is not None:
                G = G[:, np.asarray(rows)]
            acc = G.T @ fp8.decode(s.Xq, fp8.E4M3)
            bits = bf16.round_from_f64(acc * np.float64(s.sinv_G) * np.float64(s.sinv_X))
            view = arena[layer_off + mb * n : layer_off + (mb + 1) * n].reshape(self.N, self.K)
            view[slice(None) if rows is None else np.asarray(rows)] = bits
        self.bound_dest = (id(arena), layer_off)
        self.write_mask |= 1 << mb
        s.bits |= DW_BIT
        s.live, s.Xq, s.Gq = False, None, None

    def arena_finalize(self, arena: np.ndarray, layer_off: int, microbatches: int, buf: np.ndarray, off: int) -> None:
        """Before the optimizer boundary: the optimizer-visible FP32 gradient is the sum of the layer's M views,
        added in microbatch order in FP32: buf[off + i] = (...((v_0[i] + v_1[i]) + v_2[i]) ... + v_{M-1}[i]).
        Every configured microbatch must have written exactly once."""
        if self.aborted:
            raise ContractError("ABORTED")
        n = self.N * self.K
        if self.write_mask != (1 << microbatches) - 1:
            raise ContractError("INCOMPLETE", "a microbatch has not written its view")
        if self.bound_dest != (id(arena), layer_off):
            raise ContractError("DEST", "not the arena region bound this epoch")
        if buf.dtype != np.float32 or buf.ndim != 1 or off < 0 or off % 4 != 0 or off + n > buf.size:
            raise ContractError("DEST")
        total = bf16.decode(arena[layer_off : layer_off + n]).astype(np.float32)
        for m in range(1, microbatches):
            v = bf16.decode(arena[layer_off + m * n : layer_off + (m + 1) * n]).astype(np.float32)
            total = (total + v).astype(np.float32)
        buf[off : off + n] = total

    # ------------------------------------------------------------------ boundaries
    def optimizer_boundary(self, microbatches_expected: int) -> None:
        if self.aborted:
            raise ContractError("ABORTED")
        if self.live_tapes():
            raise ContractError("PENDING", "live tape at the optimizer boundary")
        if self.write_mask != (1 << microbatches_expected) - 1:
            raise ContractError("INCOMPLETE", "a microbatch has not written its gradient")
        self.e_W += 1
        self.write_mask = 0
        self.fwd_in_epoch = 0
        self.bound_dest = None
        self.registry.unbind(id(self))

    def abort_step(self) -> None:
        for s in self.slots:
            if s.live and s.key.epoch == self.e_W:
                s.live, s.Xq, s.Gq = False, None, None
        self.aborted = True

    def arena_rebuild(self) -> None:
        """Restart the epoch after an abort: arena usable again, nothing written yet."""
        if self.live_tapes():
            raise ContractError("PENDING")
        self.aborted = False
        self.write_mask = 0
        self.fwd_in_epoch = 0
        self.bound_dest = None
        self.registry.unbind(id(self))

    def invalidate_cache(self) -> None:
        self.e_C = INVALID_EPOCH

    def scale_commit(self, cls: str, amax) -> None:
        """The scale update as a standalone call (same rule F and dI apply)."""
        self.S[cls].commit(np.float32(amax))

    def checkpoint_allowed(self) -> None:
        """Invariant 4: persistent state may be serialised only at quiescence."""
        if self.live_tapes():
            raise ContractError("PENDING", "checkpoint withheld: live tape")

    # ------------------------------------------------------------------ checkpoint / restart (Sec. 3.5, Invariant 4)
    def save_state(self) -> dict:
        """Persistent state only: numerics and the weight version.  Withheld while a tape is live."""
        self.checkpoint_allowed()
        return {
            "e_W": self.e_W,
            "classes": {c: {"hist": self.S[c].hist.copy(), "count": self.S[c].count, "scale": np.float32(self.S[c].scale),
                            "scale_inv": np.float32(self.S[c].scale_inv)} for c in CLASSES},
        }

    def load_state(self, saved: dict) -> None:
        """Restart rule: restore numerics and e_W, rebuild process-local resources (generations and the
        token keep this process's values), and leave the cache stale so the first forward refreshes it."""
        if self.live_tapes():
            raise ContractError("PENDING")
        for c in CLASSES:
            d = saved["classes"][c]
            self.S[c].hist = d["hist"].copy()
            self.S[c].count = d["count"]
            self.S[c].scale, self.S[c].scale_inv = np.float32(d["scale"]), np.float32(d["scale_inv"])
        self.e_W = saved["e_W"]
        self.e_C = INVALID_EPOCH
        self.fwd_in_epoch = 0
        self.write_mask = 0
        self.aborted = False
        self.bound_dest = None
        self.registry.unbind(id(self))
        self.Wq = None

    # ------------------------------------------------------------------ inspection
    def state(self) -> dict:
        return {
            "classes": {c: self.S[c].snapshot() for c in CLASSES},
            "token": self.token,
            "e_W": self.e_W,
            "e_C": self.e_C,
            "write_mask": self.write_mask,
            "fwd_in_epoch": self.fwd_in_epoch,
            "aborted": self.aborted,
            "slots": [
                {"gen": s.gen, "live": s.live, "bits": s.bits, "key": tuple(s.key) if s.live else None}
                for s in self.slots
            ],
        }


# ---------------------------------------------------------------------- GEMM definitions
def _rows(a: np.ndarray, rows):
    return a if rows is None else a[np.asarray(rows)]


def gemm_fwd(Xq, Wq, sinv_X, sinv_W, rows=None) -> np.ndarray:
    """Y[t,n] = bf16( sum_k dec(Xq[t,k]) dec(Wq[n,k]) * sinv_X * sinv_W ), bits uint16."""
    A = fp8.decode(_rows(Xq, rows), fp8.E4M3)
    B = fp8.decode(Wq, fp8.E4M3)
    acc = A @ B.T
    return bf16.round_from_f64(acc * np.float64(sinv_X) * np.float64(sinv_W))


def gemm_dI(Gq, Wq, sinv_G, sinv_W, rows=None) -> np.ndarray:
    """dX[t,k] = bf16( sum_n dec(Gq[t,n]) dec(Wq[n,k]) * sinv_G * sinv_W ), bits uint16."""
    A = fp8.decode(_rows(Gq, rows), fp8.E5M2)
    B = fp8.decode(Wq, fp8.E4M3)
    acc = A @ B
    return bf16.round_from_f64(acc * np.float64(sinv_G) * np.float64(sinv_W))


def gemm_dW(Gq, Xq, sinv_G, sinv_X, rows=None) -> np.ndarray:
    """D[n,k] = fp32( sum_t dec(Gq[t,n]) dec(Xq[t,k]) * sinv_G * sinv_X ); rows select n."""
    G = fp8.decode(Gq, fp8.E5M2)
    if rows is not None:
        G = G[:, np.asarray(rows)]
    X = fp8.decode(Xq, fp8.E4M3)
    acc = G.T @ X
    return (acc * np.float64(sinv_G) * np.float64(sinv_X)).astype(np.float32)
