"""ctypes binding over libqe.so: the same entry points as include/qe.h, argument marshalling only.

Every step of the path runs inside the library's CUDA kernels.  There is no fallback: if the shared
library is missing the import fails, and every call raises QEError on a negative status.

torch tensors are accepted wherever the C signature takes a device pointer (their data_ptr() is
passed); streams default to torch's current CUDA stream.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqe.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} not found: build it with `python -m paper_2609_23536_b200.build` "
        "(this package has no CPU or PyTorch fallback)"
    )
lib = C.CDLL(LIB_PATH)

QE_MAX_SLOTS = 64
QE_INVALID_EPOCH = (1 << 64) - 1
EAGER, GRAPH = 0, 1
OVERLAP_DW = 1
UNSAFE_ONE_WAY_HANDOFF = 2  # diagnostic: the one-way handoff of the paper's stale-read experiment
CLASS_X, CLASS_W, CLASS_G, CLASS_Y = 0, 1, 2, 3
CLASS_NAMES = ("X", "W", "G", "Y")
E4M3, E5M2 = 0, 1


class qe_tape_key(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("epoch", "stage", "mb", "unit", "inv")]


class qe_tape_ref(C.Structure):
    _fields_ = [("slot", C.c_uint32), ("reserved", C.c_uint32), ("gen", C.c_uint64)]


class qe_tape(C.Structure):
    _fields_ = [("key", qe_tape_key), ("reserved", C.c_uint32), ("ref", qe_tape_ref)]

    def astuple(self):
        k, r = self.key, self.ref
        return ((k.epoch, k.stage, k.mb, k.unit, k.inv), (r.slot, r.gen))


class qe_slot_view(C.Structure):
    _fields_ = [("gen", C.c_uint64), ("live", C.c_uint32), ("bits", C.c_uint32), ("key", qe_tape_key), ("reserved", C.c_uint32)]


class qe_contract_view(C.Structure):
    _fields_ = [
        ("e_W", C.c_uint64), ("e_C", C.c_uint64), ("token", C.c_uint64), ("write_mask", C.c_uint64),
        ("fwd_in_epoch", C.c_uint32), ("aborted", C.c_uint32), ("slots", C.c_uint32), ("live_tapes", C.c_uint32),
        ("slot", qe_slot_view * QE_MAX_SLOTS),
    ]


class qe_ctx_config(C.Structure):
    _fields_ = [("exec_mode", C.c_uint32), ("device", C.c_int32), ("exec_stream", C.c_void_p), ("flags", C.c_uint32), ("step_window", C.c_uint32), ("reserved", C.c_uint32 * 2)]


class qe_layer_config(C.Structure):
    _fields_ = [
        ("T", C.c_uint32), ("K", C.c_uint32), ("N", C.c_uint32), ("history_len", C.c_uint32), ("margin", C.c_int32),
        ("slots", C.c_uint32), ("stage", C.c_uint32), ("unit", C.c_uint32), ("inv", C.c_uint32), ("host_io", C.c_uint32),
        ("weight_dev", C.c_void_p), ("reserved1", C.c_uint64 * 4),
    ]


class qe_step_action(C.Structure):
    _fields_ = [("kind", C.c_uint32), ("layer", C.c_uint32), ("mb", C.c_uint32), ("reserved", C.c_uint32)]


class qe_step_io(C.Structure):
    _fields_ = [("x_dev", C.c_void_p), ("y_dev", C.c_void_p), ("dy_dev", C.c_void_p), ("dx_dev", C.c_void_p)]


class qe_class_state(C.Structure):
    _fields_ = [("scale", C.c_float), ("scale_inv", C.c_float), ("count", C.c_uint32), ("reserved", C.c_uint32)]


class qe_state_view(C.Structure):
    _fields_ = [
        ("cls", qe_class_state * 4), ("cache_sinv_W", C.c_float), ("device_status", C.c_uint32),
        ("device_token", C.c_uint64), ("contract", qe_contract_view),
    ]


class qe_stats(C.Structure):
    _fields_ = [
        ("graphs_built", C.c_uint64), ("graph_replays", C.c_uint64), ("eager_launches", C.c_uint64),
        ("handoffs", C.c_uint64), ("node_param_updates", C.c_uint64), ("kernels_launched", C.c_uint64),
        ("capture_host_ms", C.c_double), ("workspace_bytes", C.c_uint64), ("grouped_dw", C.c_uint64), ("paired_f_di", C.c_uint64),
    ]

    def asdict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


# every symbol include/qe.h declares, with its signature
_P = C.c_void_p


class qe_gemm_desc(C.Structure):
    _fields_ = [
        ("a_dev", _P), ("b_dev", _P), ("d_dev", _P), ("alpha_a_dev", _P), ("alpha_b_dev", _P), ("amax_dev", _P),
        ("a_format", C.c_uint32), ("a_mn", C.c_uint32), ("b_format", C.c_uint32), ("b_mn", C.c_uint32),
        ("M", C.c_uint32), ("Nn", C.c_uint32), ("Kc", C.c_uint32), ("out_kind", C.c_uint32),
    ]


class qe_action(C.Structure):
    _fields_ = [
        ("kind", C.c_uint32), ("mb", C.c_uint32), ("gen", C.c_uint64), ("layer", _P), ("in_dev", _P), ("out_dev", _P),
        ("tape", C.POINTER(qe_tape)), ("grad_offset", C.c_uint64),
    ]


_SIGNATURES = {
    "qe_registry_create": (C.c_int32, [C.POINTER(_P)]),
    "qe_registry_destroy": (C.c_int32, [_P]),
    "qe_contract_create": (C.c_int32, [C.c_uint32] * 4 + [_P, C.POINTER(_P)]),
    "qe_contract_destroy": (C.c_int32, [_P]),
    "qe_contract_forward_check": (C.c_int32, [_P, C.c_uint32, C.c_uint64, C.POINTER(C.c_int32), C.POINTER(C.c_uint32)]),
    "qe_contract_forward_commit": (C.c_int32, [_P, C.c_uint32, C.POINTER(qe_tape)]),
    "qe_contract_dI_check": (C.c_int32, [_P, C.POINTER(qe_tape)]),
    "qe_contract_dI_commit": (C.c_int32, [_P, C.POINTER(qe_tape)]),
    "qe_contract_dW_check": (C.c_int32, [_P, C.POINTER(qe_tape), C.c_uint64, C.c_uint64, C.c_uint64, C.c_uint64, C.POINTER(C.c_int32)]),
    "qe_contract_dW_commit": (C.c_int32, [_P, C.POINTER(qe_tape), C.c_uint64, C.c_uint64, C.c_uint64]),
    "qe_contract_boundary": (C.c_int32, [_P, C.c_uint32]),
    "qe_contract_abort": (C.c_int32, [_P]),
    "qe_contract_rebuild": (C.c_int32, [_P]),
    "qe_contract_invalidate_cache": (C.c_int32, [_P]),
    "qe_contract_checkpoint_check": (C.c_int32, [_P]),
    "qe_contract_restore": (C.c_int32, [_P, C.c_uint64]),
    "qe_contract_get": (C.c_int32, [_P, C.POINTER(qe_contract_view)]),
    "qe_ctx_create": (C.c_int32, [C.POINTER(qe_ctx_config), C.POINTER(_P)]),
    "qe_ctx_destroy": (C.c_int32, [_P]),
    "qe_layer_workspace_bytes": (C.c_int32, [C.POINTER(qe_layer_config), C.POINTER(C.c_uint64)]),
    "qe_layer_create": (C.c_int32, [_P, C.POINTER(qe_layer_config), _P, C.c_uint64, C.POINTER(_P)]),
    "qe_layer_destroy": (C.c_int32, [_P]),
    "qe_forward": (C.c_int32, [_P, C.c_uint32, C.c_uint64, _P, _P, _P, C.POINTER(qe_tape)]),
    "qe_backward_dI": (C.c_int32, [_P, C.POINTER(qe_tape), _P, _P, _P]),
    "qe_forward_host": (C.c_int32, [_P, C.c_uint32, C.c_uint64, _P, _P, _P, C.POINTER(qe_tape)]),
    "qe_backward_dI_host": (C.c_int32, [_P, C.POINTER(qe_tape), _P, _P, _P]),
    "qe_backward_dW": (C.c_int32, [_P, C.POINTER(qe_tape), _P, C.c_uint64, C.c_uint64, _P]),
    "qe_backward_dW_staged": (C.c_int32, [_P, C.POINTER(qe_tape), _P, C.c_uint64, C.c_uint64, _P, _P]),
    "qe_forward_dI_pair": (C.c_int32, [_P, C.c_uint32, C.c_uint64, _P, _P, C.POINTER(qe_tape), _P, C.POINTER(qe_tape), _P, _P, _P]),
    "qe_gemm_fp8_group": (C.c_int32, [C.POINTER(qe_gemm_desc), C.c_uint32, _P, _P]),
    "qe_run_together_host": (C.c_int32, [_P, C.POINTER(qe_action), C.c_uint32, _P, C.c_uint64, _P]),
    "qe_plan_rounds": (C.c_int32, [C.POINTER(qe_step_action), C.c_uint32, C.c_uint32, C.c_uint32, C.POINTER(C.c_uint32),
                                   C.POINTER(C.c_uint32), C.c_uint32, C.c_uint32, C.POINTER(C.c_uint32), C.POINTER(C.c_uint32)]),
    "qe_run_together": (C.c_int32, [_P, C.POINTER(qe_action), C.c_uint32, _P, C.c_uint64, _P]),
    "qe_forward_chain": (C.c_int32, [C.POINTER(_P), C.c_uint32, C.c_uint32, C.c_uint64, _P, _P, _P, C.POINTER(qe_tape)]),
    "qe_backward_dI_chain": (C.c_int32, [C.POINTER(_P), C.POINTER(qe_tape), C.c_uint32, _P, _P, _P]),
    "qe_backward_dW_arena": (C.c_int32, [_P, C.POINTER(qe_tape), _P, C.c_uint64, C.c_uint64, C.c_uint32, _P]),
    "qe_arena_finalize": (C.c_int32, [_P, _P, C.c_uint64, C.c_uint64, C.c_uint32, _P, C.c_uint64, C.c_uint64, _P]),
    "qe_arena_reduce": (C.c_int32, [_P, C.c_uint64, C.c_uint32, _P, _P]),
    "qe_backward_dW_multi": (C.c_int32, [C.POINTER(_P), C.POINTER(qe_tape), C.c_uint32, _P, C.c_uint64,
                                         C.POINTER(C.c_uint64), _P]),
    "qe_step_run": (C.c_int32, [_P, C.POINTER(_P), C.c_uint32, C.POINTER(qe_step_action), C.c_uint32, C.c_uint32,
                                C.POINTER(qe_step_io), _P, C.c_uint64, C.POINTER(C.c_uint64), _P, _P]),
    "qe_optimizer_boundary": (C.c_int32, [_P, C.c_uint32]),
    "qe_optimizer_boundary_all": (C.c_int32, [C.POINTER(_P), C.c_uint32, C.c_uint32]),
    "qe_contract_boundary_check": (C.c_int32, [_P, C.c_uint32]),
    "qe_scale_commit": (C.c_int32, [_P, C.c_uint32, _P, _P]),
    "qe_abort_step": (C.c_int32, [_P]),
    "qe_arena_rebuild": (C.c_int32, [_P]),
    "qe_invalidate_cache": (C.c_int32, [_P]),
    "qe_next_slot": (C.c_int32, [_P, C.POINTER(C.c_uint32)]),
    "qe_get_state": (C.c_int32, [_P, C.POINTER(qe_state_view), _P, _P]),
    "qe_read_fp8": (C.c_int32, [_P, C.c_uint32, C.c_uint32, _P, C.c_uint64]),
    "qe_state_bytes": (C.c_int32, [_P, C.POINTER(C.c_uint64)]),
    "qe_state_save": (C.c_int32, [_P, _P, C.c_uint64]),
    "qe_state_load": (C.c_int32, [_P, _P, C.c_uint64]),
    "qe_get_stats": (C.c_int32, [_P, C.POINTER(qe_stats)]),
    "qe_quantize": (C.c_int32, [_P, C.c_uint32, C.c_uint32, _P, C.c_uint32, _P, _P, _P, _P]),
    "qe_amax": (C.c_int32, [_P, C.c_uint64, _P, _P, _P]),
    "qe_amax_partials": (C.c_uint32, []),
    "qe_accumulate": (C.c_int32, [_P, _P, C.c_uint64, C.c_int32, _P]),
    "qe_gemm_fp8": (C.c_int32, [_P, C.c_uint32, _P, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint32, _P, _P, _P, C.c_uint32, _P, _P, _P]),
    "qe_gemm_fp8_ex": (C.c_int32, [_P, C.c_uint32, C.c_uint32, _P, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint32, _P, _P, _P, C.c_uint32, _P, _P, _P]),
    "qe_gemm_fp8_staged_noalloc": (C.c_int32, [_P, C.c_uint32, _P, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint32, _P, _P, _P, C.c_int32, _P, _P]),
    "qe_noalloc_staging_elems": (C.c_uint64, []),
    "qe_last_error": (C.c_char_p, []),
    "qe_status_name": (C.c_char_p, [C.c_int32]),
    "qe_abi_version": (C.c_uint32, []),
}
for _name, (_res, _args) in _SIGNATURES.items():
    _fn = getattr(lib, _name)  # AttributeError here = the library does not export what the header declares
    _fn.restype = _res
    _fn.argtypes = _args


class QEError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        name = lib.qe_status_name(status).decode()
        self.code = name[len("QE_ERR_"):] if name.startswith("QE_ERR_") else name
        super().__init__(lib.qe_last_error().decode() or name)


def _check(status: int) -> None:
    if status != 0:
        raise QEError(status)


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch

        return torch.cuda.current_stream().cuda_stream or None
    return stream or None


# ---------------------------------------------------------------------------------------- contract core (host only)
class Contract:
    """qe_contract_* with check+commit exposed separately; no CUDA involved."""

    def __init__(self, slots, stage=0, unit=0, inv=0, registry=None):
        self.h = _P()
        self.registry = registry
        _check(lib.qe_contract_create(slots, stage, unit, inv, registry.h if registry else None, C.byref(self.h)))

    def __del__(self):
        if getattr(self, "h", None):
            lib.qe_contract_destroy(self.h)
            self.h = None

    def forward_check(self, mb, gen):
        r, p = C.c_int32(), C.c_uint32()
        _check(lib.qe_contract_forward_check(self.h, mb, gen, C.byref(r), C.byref(p)))
        return bool(r.value), p.value

    def forward_commit(self, mb) -> qe_tape:
        t = qe_tape()
        _check(lib.qe_contract_forward_commit(self.h, mb, C.byref(t)))
        return t

    def dI_check(self, tape):
        _check(lib.qe_contract_dI_check(self.h, C.byref(tape)))

    def dI_commit(self, tape):
        _check(lib.qe_contract_dI_commit(self.h, C.byref(tape)))

    def dW_check(self, tape, dest_addr, dest_elems, offset, slice_elems) -> bool:
        a = C.c_int32()
        _check(lib.qe_contract_dW_check(self.h, C.byref(tape), dest_addr, dest_elems, offset, slice_elems, C.byref(a)))
        return bool(a.value)

    def dW_commit(self, tape, dest_addr, offset, slice_elems):
        _check(lib.qe_contract_dW_commit(self.h, C.byref(tape), dest_addr, offset, slice_elems))

    def boundary(self, expected):
        _check(lib.qe_contract_boundary(self.h, expected))

    def boundary_check(self, expected):
        _check(lib.qe_contract_boundary_check(self.h, expected))

    def abort(self):
        _check(lib.qe_contract_abort(self.h))

    def rebuild(self):
        _check(lib.qe_contract_rebuild(self.h))

    def invalidate_cache(self):
        _check(lib.qe_contract_invalidate_cache(self.h))

    def checkpoint_check(self):
        _check(lib.qe_contract_checkpoint_check(self.h))

    def restore(self, e_W):
        _check(lib.qe_contract_restore(self.h, e_W))

    def get(self) -> dict:
        v = qe_contract_view()
        _check(lib.qe_contract_get(self.h, C.byref(v)))
        return contract_view_to_dict(v)


class Registry:
    def __init__(self):
        self.h = _P()
        _check(lib.qe_registry_create(C.byref(self.h)))

    def __del__(self):
        if getattr(self, "h", None):
            lib.qe_registry_destroy(self.h)
            self.h = None


def contract_view_to_dict(v: qe_contract_view) -> dict:
    slots = []
    for p in range(v.slots):
        s = v.slot[p]
        k = s.key
        slots.append({"gen": s.gen, "live": bool(s.live), "bits": s.bits,
                      "key": (k.epoch, k.stage, k.mb, k.unit, k.inv) if s.live else None})
    return {"e_W": v.e_W, "e_C": v.e_C, "token": v.token, "write_mask": v.write_mask,
            "fwd_in_epoch": v.fwd_in_epoch, "aborted": bool(v.aborted), "slots": slots}


# ---------------------------------------------------------------------------------------- layer API
class Context:
    def __init__(self, exec_mode=EAGER, device=0, exec_stream=None, overlap_dw=False, unsafe_one_way=False, step_window=0):
        """exec_stream: a cudaStream_t (int) the context should execute on, or None for a context-owned stream.
        overlap_dw: QE_CTX_OVERLAP_DW (dW actions on a second stream, joined at the optimizer boundary)."""
        cfg = qe_ctx_config(exec_mode=exec_mode, device=device, exec_stream=exec_stream, flags=(OVERLAP_DW if overlap_dw else 0) | (UNSAFE_ONE_WAY_HANDOFF if unsafe_one_way else 0), step_window=step_window)
        self.h = _P()
        _check(lib.qe_ctx_create(C.byref(cfg), C.byref(self.h)))
        self.exec_mode = exec_mode

    def stats(self) -> dict:
        s = qe_stats()
        _check(lib.qe_get_stats(self.h, C.byref(s)))
        return s.asdict()

    def close(self):
        if getattr(self, "h", None):
            lib.qe_ctx_destroy(self.h)
            self.h = None

    def __del__(self):
        self.close()


class Layer:
    """One FP8 delayed-scaling linear.  Holds the torch-allocated workspace and the weight tensor alive."""

    def __init__(self, ctx: Context, T, K, N, H, margin, slots, weight, stage=0, unit=0, inv=0, host_io=False):
        import torch

        assert weight.dtype == torch.bfloat16 and weight.is_cuda and weight.is_contiguous() and tuple(weight.shape) == (N, K)
        self.ctx, self.T, self.K, self.N, self.H, self.P = ctx, T, K, N, H, slots
        self.weight = weight
        self.cfg = qe_layer_config(T=T, K=K, N=N, history_len=H, margin=margin, slots=slots, stage=stage, unit=unit,
                                   inv=inv, host_io=int(host_io), weight_dev=weight.data_ptr())
        nbytes = C.c_uint64()
        _check(lib.qe_layer_workspace_bytes(C.byref(self.cfg), C.byref(nbytes)))
        self.workspace = torch.empty(nbytes.value + 256, dtype=torch.uint8, device=weight.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        self.h = _P()
        # torch's allocator is stream-ordered: the block may still be written by earlier work of the current stream,
        # while the library initialises it on the context's execution stream
        torch.cuda.current_stream(weight.device).synchronize()
        _check(lib.qe_layer_create(ctx.h, C.byref(self.cfg), base, nbytes.value, C.byref(self.h)))

    # the five calls of the path
    def forward(self, mb, gen, x, y, stream=None) -> qe_tape:
        t = qe_tape()
        _check(lib.qe_forward(self.h, mb, gen, _ptr(x), _ptr(y), _stream(stream), C.byref(t)))
        return t

    def forward_host(self, mb, gen, x_host, y_host, stream=None) -> qe_tape:
        """x_host / y_host: CPU tensors (pinned for asynchronous copies); y_host may be None."""
        t = qe_tape()
        _check(lib.qe_forward_host(self.h, mb, gen, _ptr(x_host), _ptr(y_host), _stream(stream), C.byref(t)))
        return t

    def backward_dI_host(self, tape, dy_host, dx_host, stream=None):
        _check(lib.qe_backward_dI_host(self.h, C.byref(tape), _ptr(dy_host), _ptr(dx_host), _stream(stream)))

    def backward_dI(self, tape, dy, dx, stream=None):
        _check(lib.qe_backward_dI(self.h, C.byref(tape), _ptr(dy), _ptr(dx), _stream(stream)))

    def backward_dW(self, tape, grad_buf, offset, stream=None):
        _check(lib.qe_backward_dW(self.h, C.byref(tape), _ptr(grad_buf), grad_buf.numel(), offset, _stream(stream)))

    def backward_dW_staged(self, tape, grad_buf, offset, temp, stream=None):
        _check(lib.qe_backward_dW_staged(self.h, C.byref(tape), _ptr(grad_buf), grad_buf.numel(), offset, _ptr(temp), _stream(stream)))

    def backward_dW_arena(self, tape, arena, layer_offset, microbatches, stream=None):
        _check(lib.qe_backward_dW_arena(self.h, C.byref(tape), _ptr(arena), arena.numel(), layer_offset, microbatches, _stream(stream)))

    def arena_finalize(self, arena, layer_offset, microbatches, grad_buf, offset, stream=None):
        _check(lib.qe_arena_finalize(self.h, _ptr(arena), arena.numel(), layer_offset, microbatches, _ptr(grad_buf),
                                     grad_buf.numel(), offset, _stream(stream)))

    def optimizer_boundary(self, expected):
        _check(lib.qe_optimizer_boundary(self.h, expected))

    def scale_commit(self, cls, amax_dev, stream=None):
        _check(lib.qe_scale_commit(self.h, cls, _ptr(amax_dev), _stream(stream)))

    def abort_step(self):
        _check(lib.qe_abort_step(self.h))

    def arena_rebuild(self):
        _check(lib.qe_arena_rebuild(self.h))

    def invalidate_cache(self):
        _check(lib.qe_invalidate_cache(self.h))

    def next_slot(self) -> int:
        p = C.c_uint32()
        _check(lib.qe_next_slot(self.h, C.byref(p)))
        return p.value

    def state(self) -> dict:
        """Same shape as the oracle's state(): bit-comparable."""
        v = qe_state_view()
        win = np.zeros(4 * self.H, np.float32)
        sinv = np.zeros(2 * self.P, np.float32)
        _check(lib.qe_get_state(self.h, C.byref(v), win.ctypes.data, sinv.ctypes.data))
        d = contract_view_to_dict(v.contract)
        d["classes"] = {
            CLASS_NAMES[c]: {
                "window": win[c * self.H:(c + 1) * self.H].copy(),
                "scale": np.float32(v.cls[c].scale),
                "scale_inv": np.float32(v.cls[c].scale_inv),
                "count": v.cls[c].count,
            }
            for c in range(4)
        }
        d["cache_sinv_W"] = np.float32(v.cache_sinv_W)
        d["device_status"] = v.device_status
        d["device_token"] = v.device_token
        d["slot_sinv_X"] = sinv[: self.P].copy()
        d["slot_sinv_G"] = sinv[self.P:].copy()
        return d

    def state_save(self) -> bytes:
        n = C.c_uint64()
        _check(lib.qe_state_bytes(self.h, C.byref(n)))
        buf = (C.c_ubyte * n.value)()
        _check(lib.qe_state_save(self.h, buf, n.value))
        return bytes(buf)

    def state_load(self, payload: bytes):
        buf = (C.c_ubyte * len(payload)).from_buffer_copy(payload)
        _check(lib.qe_state_load(self.h, buf, len(payload)))

    def read_fp8(self, which: int, slot: int = 0) -> np.ndarray:
        shape = {0: (self.T, self.K), 1: (self.K, self.T), 2: (self.T, self.N), 3: (self.N, self.T),
                 4: (self.N, self.K), 5: (self.K, self.N)}[which]
        out = np.empty(shape, np.uint8)
        _check(lib.qe_read_fp8(self.h, which, slot, out.ctypes.data, out.size))
        return out

    def close(self):
        if getattr(self, "h", None):
            lib.qe_layer_destroy(self.h)
            self.h = None

    def __del__(self):
        self.close()


# ---------------------------------------------------------------------------------------- standalone kernels
def qe_quantize(x, scale_dev, fmt, q, qT=None, amax_dev=None, stream=None):
    rows, cols = x.shape
    _check(lib.qe_quantize(_ptr(x), rows, cols, _ptr(scale_dev), fmt, _ptr(q), _ptr(qT), _ptr(amax_dev), _stream(stream)))


def qe_amax_partials() -> int:
    return lib.qe_amax_partials()


def qe_amax(x, partials_dev, amax_dev, stream=None):
    _check(lib.qe_amax(_ptr(x), x.numel(), _ptr(partials_dev), _ptr(amax_dev), _stream(stream)))


def qe_accumulate(dst, src, accumulate: bool, stream=None):
    _check(lib.qe_accumulate(_ptr(dst), _ptr(src), dst.numel(), int(accumulate), _stream(stream)))


def qe_gemm_fp8(a, a_fmt, b, b_fmt, alpha_a_dev, alpha_b_dev, d, out_kind, amax_dev=None, status_dev=None, stream=None):
    M, Kc = a.shape
    Nn, Kc2 = b.shape
    assert Kc == Kc2
    _check(lib.qe_gemm_fp8(_ptr(a), a_fmt, _ptr(b), b_fmt, M, Nn, Kc, _ptr(alpha_a_dev), _ptr(alpha_b_dev), _ptr(d),
                           out_kind, _ptr(amax_dev), _ptr(status_dev), _stream(stream)))


def qe_gemm_fp8_ex(a, a_fmt, a_mn, b, b_fmt, b_mn, alpha_a_dev, alpha_b_dev, d, out_kind, amax_dev=None, status_dev=None, stream=None):
    """a is [M, Kc] (a_mn False) or [Kc, M] (a_mn True); likewise b with Nn."""
    M, Kc = (a.shape[1], a.shape[0]) if a_mn else a.shape
    Nn = b.shape[1] if b_mn else b.shape[0]
    _check(lib.qe_gemm_fp8_ex(_ptr(a), a_fmt, int(a_mn), _ptr(b), b_fmt, int(b_mn), M, Nn, Kc, _ptr(alpha_a_dev), _ptr(alpha_b_dev),
                              _ptr(d), out_kind, _ptr(amax_dev), _ptr(status_dev), _stream(stream)))


def qe_gemm_fp8_staged_noalloc(a, a_fmt, b, b_fmt, alpha_a_dev, alpha_b_dev, dst, accumulate: bool, status_dev, stream=None):
    """Copied-gradient step with the library's built-in staging area (no device allocation anywhere underneath):
    for callers that may not allocate where they run.  dst is FP32 [M, Nn] with M*Nn <= qe_noalloc_staging_elems()."""
    M, Kc = a.shape
    Nn, Kc2 = b.shape
    assert Kc == Kc2
    _check(lib.qe_gemm_fp8_staged_noalloc(_ptr(a), a_fmt, _ptr(b), b_fmt, M, Nn, Kc, _ptr(alpha_a_dev), _ptr(alpha_b_dev),
                                          _ptr(dst), int(accumulate), _ptr(status_dev), _stream(stream)))


def qe_noalloc_staging_elems() -> int:
    return lib.qe_noalloc_staging_elems()


ACT = {"F": 0, "dI": 1, "dW": 2}


def forward_dI_pair(layer_f, mb, gen, x, y, layer_b, tape_b, dy, dx, stream=None):
    """qe_forward_dI_pair: F of layer_f and dI of layer_b (another layer) in one call; returns layer_f's tape."""
    t = qe_tape()
    _check(lib.qe_forward_dI_pair(layer_f.h, mb, gen, _ptr(x), _ptr(y), C.byref(t), layer_b.h, C.byref(tape_b),
                                  _ptr(dy), _ptr(dx), _stream(stream)))
    return t


def qe_gemm_fp8_group(problems, status, stream=None):
    """problems: 2..4 tuples (a, a_format, a_mn, b, b_format, b_mn, alpha_a, alpha_b, d, out_kind, amax or None);
    shapes are taken from the tensors (MN-major operands are [Kc, rows])."""
    n = len(problems)
    arr = (qe_gemm_desc * n)()
    for i, (a, af, amn, b, bf, bmn, sa, sb, d, kind, amax) in enumerate(problems):
        M, Nn = d.shape
        Kc = a.shape[0] if amn else a.shape[1]
        arr[i] = qe_gemm_desc(_ptr(a), _ptr(b), _ptr(d), _ptr(sa), _ptr(sb), _ptr(amax), af, int(amn), bf, int(bmn), M, Nn, Kc, kind)
    _check(lib.qe_gemm_fp8_group(arr, n, _ptr(status), _stream(stream)))


def plan_rounds(actions, n_layers, microbatches, slots, window, max_group=8, live_now=None):
    """qe_plan_rounds (host only).  actions: (kind name, layer, mb) triples; returns the rounds as lists of triples."""
    n = len(actions)
    arr = (qe_step_action * n)(*[qe_step_action(ACT[k], l, m, 0) for k, l, m in actions])
    sl = (C.c_uint32 * n_layers)(*([slots] * n_layers if isinstance(slots, int) else slots))
    lv = (C.c_uint32 * n_layers)(*live_now) if live_now is not None else None
    rnd = (C.c_uint32 * n)()
    nr = C.c_uint32()
    _check(lib.qe_plan_rounds(arr, n, n_layers, microbatches, sl, lv, window, max_group, rnd, C.byref(nr)))
    out = [[] for _ in range(nr.value)]
    for i, a in enumerate(actions):
        out[rnd[i]].append(tuple(a))
    return out


def run_together(ctx, actions, grad_buf=None, stream=None, host=False):
    """qe_run_together (host=True: qe_run_together_host, x / y / dy / dx are pinned host tensors, y / dx may be None).  actions: ("F", layer, mb, gen, x, y) | ("dI", layer, tape, dy, dx) | ("dW", layer, tape, offset).
    Returns the tapes of the F actions, in order."""
    n = len(actions)
    arr = (qe_action * n)()
    new_tapes = []
    for i, a in enumerate(actions):
        if a[0] == "F":
            _, L, mb, gen, x, y = a
            t = qe_tape()
            new_tapes.append(t)
            arr[i] = qe_action(ACT["F"], mb, gen, L.h, _ptr(x), _ptr(y), C.pointer(t), 0)
        elif a[0] == "dI":
            _, L, tape, dy, dx = a
            arr[i] = qe_action(ACT["dI"], 0, 0, L.h, _ptr(dy), _ptr(dx), C.pointer(tape), 0)
        else:
            _, L, tape, off = a
            arr[i] = qe_action(ACT["dW"], 0, 0, L.h, None, None, C.pointer(tape), off)
    fn = lib.qe_run_together_host if host else lib.qe_run_together
    _check(fn(ctx.h, arr, n, _ptr(grad_buf), grad_buf.numel() if grad_buf is not None else 0, _stream(stream)))
    return new_tapes


def optimizer_boundary_all(layers, expected):
    """qe_optimizer_boundary_all: the boundary of every layer of a stage (one context) with one drain and one read."""
    n = len(layers)
    hs = (_P * n)(*[L.h for L in layers])
    _check(lib.qe_optimizer_boundary_all(hs, n, expected))


def forward_chain(layers, mb, gen, x, y, stream=None):
    """qe_forward_chain: F of directly chained linears with FP8 hand-off; returns one tape per layer."""
    n = len(layers)
    hs = (_P * n)(*[L.h for L in layers])
    tapes = (qe_tape * n)()
    _check(lib.qe_forward_chain(hs, n, mb, gen, _ptr(x), _ptr(y), _stream(stream), tapes))
    out = []
    for t in tapes:  # copies that outlive the ctypes array
        c = qe_tape()
        C.memmove(C.byref(c), C.byref(t), C.sizeof(qe_tape))
        out.append(c)
    return out


def backward_dI_chain(layers, tapes, dy, dx, stream=None):
    n = len(layers)
    hs = (_P * n)(*[L.h for L in layers])
    ts = (qe_tape * n)(*tapes)
    _check(lib.qe_backward_dI_chain(hs, ts, n, _ptr(dy), _ptr(dx), _stream(stream)))


def qe_arena_reduce(views, M, dst, stream=None):
    """views: bf16 tensor of M contiguous views; dst: FP32 tensor of one view's size."""
    _check(lib.qe_arena_reduce(_ptr(views), views.numel() // M, M, _ptr(dst), _stream(stream)))


def backward_dW_multi(layers, tapes, grad_buf, offsets, stream=None):
    """qe_backward_dW_multi: the weight gradients of several layers (distinct, one context) in one call."""
    n = len(layers)
    hs = (_P * n)(*[L.h for L in layers])
    ts = (qe_tape * n)(*tapes)
    offs = (C.c_uint64 * n)(*offsets)
    _check(lib.qe_backward_dW_multi(hs, ts, n, _ptr(grad_buf), grad_buf.numel(), offs, _stream(stream)))


class StepPlan:
    """Arguments of qe_step_run marshalled once: a list of (kind, layer index, microbatch) over `layers`, the device
    tensors of every (layer, microbatch) unit, the flat gradient buffer with per-layer element offsets, and the
    optional temporary of the copied-gradient path.  run() is one C call."""

    def __init__(self, ctx: Context, layers, actions, microbatches, X, Y, dY, dX, grad_buf, offsets, temp=None):
        self.ctx, self.layers, self.M = ctx, list(layers), microbatches
        self.keep = (X, Y, dY, dX, grad_buf, temp)  # the tensors must outlive the plan
        n = len(self.layers)
        self.c_layers = (_P * n)(*[L.h for L in self.layers])
        self.c_actions = (qe_step_action * len(actions))(*[qe_step_action(ACT[k], l, m, 0) for k, l, m in actions])
        self.c_io = (qe_step_io * (n * microbatches))()
        for l in range(n):
            for m in range(microbatches):
                self.c_io[l * microbatches + m] = qe_step_io(_ptr(X[m][l]), _ptr(Y[m][l]), _ptr(dY[m][l]), _ptr(dX[m][l]))
        self.c_offsets = (C.c_uint64 * n)(*offsets)
        self.grad, self.temp = grad_buf, temp

    def run(self, stream=None):
        _check(lib.qe_step_run(self.ctx.h, self.c_layers, len(self.layers), self.c_actions, len(self.c_actions), self.M,
                               self.c_io, _ptr(self.grad), self.grad.numel(), self.c_offsets, _ptr(self.temp), _stream(stream)))
