"""Thin Python binding of the C ABI declared in include/apms.h.

Argument marshalling only: every step of the path runs in the CUDA library.  The
module-level functions carry the C names; `Context` bundles a handle with a
torch-allocated workspace and stream (PyTorch is used for device memory and streams
only).  There is no CPU fallback: if the shared library is missing or no CUDA device
is present, the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("APMS_LIBRARY") or os.path.join(HERE, "libapms.so")   # override: another build of the same ABI

OK, ERR_INVALID_ARG, ERR_BAD_STATE, ERR_CUDA, ERR_OOM, ERR_TIMEOUT, ERR_BOUNDS = range(7)
PHASE_CREATED, PHASE_WARMUP, PHASE_COMPRESSED = range(3)
(STATE_X, STATE_V, STATE_M, STATE_WORKER_ERR, STATE_WORKER_BITS, STATE_WORKER_SCALES,
 STATE_SERVER_ERR, STATE_SERVER_BITS, STATE_SERVER_SCALES) = range(9)
KERNEL_WARMUP_ADAM, KERNEL_WORKER, KERNEL_SERVER, KERNEL_APPLY = range(4)
KERNEL_NAMES = ("warmup_adam", "worker", "server", "apply")
TEAM_AUTO, TEAM_CTA, TEAM_WARP, TEAM_STAGED = range(4)
GRAD_F32, GRAD_BF16, GRAD_F16 = range(3)
SCALE_L2, SCALE_L1_MEAN = range(2)
VARIANT_MOMENTUM, VARIANT_GRADIENT = range(2)
COMPRESSOR_ONEBIT, COMPRESSOR_TOPK = range(2)
MAX_WORKERS = 64
NOALLOC_MAX_TILES = 16384

_FP = C.POINTER(C.c_float)
_FPP = C.POINTER(_FP)

# name -> (restype, argtypes); mirrors include/apms.h one to one
SIGNATURES = {
    "apms_workspace_bytes": (C.c_size_t, [C.c_int64, C.c_int, C.c_int64]),
    "apms_create": (C.c_int, [C.POINTER(C.c_void_p), C.c_int64, C.c_int, C.c_float, C.c_float,
                              C.c_float, C.c_float, C.c_int64]),
    "apms_bind": (C.c_int, [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "apms_set_params": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int]),
    "apms_set_lr": (C.c_int, [C.c_void_p, C.c_float]),
    "apms_warmup_step": (C.c_int, [C.c_void_p, C.POINTER(C.c_void_p)]),
    "apms_freeze_v": (C.c_int, [C.c_void_p]),
    "apms_compressed_step": (C.c_int, [C.c_void_p, C.POINTER(C.c_void_p)]),
    "apms_compressed_step_host": (C.c_int, [C.c_void_p, C.POINTER(C.c_void_p), C.c_void_p]),
    "apms_warmup_step_typed": (C.c_int, [C.c_void_p, C.POINTER(C.c_void_p), C.c_int]),
    "apms_compressed_step_typed": (C.c_int, [C.c_void_p, C.POINTER(C.c_void_p), C.c_int]),
    "apms_compressed_step_host_typed": (C.c_int, [C.c_void_p, C.POINTER(C.c_void_p), C.c_int, C.c_void_p]),
    "apms_worker_phase": (C.c_int, [C.c_void_p, C.POINTER(C.c_void_p), C.c_int]),
    "apms_worker_phase_range": (C.c_int, [C.c_void_p, C.POINTER(C.c_void_p), C.c_int, C.c_int64, C.c_int64]),
    "apms_get_message": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_void_p), C.POINTER(C.c_void_p)]),
    "apms_server_phase": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_int, C.c_int64, C.c_int64]),
    "apms_apply_phase": (C.c_int, [C.c_void_p]),
    "apms_topk_values_per_chunk": (C.c_int64, [C.c_void_p]),
    "apms_topk_route_counts": (C.c_int, [C.c_void_p, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]),
    "apms_topk_pack_values": (C.c_int, [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_void_p]),
    "apms_topk_server_scratch_bytes": (C.c_size_t, [C.c_void_p, C.c_int, C.c_int64, C.c_int64]),
    "apms_topk_server_phase": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_int, C.c_int64, C.c_int64,
                                         C.c_void_p, C.c_size_t]),
    "apms_topk_put_server_range": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64]),
    "apms_server_phase_rows": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_int64]),
    "apms_put_server_range": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64]),
    "apms_message_offsets": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]),
    "apms_ipc_export": (C.c_int, [C.c_void_p, C.c_void_p]),
    "apms_ipc_open": (C.c_int, [C.c_void_p, C.POINTER(C.c_void_p)]),
    "apms_ipc_close": (C.c_int, [C.c_void_p]),
    "apms_get_params": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int]),
    "apms_get_state": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_void_p]),
    "apms_get_state_slice": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_int64, C.c_int64, C.c_void_p]),
    "apms_set_state": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_void_p]),
    "apms_restore": (C.c_int, [C.c_void_p, C.c_int, C.c_int]),
    "apms_schedule_lr": (C.c_float, [C.c_void_p, C.c_int64]),
    "apms_set_schedule": (C.c_int, [C.c_void_p, C.c_void_p]),
    "apms_step": (C.c_int, [C.c_void_p, C.POINTER(C.c_void_p), C.c_int]),
    "apms_get_step": (C.c_int64, [C.c_void_p]),
    "apms_set_step": (C.c_int, [C.c_void_p, C.c_int64]),
    "apms_error_norms": (C.c_int, [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_double)]),
    "apms_get_phase": (C.c_int, [C.c_void_p]),
    "apms_get_t": (C.c_int, [C.c_void_p]),
    "apms_set_scale_kind": (C.c_int, [C.c_void_p, C.c_int]),
    "apms_set_variant": (C.c_int, [C.c_void_p, C.c_int]),
    "apms_set_compressor": (C.c_int, [C.c_void_p, C.c_int, C.c_double]),
    "apms_uncompressed_step_typed": (C.c_int, [C.c_void_p, C.POINTER(C.c_void_p), C.c_int]),
    "apms_set_team_mode": (C.c_int, [C.c_void_p, C.c_int]),
    "apms_build_is_checked": (C.c_int, []),
    "apms_selftest_bounds": (C.c_int, [C.c_void_p]),
    "apms_set_guard_bytes": (C.c_int, [C.c_size_t]),
    "apms_check_guards": (C.c_int, [C.c_void_p, C.POINTER(C.c_int64)]),
    "apms_set_timing": (C.c_int, [C.c_void_p, C.c_int]),
    "apms_kernel_time": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_int64)]),
    "apms_selftest_wait_report": (C.c_int, [C.c_void_p, C.c_int]),
    "apms_launch_count": (C.c_int64, [C.c_void_p]),
    "apms_last_error": (C.c_char_p, [C.c_void_p]),
    "apms_destroy": (None, [C.c_void_p]),
    "apms_compress_noalloc": (C.c_int, [C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p]),
}

_lib: Optional[C.CDLL] = None


class ApmsError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"apms status {status}: {message}")
        self.status = status


def load() -> C.CDLL:
    """Load paper_2008_11343_b200/libapms.so (built by build.py); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is not built; run `python -m paper_2008_11343_b200.build` "
                              "(there is no fallback path)")
        lib = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def _ptr_array(ptrs: Sequence[int]):
    return (C.c_void_p * len(ptrs))(*ptrs)


# --- functions with the C names ------------------------------------------------------------

def apms_workspace_bytes(d: int, n: int, chunk: int) -> int:
    return int(load().apms_workspace_bytes(d, n, chunk))


def apms_create(d, n, beta1, beta2, eps, lr, chunk) -> int:
    h = C.c_void_p()
    st = load().apms_create(C.byref(h), d, n, beta1, beta2, eps, lr, chunk)
    if st != OK:
        raise ApmsError(st, load().apms_last_error(None).decode())
    return h.value


def _check(h, st):
    if st != OK:
        raise ApmsError(st, load().apms_last_error(h).decode())


def apms_bind(h, workspace_ptr: int, nbytes: int, stream: int):
    _check(h, load().apms_bind(h, workspace_ptr, nbytes, stream))


def apms_set_params(h, x0_ptr: int, src_is_device: bool):
    _check(h, load().apms_set_params(h, x0_ptr, int(src_is_device)))


def apms_set_lr(h, lr: float):
    _check(h, load().apms_set_lr(h, lr))


def apms_warmup_step(h, grad_ptrs: Sequence[int]):
    _check(h, load().apms_warmup_step(h, _ptr_array(grad_ptrs)))


def apms_freeze_v(h):
    _check(h, load().apms_freeze_v(h))


def apms_compressed_step(h, grad_ptrs: Sequence[int]):
    _check(h, load().apms_compressed_step(h, _ptr_array(grad_ptrs)))


def apms_compressed_step_host(h, grad_host_ptrs: Sequence[int], x_out_host_ptr: Optional[int]):
    _check(h, load().apms_compressed_step_host(h, _ptr_array(grad_host_ptrs), x_out_host_ptr))


def apms_warmup_step_typed(h, grad_ptrs: Sequence[int], grad_type: int):
    _check(h, load().apms_warmup_step_typed(h, _ptr_array(grad_ptrs), grad_type))


def apms_compressed_step_typed(h, grad_ptrs: Sequence[int], grad_type: int):
    _check(h, load().apms_compressed_step_typed(h, _ptr_array(grad_ptrs), grad_type))


def apms_compressed_step_host_typed(h, grad_host_ptrs: Sequence[int], grad_type: int, x_out_host_ptr: Optional[int]):
    _check(h, load().apms_compressed_step_host_typed(h, _ptr_array(grad_host_ptrs), grad_type, x_out_host_ptr))


def apms_worker_phase(h, grad_ptrs: Sequence[int], grad_type: int):
    _check(h, load().apms_worker_phase(h, _ptr_array(grad_ptrs), grad_type))


def apms_worker_phase_range(h, grad_ptrs: Sequence[int], grad_type: int, chunk_begin: int, chunk_end: int):
    _check(h, load().apms_worker_phase_range(h, _ptr_array(grad_ptrs), grad_type, chunk_begin, chunk_end))


def apms_topk_values_per_chunk(h) -> int:
    return int(load().apms_topk_values_per_chunk(h))


def apms_topk_route_counts(h):
    """(worker routes, server routes): 6 counters each, reset by the call."""
    wr, sr = (C.c_int64 * 6)(), (C.c_int64 * 6)()
    _check(h, load().apms_topk_route_counts(h, wr, sr))
    return list(wr), list(sr)


def apms_topk_pack_values(h, worker: int, chunk_begin: int, chunk_end: int, vals_ptr: int):
    _check(h, load().apms_topk_pack_values(h, worker, chunk_begin, chunk_end, vals_ptr))


def apms_topk_server_scratch_bytes(h, rows: int, chunk_begin: int, chunk_end: int) -> int:
    return int(load().apms_topk_server_scratch_bytes(h, rows, chunk_begin, chunk_end))


def apms_topk_server_phase(h, mask_rows_ptr: int, row_words: int, val_rows_ptr: int, row_vals: int, rows: int,
                           chunk_begin: int, chunk_end: int, scratch_ptr: int, scratch_bytes: int):
    _check(h, load().apms_topk_server_phase(h, mask_rows_ptr, row_words, val_rows_ptr, row_vals, rows, chunk_begin, chunk_end,
                                            scratch_ptr, scratch_bytes))


def apms_topk_put_server_range(h, mask_words_ptr: int, vals_ptr: int, chunk_begin: int, chunk_end: int):
    _check(h, load().apms_topk_put_server_range(h, mask_words_ptr, vals_ptr, chunk_begin, chunk_end))


def apms_get_message(h, worker: int):
    """(device address of the sign words, device address of the scales) of worker `worker` (-1: the server)."""
    bits, scales = C.c_void_p(), C.c_void_p()
    _check(h, load().apms_get_message(h, worker, C.byref(bits), C.byref(scales)))
    return bits.value, scales.value


def apms_server_phase(h, bits_rows_ptr: int, row_words: int, scale_rows_ptr: int, row_scales: int, rows: int,
                      chunk_begin: int, chunk_end: int):
    _check(h, load().apms_server_phase(h, bits_rows_ptr, row_words, scale_rows_ptr, row_scales, rows,
                                       chunk_begin, chunk_end))


def apms_apply_phase(h):
    _check(h, load().apms_apply_phase(h))


def apms_server_phase_rows(h, bits_row_ptrs: Sequence[int], scale_row_ptrs: Sequence[int], chunk_begin: int, chunk_end: int):
    rows = len(bits_row_ptrs)
    assert len(scale_row_ptrs) == rows
    barr = (C.c_void_p * rows)(*bits_row_ptrs)
    sarr = (C.c_void_p * rows)(*scale_row_ptrs)
    _check(h, load().apms_server_phase_rows(h, barr, sarr, rows, chunk_begin, chunk_end))


def apms_put_server_range(h, dst_bits_ptr: int, dst_scales_ptr: int, chunk_begin: int, chunk_end: int):
    _check(h, load().apms_put_server_range(h, dst_bits_ptr, dst_scales_ptr, chunk_begin, chunk_end))


def apms_message_offsets(h, worker: int):
    b, s = C.c_size_t(), C.c_size_t()
    _check(h, load().apms_message_offsets(h, worker, C.byref(b), C.byref(s)))
    return int(b.value), int(s.value)


IPC_HANDLE_BYTES = 64


def apms_ipc_export(h) -> bytes:
    buf = C.create_string_buffer(IPC_HANDLE_BYTES)
    _check(h, load().apms_ipc_export(h, buf))
    return buf.raw


def apms_ipc_open(handle: bytes) -> int:
    assert len(handle) == IPC_HANDLE_BYTES
    base = C.c_void_p()
    st = load().apms_ipc_open(C.c_char_p(handle), C.byref(base))
    if st != OK:
        raise ApmsError(st, load().apms_last_error(None).decode())
    return int(base.value)


def apms_ipc_close(base: int):
    st = load().apms_ipc_close(C.c_void_p(base))
    if st != OK:
        raise ApmsError(st, load().apms_last_error(None).decode())


def apms_get_params(h, dst_ptr: int, dst_is_device: bool):
    _check(h, load().apms_get_params(h, dst_ptr, int(dst_is_device)))


def apms_get_state(h, which: int, worker: int, dst_host_ptr: int):
    _check(h, load().apms_get_state(h, which, worker, dst_host_ptr))


def apms_get_state_slice(h, which: int, worker: int, first: int, count: int, dst_host_ptr: int):
    _check(h, load().apms_get_state_slice(h, which, worker, first, count, dst_host_ptr))


def apms_set_state(h, which: int, worker: int, src_host_ptr: int):
    _check(h, load().apms_set_state(h, which, worker, src_host_ptr))


def apms_restore(h, t: int, phase: int):
    _check(h, load().apms_restore(h, t, phase))


class Schedule(C.Structure):
    """Mirror of the C struct apms_schedule."""
    _fields_ = [("warmup_steps", C.c_int64), ("peak_lr", C.c_float), ("lr_ramp_steps", C.c_int64),
                ("lr_decay", C.c_float), ("lr_decay_every", C.c_int64)]


def apms_schedule_lr(schedule: Schedule, step: int) -> float:
    return float(load().apms_schedule_lr(C.byref(schedule), step))


def apms_set_schedule(h, schedule: Optional[Schedule]):
    _check(h, load().apms_set_schedule(h, None if schedule is None else C.byref(schedule)))


def apms_step(h, grad_ptrs: Sequence[int], grad_type: int):
    _check(h, load().apms_step(h, _ptr_array(grad_ptrs), grad_type))


def apms_get_step(h) -> int:
    return int(load().apms_get_step(h))


def apms_set_step(h, steps: int):
    _check(h, load().apms_set_step(h, steps))


def apms_error_norms(h, n: int):
    """(worker squared norms [n], server squared norm) as Python floats."""
    w = (C.c_double * n)()
    s = C.c_double(0.0)
    _check(h, load().apms_error_norms(h, w, C.byref(s)))
    return [float(v) for v in w], float(s.value)


def apms_get_phase(h) -> int:
    return int(load().apms_get_phase(h))


def apms_get_t(h) -> int:
    return int(load().apms_get_t(h))


def apms_set_compressor(h, kind: int, topk_fraction: float = 0.01):
    _check(h, load().apms_set_compressor(h, kind, topk_fraction))


def apms_set_variant(h, variant: int):
    _check(h, load().apms_set_variant(h, variant))


def apms_uncompressed_step_typed(h, grad_ptrs: Sequence[int], grad_type: int):
    _check(h, load().apms_uncompressed_step_typed(h, _ptr_array(grad_ptrs), grad_type))


def apms_set_scale_kind(h, kind: int):
    _check(h, load().apms_set_scale_kind(h, kind))


def apms_set_team_mode(h, mode: int):
    _check(h, load().apms_set_team_mode(h, mode))


def apms_build_is_checked() -> bool:
    return bool(load().apms_build_is_checked())


def apms_selftest_bounds(h):
    _check(h, load().apms_selftest_bounds(h))


def apms_set_guard_bytes(nbytes: int):
    st = load().apms_set_guard_bytes(nbytes)
    if st != OK:
        raise ApmsError(st, load().apms_last_error(None).decode())


def apms_check_guards(h) -> int:
    """Raises ApmsError(ERR_BOUNDS) naming the array whose guard bytes changed; its .bad_offset is the workspace offset."""
    bad = C.c_int64(-1)
    st = load().apms_check_guards(h, C.byref(bad))
    if st != OK:
        err = ApmsError(st, load().apms_last_error(h).decode())
        err.bad_offset = int(bad.value)
        raise err
    return int(bad.value)


def apms_set_timing(h, enabled: bool):
    _check(h, load().apms_set_timing(h, int(enabled)))


def apms_kernel_time(h, which: int):
    ms, cnt = C.c_double(0.0), C.c_int64(0)
    _check(h, load().apms_kernel_time(h, which, C.byref(ms), C.byref(cnt)))
    return ms.value, cnt.value


def apms_selftest_wait_report(h, leave_reported: bool = False):
    _check(h, load().apms_selftest_wait_report(h, int(leave_reported)))


def apms_launch_count(h) -> int:
    return int(load().apms_launch_count(h))


def apms_last_error(h) -> str:
    return load().apms_last_error(h).decode()


def apms_destroy(h):
    load().apms_destroy(h)


def apms_compress_noalloc(z_ptr: int, d: int, chunk: int, bits_ptr: int, scales_ptr: int, stream: int = 0):
    """Sign words and chunk scales of the d floats at device address z_ptr, written to the
    caller's device buffers.  For callers that may not allocate device memory: the library
    allocates nothing here (its only scratch is a fixed 128 KiB array inside the library), so
    the shape is limited (see APMS_NOALLOC_MAX_TILES in apms.h) and calls that overlap on the
    GPU must be ordered by the caller.  Raises ApmsError with the library's message otherwise."""
    st = load().apms_compress_noalloc(z_ptr, d, chunk, bits_ptr, scales_ptr, stream or None)
    if st != OK:
        raise ApmsError(st, load().apms_last_error(None).decode())


# --- convenience wrapper: handle + torch workspace + stream ---------------------------------

class Context:
    """An apms context whose workspace is a torch CUDA tensor and whose stream is torch's.
    With library_workspace=True the library allocates the workspace itself (cudaMalloc): the form that
    apms_ipc_export needs, without the tensor views of message()."""

    def __init__(self, d: int, n: int, beta1: float, beta2: float, eps: float, lr: float, chunk: int,
                 device: str = "cuda:0", stream=None, library_workspace: bool = False):
        import torch

        if not torch.cuda.is_available():
            raise RuntimeError("apms needs a CUDA device; there is no CPU path")
        self.d, self.n, self.chunk = d, n, chunk
        self.C = (d + chunk - 1) // chunk
        self.W = (d + 31) // 32
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self._h = apms_create(d, n, beta1, beta2, eps, lr, chunk)
        self.topk = False
        nbytes = apms_workspace_bytes(d, n, chunk)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        if library_workspace:
            self.workspace = None
            apms_bind(self._h, None, 0, self.stream.cuda_stream)
        else:
            self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            apms_bind(self._h, self.workspace.data_ptr(), nbytes, self.stream.cuda_stream)

    def close(self):
        if getattr(self, "_h", None):
            apms_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @staticmethod
    def _grad_type(grads) -> int:
        """GRAD_* constant of a list of torch tensors or numpy arrays that share one dtype."""
        import torch

        names = {str(g.dtype).replace("torch.", "") for g in grads}
        assert len(names) == 1, f"gradients of mixed types: {names}"
        return {"float32": GRAD_F32, "bfloat16": GRAD_BF16, "float16": GRAD_F16}[names.pop()]

    @staticmethod
    def _dev_ptrs(grads) -> list:
        ptrs = []
        for g in grads:
            assert g.is_cuda and g.is_contiguous()
            ptrs.append(g.data_ptr())
        return ptrs

    def set_params(self, x0):
        """x0: torch CUDA float32 tensor or numpy float32 array of d elements."""
        if isinstance(x0, np.ndarray):
            x0 = np.ascontiguousarray(x0, dtype=np.float32)
            assert x0.size == self.d
            apms_set_params(self._h, x0.ctypes.data, False)
        else:
            assert x0.numel() == self.d and x0.is_contiguous()
            apms_set_params(self._h, x0.data_ptr(), x0.is_cuda)

    def set_lr(self, lr: float):
        apms_set_lr(self._h, lr)

    def warmup_step(self, grads):
        assert len(grads) == self.n
        apms_warmup_step_typed(self._h, self._dev_ptrs(grads), self._grad_type(grads))

    def freeze_v(self):
        apms_freeze_v(self._h)

    def compressed_step(self, grads):
        assert len(grads) == self.n
        apms_compressed_step_typed(self._h, self._dev_ptrs(grads), self._grad_type(grads))

    def compressed_step_host(self, grads_host, x_out_host=None):
        """grads_host: n CPU float32 tensors/arrays (pinned for overlap); x_out_host: CPU buffer or None."""
        assert len(grads_host) == self.n

        def hp(a):
            return a.ctypes.data if isinstance(a, np.ndarray) else a.data_ptr()

        apms_compressed_step_host_typed(self._h, [hp(g) for g in grads_host], self._grad_type(grads_host),
                                        None if x_out_host is None else hp(x_out_host))

    def get_params(self, out=None) -> np.ndarray:
        if out is not None and not isinstance(out, np.ndarray):
            apms_get_params(self._h, out.data_ptr(), out.is_cuda)
            return out
        out = np.empty(self.d, dtype=np.float32) if out is None else out
        apms_get_params(self._h, out.ctypes.data, False)
        return out

    def get_state(self, which: int, worker: int = 0) -> np.ndarray:
        if which in (STATE_WORKER_BITS, STATE_SERVER_BITS):
            out = np.empty(self.W, dtype=np.uint32)
        elif which in (STATE_WORKER_SCALES, STATE_SERVER_SCALES):
            out = np.empty(self.C, dtype=np.float32)
        else:
            out = np.empty(self.d, dtype=np.float32)
        apms_get_state(self._h, which, worker, out.ctypes.data)
        return out

    def get_state_slice(self, which: int, first: int, count: int, worker: int = 0) -> np.ndarray:
        dtype = np.uint32 if which in (STATE_WORKER_BITS, STATE_SERVER_BITS) else np.float32
        out = np.empty(count, dtype=dtype)
        apms_get_state_slice(self._h, which, worker, first, count, out.ctypes.data)
        return out

    def set_state(self, which: int, value: np.ndarray, worker: int = 0):
        value = np.ascontiguousarray(value, dtype=np.float32)
        assert value.size == self.d
        apms_set_state(self._h, which, worker, value.ctypes.data)

    # phase-wise step (the caller carries out the exchanges; see paper_2008_11343_b200/sharded.py)
    def worker_phase(self, grads):
        assert len(grads) == self.n
        apms_worker_phase(self._h, self._dev_ptrs(grads), self._grad_type(grads))

    def worker_phase_range(self, grads, chunk_begin: int, chunk_end: int):
        """Steps 1-2 for chunks [chunk_begin, chunk_end) only; one step's ranges must cover every chunk once."""
        assert len(grads) == self.n
        apms_worker_phase_range(self._h, self._dev_ptrs(grads), self._grad_type(grads), chunk_begin, chunk_end)

    def message(self, worker: int):
        """Torch views (int32 sign words [W], float32 scales [C]) onto worker `worker`'s message inside the
        workspace (-1: the server's message).  No copy: the library writes these buffers."""
        import torch

        if self.workspace is None:
            raise RuntimeError("message() views need the torch workspace; use message_ptrs() with a library workspace")
        bits_ptr, scales_ptr = apms_get_message(self._h, worker)
        base = self.workspace.data_ptr()
        b0, s0 = bits_ptr - base, scales_ptr - base
        bits = self.workspace[b0:b0 + 4 * self.W].view(torch.int32)
        scales = self.workspace[s0:s0 + 4 * self.C].view(torch.float32)
        return bits, scales

    def server_phase(self, bits_rows, scale_rows, chunk_begin: int, chunk_end: int):
        """bits_rows: int32 CUDA tensor [rows, row_words]; scale_rows: float32 CUDA tensor [rows, row_scales]."""
        assert bits_rows.is_contiguous() and scale_rows.is_contiguous() and bits_rows.shape[0] == scale_rows.shape[0]
        apms_server_phase(self._h, bits_rows.data_ptr(), bits_rows.shape[1], scale_rows.data_ptr(), scale_rows.shape[1],
                          bits_rows.shape[0], chunk_begin, chunk_end)

    def apply_phase(self):
        apms_apply_phase(self._h)

    def message_ptrs(self, worker: int):
        """Device addresses (sign words, scales) of worker `worker`'s message (-1: the server's)."""
        return apms_get_message(self._h, worker)

    def message_offsets(self, worker: int):
        """Byte offsets of that message inside the workspace (equal for contexts of equal shape)."""
        return apms_message_offsets(self._h, worker)

    def server_phase_rows(self, bits_row_ptrs, scale_row_ptrs, chunk_begin: int, chunk_end: int):
        """One device address per sender and array: where its sign words / scales of chunk_begin lie."""
        apms_server_phase_rows(self._h, bits_row_ptrs, scale_row_ptrs, chunk_begin, chunk_end)

    def put_server_range(self, dst_bits_ptr: int, dst_scales_ptr: int, chunk_begin: int, chunk_end: int):
        apms_put_server_range(self._h, dst_bits_ptr, dst_scales_ptr, chunk_begin, chunk_end)

    def ipc_export(self) -> bytes:
        return apms_ipc_export(self._h)

    def synchronize(self):
        self.stream.synchronize()

    def record_event(self):
        """A torch CUDA event recorded on the context's stream (its synchronize() waits for the work enqueued so far)."""
        import torch

        ev = torch.cuda.Event()
        ev.record(self.stream)
        return ev

    def set_schedule(self, schedule: Optional[Schedule]):
        apms_set_schedule(self._h, schedule)

    def step(self, grads):
        """One step of Algorithm 1 under the attached schedule (warmup, phase switch or compressed step)."""
        assert len(grads) == self.n
        apms_step(self._h, self._dev_ptrs(grads), self._grad_type(grads))

    @property
    def steps_taken(self) -> int:
        return apms_get_step(self._h)

    def error_norms(self):
        return apms_error_norms(self._h, self.n)

    def restore(self, t: int, phase: int, steps: Optional[int] = None):
        """Counters of a checkpoint: Adam steps t, phase, and (if given) the schedule's step counter."""
        apms_restore(self._h, t, phase)
        if steps is not None:
            apms_set_step(self._h, steps)

    @property
    def phase(self) -> int:
        return apms_get_phase(self._h)

    @property
    def t(self) -> int:
        return apms_get_t(self._h)

    def set_compressor(self, kind: int, topk_fraction: float = 0.01):
        apms_set_compressor(self._h, kind, topk_fraction)
        self.topk = kind == COMPRESSOR_TOPK

    # phase-wise step with the top-k compressor: masks travel as the sign words do, the kept values packed
    def topk_values_per_chunk(self) -> int:
        return apms_topk_values_per_chunk(self._h)

    def topk_route_counts(self):
        return apms_topk_route_counts(self._h)

    def topk_pack_values(self, worker: int, chunk_begin: int, chunk_end: int, out):
        """out: float32 CUDA tensor of (chunk_end - chunk_begin) * topk_values_per_chunk() elements."""
        assert out.is_cuda and out.is_contiguous() and out.numel() >= (chunk_end - chunk_begin) * self.topk_values_per_chunk()
        apms_topk_pack_values(self._h, worker, chunk_begin, chunk_end, out.data_ptr())

    def topk_server_phase(self, mask_rows, val_rows, chunk_begin: int, chunk_end: int):
        """mask_rows: int32 CUDA tensor [rows, row_words]; val_rows: float32 CUDA tensor [rows, row_vals]."""
        import torch

        assert mask_rows.is_contiguous() and val_rows.is_contiguous() and mask_rows.shape[0] == val_rows.shape[0]
        need = apms_topk_server_scratch_bytes(self._h, mask_rows.shape[0], chunk_begin, chunk_end)
        if getattr(self, "_topk_scratch", None) is None or self._topk_scratch.numel() < need:
            self._topk_scratch = torch.empty(max(need, 16), dtype=torch.uint8, device=self.device)
        apms_topk_server_phase(self._h, mask_rows.data_ptr(), mask_rows.shape[1], val_rows.data_ptr(), val_rows.shape[1],
                               mask_rows.shape[0], chunk_begin, chunk_end, self._topk_scratch.data_ptr(), self._topk_scratch.numel())

    def topk_put_server_range(self, mask_words, vals, chunk_begin: int, chunk_end: int):
        assert mask_words.is_cuda and vals.is_cuda and mask_words.is_contiguous() and vals.is_contiguous()
        apms_topk_put_server_range(self._h, mask_words.data_ptr(), vals.data_ptr(), chunk_begin, chunk_end)

    def set_variant(self, variant: int):
        apms_set_variant(self._h, variant)

    def uncompressed_step(self, grads):
        """v frozen, nothing compressed ("APMSqueeze (Uncompressed)")."""
        assert len(grads) == self.n
        apms_uncompressed_step_typed(self._h, self._dev_ptrs(grads), self._grad_type(grads))

    def set_scale_kind(self, kind: int):
        apms_set_scale_kind(self._h, kind)

    def set_team_mode(self, mode: int):
        apms_set_team_mode(self._h, mode)

    def set_timing(self, enabled: bool):
        apms_set_timing(self._h, enabled)

    def check_guards(self):
        apms_check_guards(self._h)

    def kernel_time(self, which: int):
        return apms_kernel_time(self._h, which)

    @property
    def launch_count(self) -> int:
        return apms_launch_count(self._h)
