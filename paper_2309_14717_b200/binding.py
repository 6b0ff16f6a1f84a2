"""Thin ctypes binding of libqalora.so (include/qalora.h).

Argument marshalling only: every step of the layer runs in the library's CUDA
kernels.  torch supplies device memory and the current stream.  There is no CPU
fallback: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_float, c_int, c_int32, c_int64, c_size_t, c_void_p

import torch

# QALORA_LIBRARY=debug selects the bounds-check build (libqalora_debug.so, made by
# `python -m paper_2309_14717_b200.build --debug`); anything else the ordinary library.
DEBUG_LIBRARY = os.environ.get("QALORA_LIBRARY", "") == "debug"
_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)),
                         "libqalora_debug.so" if DEBUG_LIBRARY else "libqalora.so")

OP_FORWARD, OP_BACKWARD, OP_TRAIN = 0, 1, 2

EXPORTS = (
    "qalora_version", "qalora_status_string", "qalora_packed_bytes", "qalora_workspace_bytes",
    "qalora_quantize", "qalora_forward", "qalora_backward", "qalora_merge",
    "qalora_kernel_launches", "qalora_profile_next_main_kernel", "qalora_main_kernel_name",
    "qalora_forward_static", "qalora_step_host_bytes", "qalora_step_host",
    "qalora_adamw_workspace_bytes", "qalora_adamw_step",
    "qalora_dequantize", "qalora_qparams_from_zero_point", "qalora_qparams_to_zero_point",
    "qalora_forward_group_workspace_bytes", "qalora_forward_group",
    "qalora_forward_train", "qalora_backward_train",
    "qalora_debug_checks", "qalora_debug_report",
)

STATIC_SCRATCH_BYTES = 1 << 20


class QaloraDesc(Structure):
    _fields_ = [("d_in", c_int32), ("d_out", c_int32), ("group_size", c_int32), ("bits", c_int32),
                ("rank", c_int32), ("scale", c_float)]


class GroupLayer(Structure):
    _fields_ = [("desc", QaloraDesc), ("x", c_void_p), ("codes", c_void_p), ("qparams", c_void_p),
                ("A", c_void_p), ("B", c_void_p), ("y", c_void_p)]


class AdamwHyper(Structure):
    _fields_ = [("lr", c_float), ("beta1", c_float), ("beta2", c_float), ("eps", c_float),
                ("weight_decay", c_float), ("max_grad_norm", c_float), ("step", c_int64)]


class QaloraError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        super().__init__(f"{fn} failed: {status_string(status)} ({status})")


_lib = None


def load() -> ctypes.CDLL:
    """Loads libqalora.so (built in-tree by paper_2309_14717_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: run `python -m paper_2309_14717_b200.build` first "
                          "(there is no CPU fallback)")
    lib = ctypes.CDLL(_LIB_PATH)
    D = POINTER(QaloraDesc)
    lib.qalora_version.restype = c_int
    lib.qalora_version.argtypes = []
    lib.qalora_debug_checks.restype = c_int
    lib.qalora_debug_checks.argtypes = []
    lib.qalora_debug_report.restype = c_int
    lib.qalora_debug_report.argtypes = [POINTER(c_int32)]
    lib.qalora_status_string.restype = c_char_p
    lib.qalora_status_string.argtypes = [c_int]
    lib.qalora_packed_bytes.restype = c_int
    lib.qalora_packed_bytes.argtypes = [D, POINTER(c_size_t), POINTER(c_size_t)]
    lib.qalora_workspace_bytes.restype = c_int
    lib.qalora_workspace_bytes.argtypes = [D, c_int64, c_int, POINTER(c_size_t)]
    lib.qalora_quantize.restype = c_int
    lib.qalora_quantize.argtypes = [D, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.qalora_forward.restype = c_int
    lib.qalora_forward.argtypes = [D, c_int64] + [c_void_p] * 6 + [c_void_p, c_size_t, c_void_p]
    lib.qalora_backward.restype = c_int
    lib.qalora_backward.argtypes = [D, c_int64] + [c_void_p] * 9 + [c_void_p, c_size_t, c_void_p]
    lib.qalora_forward_train.restype = c_int
    lib.qalora_forward_train.argtypes = lib.qalora_forward.argtypes
    lib.qalora_backward_train.restype = c_int
    lib.qalora_backward_train.argtypes = lib.qalora_backward.argtypes
    lib.qalora_merge.restype = c_int
    lib.qalora_merge.argtypes = [D, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.qalora_forward_static.restype = c_int
    lib.qalora_forward_static.argtypes = [D, c_int64] + [c_void_p] * 6 + [c_void_p]
    lib.qalora_step_host_bytes.restype = c_int
    lib.qalora_step_host_bytes.argtypes = [D, c_int64, POINTER(c_size_t)]
    lib.qalora_step_host.restype = c_int
    lib.qalora_step_host.argtypes = [D, c_int64] + [c_void_p] * 10 + [c_void_p, c_size_t, c_void_p]
    lib.qalora_dequantize.restype = c_int
    lib.qalora_dequantize.argtypes = [D, c_void_p, c_void_p, c_void_p, c_int, c_void_p]
    lib.qalora_qparams_from_zero_point.restype = c_int
    lib.qalora_qparams_from_zero_point.argtypes = [D, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.qalora_qparams_to_zero_point.restype = c_int
    lib.qalora_qparams_to_zero_point.argtypes = [D, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.qalora_adamw_workspace_bytes.restype = c_int
    lib.qalora_adamw_workspace_bytes.argtypes = [POINTER(c_size_t)]
    lib.qalora_adamw_step.restype = c_int
    lib.qalora_adamw_step.argtypes = [POINTER(AdamwHyper), c_int64] + [c_void_p] * 6 + [c_void_p, c_size_t, c_void_p]
    lib.qalora_forward_group_workspace_bytes.restype = c_int
    lib.qalora_forward_group_workspace_bytes.argtypes = [POINTER(GroupLayer), c_int, c_int64, POINTER(c_size_t)]
    lib.qalora_forward_group.restype = c_int
    lib.qalora_forward_group.argtypes = [POINTER(GroupLayer), c_int, c_int64, c_void_p, c_size_t, c_void_p]
    lib.qalora_kernel_launches.restype = ctypes.c_uint64
    lib.qalora_kernel_launches.argtypes = []
    lib.qalora_profile_next_main_kernel.restype = c_int
    lib.qalora_profile_next_main_kernel.argtypes = [c_void_p, c_void_p]
    lib.qalora_main_kernel_name.restype = c_char_p
    lib.qalora_main_kernel_name.argtypes = []
    _lib = lib
    return lib


def desc(d_in: int, d_out: int, group_size: int, bits: int, rank: int, scale: float) -> QaloraDesc:
    return QaloraDesc(d_in, d_out, group_size, bits, rank, scale)


def _ptr(t):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("tensors must live on a CUDA device")
    if not t.is_contiguous():
        raise ValueError("tensors must be contiguous")
    return c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return c_void_p(s.cuda_stream)


def _check(fn: str, status: int):
    if status != 0:
        raise QaloraError(fn, status)


def qalora_version() -> int:
    return int(load().qalora_version())


def status_string(status: int) -> str:
    return load().qalora_status_string(int(status)).decode()


def qalora_packed_bytes(d: QaloraDesc):
    cb, qb = c_size_t(), c_size_t()
    _check("qalora_packed_bytes", load().qalora_packed_bytes(byref(d), byref(cb), byref(qb)))
    return cb.value, qb.value


def qalora_workspace_bytes(d: QaloraDesc, m: int, op: int) -> int:
    b = c_size_t()
    _check("qalora_workspace_bytes", load().qalora_workspace_bytes(byref(d), m, op, byref(b)))
    return b.value


def alloc_packed(d: QaloraDesc, device="cuda"):
    """Allocates (codes int32 [K/32, N, words], qparams float32 [G, N, 2]) on the device."""
    cb, qb = qalora_packed_bytes(d)
    words = cb // 4 // ((d.d_in // 32) * d.d_out)
    codes = torch.empty((d.d_in // 32, d.d_out, words), dtype=torch.int32, device=device)
    qparams = torch.empty((d.d_in // d.group_size, d.d_out, 2), dtype=torch.float32, device=device)
    return codes, qparams


def alloc_workspace(d: QaloraDesc, m: int, op: int, device="cuda") -> torch.Tensor:
    """Zeroed scratch of qalora_workspace_bytes() bytes (at least 16) for `m` rows."""
    return torch.zeros(max(qalora_workspace_bytes(d, m, op), 16), dtype=torch.uint8, device=device)


def workspace_status(workspace: torch.Tensor) -> int:
    """Device status word at the head of a workspace (synchronizes): 0 = ok,
    1 = a bounded wait inside a tensor-core kernel expired (results invalid)."""
    return int(workspace[:4].view(torch.int32).item())


def qalora_quantize(d: QaloraDesc, W, codes, qparams, dev_status=None, stream=None):
    _check("qalora_quantize", load().qalora_quantize(byref(d), _ptr(W), _ptr(codes), _ptr(qparams),
                                                     _ptr(dev_status), _stream(stream)))


def qalora_forward(d: QaloraDesc, m: int, x, codes, qparams, A, B, y, workspace, stream=None):
    _check("qalora_forward", load().qalora_forward(byref(d), m, _ptr(x), _ptr(codes), _ptr(qparams), _ptr(A),
                                                   _ptr(B), _ptr(y), _ptr(workspace),
                                                   workspace.numel() if workspace is not None else 0,
                                                   _stream(stream)))


def qalora_forward_static(d: QaloraDesc, m: int, x, codes, qparams, A, B, y, stream=None):
    """qalora_forward without a workspace argument: the scratch is a fixed array
    inside the library (STATIC_SCRATCH_BYTES), for callers that cannot allocate
    device memory.  Raises QaloraError(-7) when m * rank needs more than that.
    Calls that overlap on the GPU share the array and must be serialized."""
    _check("qalora_forward_static", load().qalora_forward_static(byref(d), m, _ptr(x), _ptr(codes), _ptr(qparams),
                                                                 _ptr(A), _ptr(B), _ptr(y), _stream(stream)))


def group_layers(layers):
    """ctypes array for qalora_forward_group from (desc, x, codes, qparams, A, B, y) tuples of tensors."""
    arr = (GroupLayer * len(layers))()
    for i, (d, x, codes, qparams, A, B, y) in enumerate(layers):
        ptr = lambda t: _ptr(t).value if t is not None else None
        arr[i] = GroupLayer(d, ptr(x), ptr(codes), ptr(qparams), ptr(A), ptr(B), ptr(y))
    return arr


def qalora_forward_group_workspace_bytes(layers, m: int) -> int:
    arr = layers if isinstance(layers, ctypes.Array) else group_layers(layers)
    b = c_size_t()
    _check("qalora_forward_group_workspace_bytes", load().qalora_forward_group_workspace_bytes(arr, len(arr), m, byref(b)))
    return b.value


def qalora_forward_group(layers, m: int, workspace, stream=None):
    """Forward of several independent layers ((desc, x, codes, qparams, A, B, y) tuples, or the
    array group_layers() made of them) on m rows each; one launch when the layers allow it."""
    arr = layers if isinstance(layers, ctypes.Array) else group_layers(layers)
    _check("qalora_forward_group", load().qalora_forward_group(arr, len(arr), m, _ptr(workspace), workspace.numel(),
                                                               _stream(stream)))


def qalora_step_host_bytes(d: QaloraDesc, m: int) -> int:
    b = c_size_t()
    _check("qalora_step_host_bytes", load().qalora_step_host_bytes(byref(d), m, byref(b)))
    return b.value


def _hptr(t):
    if t.is_cuda or not t.is_contiguous():
        raise ValueError("host tensors must be contiguous CPU tensors")
    return c_void_p(t.data_ptr())


def qalora_step_host(d: QaloraDesc, m: int, x_host, dy_host, codes, qparams, A, B, y_host, dx_host, dA_host, dB_host,
                     staging, stream=None):
    """Forward + backward from (pinned) host tensors; outputs land in host tensors
    once the stream is synchronized."""
    _check("qalora_step_host", load().qalora_step_host(byref(d), m, _hptr(x_host), _hptr(dy_host), _ptr(codes),
                                                       _ptr(qparams), _ptr(A), _ptr(B), _hptr(y_host), _hptr(dx_host),
                                                       _hptr(dA_host), _hptr(dB_host), _ptr(staging), staging.numel(),
                                                       _stream(stream)))


def qalora_backward(d: QaloraDesc, m: int, x, dy, codes, qparams, A, B, dx, dA, dB, workspace, stream=None):
    _check("qalora_backward", load().qalora_backward(byref(d), m, _ptr(x), _ptr(dy), _ptr(codes), _ptr(qparams),
                                                     _ptr(A), _ptr(B), _ptr(dx), _ptr(dA), _ptr(dB),
                                                     _ptr(workspace),
                                                     workspace.numel() if workspace is not None else 0,
                                                     _stream(stream)))


def qalora_forward_train(d: QaloraDesc, m: int, x, codes, qparams, A, B, y, workspace, stream=None):
    """qalora_forward that leaves pool(x) and T in a workspace of OP_TRAIN size for qalora_backward_train."""
    _check("qalora_forward_train", load().qalora_forward_train(byref(d), m, _ptr(x), _ptr(codes), _ptr(qparams), _ptr(A),
                                                               _ptr(B), _ptr(y), _ptr(workspace),
                                                               workspace.numel() if workspace is not None else 0,
                                                               _stream(stream)))


def qalora_backward_train(d: QaloraDesc, m: int, x, dy, codes, qparams, A, B, dx, dA, dB, workspace, stream=None):
    """qalora_backward on the workspace the preceding qalora_forward_train of the same step filled."""
    _check("qalora_backward_train", load().qalora_backward_train(byref(d), m, _ptr(x), _ptr(dy), _ptr(codes),
                                                                 _ptr(qparams), _ptr(A), _ptr(B), _ptr(dx), _ptr(dA),
                                                                 _ptr(dB), _ptr(workspace),
                                                                 workspace.numel() if workspace is not None else 0,
                                                                 _stream(stream)))


def qalora_merge(d: QaloraDesc, qparams_in, A, B, qparams_out, stream=None):
    _check("qalora_merge", load().qalora_merge(byref(d), _ptr(qparams_in), _ptr(A), _ptr(B), _ptr(qparams_out),
                                               _stream(stream)))


def qalora_dequantize(d: QaloraDesc, codes, qparams, W, stream=None):
    """W [d_in][d_out] (float32 or bfloat16, by W's dtype) = alpha * codes + beta."""
    import torch
    if W.dtype not in (torch.float32, torch.bfloat16):
        raise ValueError("W must be float32 or bfloat16")
    _check("qalora_dequantize", load().qalora_dequantize(byref(d), _ptr(codes), _ptr(qparams), _ptr(W),
                                                         1 if W.dtype == torch.bfloat16 else 0, _stream(stream)))


def qalora_qparams_from_zero_point(d: QaloraDesc, alpha, zero, qparams, stream=None):
    _check("qalora_qparams_from_zero_point", load().qalora_qparams_from_zero_point(
        byref(d), _ptr(alpha), _ptr(zero), _ptr(qparams), _stream(stream)))


def qalora_qparams_to_zero_point(d: QaloraDesc, qparams, alpha, zero, stream=None):
    _check("qalora_qparams_to_zero_point", load().qalora_qparams_to_zero_point(
        byref(d), _ptr(qparams), _ptr(alpha), _ptr(zero), _stream(stream)))


def qalora_adamw_workspace_bytes() -> int:
    b = c_size_t()
    _check("qalora_adamw_workspace_bytes", load().qalora_adamw_workspace_bytes(byref(b)))
    return b.value


def adamw_hyper(step: int, lr: float, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
                weight_decay: float = 0.0, max_grad_norm: float = 0.3) -> AdamwHyper:
    return AdamwHyper(lr, beta1, beta2, eps, weight_decay, max_grad_norm, step)


def qalora_adamw_step(hyper: AdamwHyper, n: int, grad, param, exp_avg, exp_avg_sq, param_bf16, norm_out, workspace,
                      stream=None):
    """Clipped AdamW over one flat array of n trained values (all on the device)."""
    _check("qalora_adamw_step", load().qalora_adamw_step(byref(hyper), n, _ptr(grad), _ptr(param), _ptr(exp_avg),
                                                         _ptr(exp_avg_sq), _ptr(param_bf16), _ptr(norm_out),
                                                         _ptr(workspace),
                                                         workspace.numel() * workspace.element_size()
                                                         if workspace is not None else 0, _stream(stream)))


def qalora_kernel_launches() -> int:
    return int(load().qalora_kernel_launches())


def qalora_debug_checks() -> bool:
    """True when the loaded library is the bounds-check build."""
    return bool(load().qalora_debug_checks())


def qalora_debug_report() -> list:
    """Waits for the device, returns the bounds-check build's eight record words and clears them
    (all zero when no check failed and no guard word was overwritten; always zero in the ordinary build)."""
    words = (c_int32 * 8)()
    _check("qalora_debug_report", load().qalora_debug_report(words))
    return list(words)


def qalora_profile_next_main_kernel(start_event, stop_event):
    """start_event/stop_event: torch.cuda.Event(enable_timing=True) that have been
    recorded at least once (so that their CUDA handles exist), or None to disarm."""
    a = c_void_p(start_event.cuda_event) if start_event is not None else None
    b = c_void_p(stop_event.cuda_event) if stop_event is not None else None
    _check("qalora_profile_next_main_kernel", load().qalora_profile_next_main_kernel(a, b))


def qalora_main_kernel_name() -> str:
    return load().qalora_main_kernel_name().decode()
