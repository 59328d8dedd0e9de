"""ctypes binding: one Python function per C entry point, same names, argument marshalling only."""

from __future__ import annotations

import ctypes
import os
from ctypes import c_char_p, c_int, c_size_t, c_uint, c_ulonglong, c_void_p

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None

FLAG_SKIP_OFFSET = 0x1
FLAG_OFFSET_ONLY = 0x2
FLAG_OUT_F32 = 0x4
FLAG_ACCUMULATE = 0x8
FLAG_PLAIN_G4 = 0x10
FLAG_CLUSTER_REDUCE = 0x20
FLAG_MIRROR = 0x40
FLAG_LUT_ONLY = 0x80
FLAG_TABLE_F16 = 0x100
FLAG_TABLE_I8 = 0x200


class GemvCall(ctypes.Structure):
    """elutq_gemv_call: one M = 1 call of a chain."""
    _fields_ = [("X", c_void_p), ("packed", c_void_p), ("Y", c_void_p), ("N", c_int), ("K", c_int), ("flags", c_uint)]


class ElutqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().elutq_status_string(status).decode()
        extra = f" (cudaError {lib().elutq_last_cuda_error()})" if status == -6 else ""
        super().__init__(f"{where}: {msg}{extra} [{status}]")


def library_path() -> str:
    return os.path.join(_HERE, "libelutq.so")


_SIGNATURES = {
    "elutq_status_string": (c_char_p, [c_int]),
    "elutq_last_cuda_error": (c_int, []),
    "elutq_packed_bytes": (c_int, [c_int, c_int, c_int, c_int, ctypes.POINTER(c_size_t)]),
    "elutq_pack": (c_int, [c_void_p, c_void_p, c_void_p, c_int, c_int, c_int, c_int, c_void_p, c_size_t, c_void_p]),
    "elutq_unpack": (c_int, [c_void_p, c_int, c_int, c_void_p, c_void_p, c_void_p, c_void_p]),
    "elutq_describe": (c_int, [c_void_p, c_int, c_int, ctypes.POINTER(c_int), ctypes.POINTER(c_int)]),
    "elutq_forget": (c_int, [c_void_p]),
    "elutq_workspace_bytes": (c_int, [c_int, c_int, c_int, ctypes.POINTER(c_size_t)]),
    "elutq_workspace_init": (c_int, [c_void_p, c_size_t, c_void_p]),
    "elutq_lut_gemm": (c_int, [c_void_p, c_void_p, c_void_p, c_int, c_int, c_int, c_void_p]),
    "elutq_lut_gemm_bias": (c_int, [c_void_p, c_void_p, c_void_p, c_int, c_int, c_int, c_int, c_void_p]),
    "elutq_lut_gemm_f32": (c_int, [c_void_p, c_void_p, c_void_p, c_int, c_int, c_int, c_uint, c_void_p]),
    "elutq_lut_gemm_ws": (c_int, [c_void_p, c_void_p, c_void_p, c_int, c_int, c_int, c_uint, c_void_p, c_size_t, c_void_p]),
    "elutq_lut_gemm_host": (c_int, [c_void_p, c_void_p, c_void_p, c_int, c_int, c_int, c_void_p]),
    "elutq_lut_gemm_static": (c_int, [c_void_p, c_void_p, c_void_p, c_int, c_int, c_int, c_void_p]),
    "elutq_takes_tensor_path": (c_int, [c_int, c_int, c_int, c_int, c_uint]),
    "elutq_hlq_fit": (c_int, [c_void_p, c_int, c_int, c_int, c_int, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "elutq_chain_plan_bytes": (c_int, [ctypes.POINTER(GemvCall), c_int, ctypes.POINTER(c_size_t)]),
    "elutq_chain_plan": (c_int, [ctypes.POINTER(GemvCall), c_int, c_void_p, c_size_t, c_void_p]),
    "elutq_chain_run": (c_int, [c_void_p, c_int, c_void_p]),
    "elutq_chain_run_opts": (c_int, [c_void_p, c_int, c_uint, c_void_p]),
    "elutq_chain_run_host": (c_int, [c_void_p, c_int, c_void_p, c_void_p, c_size_t, c_void_p, c_void_p, c_size_t, c_void_p]),
    "elutq_chain_status": (c_int, [c_void_p, c_void_p, ctypes.POINTER(c_int)]),
    "elutq_chain_forget": (c_int, [c_void_p]),
    "elutq_chain_shares": (c_int, [c_int, c_int, c_int, c_int, c_int, ctypes.POINTER(c_int), ctypes.POINTER(c_int)]),
    "elutq_device_status": (c_int, [c_void_p, ctypes.POINTER(c_int)]),
    "elutq_launch_count": (c_ulonglong, []),
    "elutq_release_scratch": (c_int, []),
    "elutq_test_wait_expiry": (c_int, [c_void_p, c_void_p, c_void_p, c_int, c_int, c_int, c_uint, c_void_p]),
    "elutq_reserve": (c_int, [c_int, c_int, c_int, c_void_p]),
    "elutq_scratch_address": (c_int, [c_void_p, c_int, ctypes.POINTER(c_void_p), ctypes.POINTER(c_size_t)]),
}


def lib() -> ctypes.CDLL:
    """Load libelutq.so (built in-tree by `paper_2510_19482_b200.build`); raises if it is missing."""
    global _LIB
    if _LIB is None:
        path = library_path()
        if not os.path.exists(path):
            raise ImportError(f"{path} not found: build it with `python -m paper_2510_19482_b200.build` "
                              "(there is no CPU fallback)")
        handle = ctypes.CDLL(path)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype = res
            fn.argtypes = args
        _LIB = handle
    return _LIB


def _check(status: int, where: str) -> None:
    if status != 0:
        raise ElutqError(status, where)


def _ptr(t) -> int:
    """Raw address of a torch tensor (device or host); None -> NULL."""
    return 0 if t is None else t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def elutq_status_string(status: int) -> str:
    return lib().elutq_status_string(status).decode()


def elutq_last_cuda_error() -> int:
    return lib().elutq_last_cuda_error()


def elutq_launch_count() -> int:
    return int(lib().elutq_launch_count())


def elutq_release_scratch() -> None:
    _check(lib().elutq_release_scratch(), "elutq_release_scratch")


def elutq_packed_bytes(q: int, G: int, N: int, K: int) -> int:
    out = c_size_t(0)
    _check(lib().elutq_packed_bytes(q, G, N, K, ctypes.byref(out)), "elutq_packed_bytes")
    return out.value


def elutq_pack(planes, scales, offsets, q: int, G: int, N: int, K: int, packed=None, stream=None):
    """planes uint8 [q,N,K], scales fp16 [N,K/G,q], offsets fp16 [N,K/G] (CUDA tensors) -> packed uint8 blob."""
    import torch
    if packed is None:
        packed = torch.empty(elutq_packed_bytes(q, G, N, K), dtype=torch.uint8, device=planes.device)
    _check(lib().elutq_pack(_ptr(planes), _ptr(scales), _ptr(offsets), q, G, N, K,
                            _ptr(packed), packed.numel() * packed.element_size(), _stream(stream)), "elutq_pack")
    return packed


def elutq_unpack(packed, N: int, K: int, planes, scales, offsets, stream=None) -> None:
    _check(lib().elutq_unpack(_ptr(packed), N, K, _ptr(planes), _ptr(scales), _ptr(offsets), _stream(stream)),
           "elutq_unpack")


def elutq_describe(packed, N: int, K: int):
    q, G = c_int(0), c_int(0)
    _check(lib().elutq_describe(_ptr(packed), N, K, ctypes.byref(q), ctypes.byref(G)), "elutq_describe")
    return q.value, G.value


def elutq_forget(packed) -> None:
    _check(lib().elutq_forget(_ptr(packed)), "elutq_forget")


def elutq_workspace_bytes(M: int, N: int, K: int) -> int:
    out = c_size_t(0)
    _check(lib().elutq_workspace_bytes(M, N, K, ctypes.byref(out)), "elutq_workspace_bytes")
    return out.value


def elutq_workspace_init(workspace, stream=None) -> None:
    _check(lib().elutq_workspace_init(_ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "elutq_workspace_init")


def elutq_lut_gemm(X, packed, Y, M: int, N: int, K: int, stream=None) -> None:
    _check(lib().elutq_lut_gemm(_ptr(X), _ptr(packed), _ptr(Y), M, N, K, _stream(stream)), "elutq_lut_gemm")


def elutq_lut_gemm_bias(X, packed, Y, M: int, N: int, K: int, accumulate: bool = False, stream=None) -> None:
    _check(lib().elutq_lut_gemm_bias(_ptr(X), _ptr(packed), _ptr(Y), M, N, K, int(bool(accumulate)), _stream(stream)),
           "elutq_lut_gemm_bias")


def elutq_lut_gemm_f32(X, packed, Y, M: int, N: int, K: int, flags: int = 0, stream=None) -> None:
    _check(lib().elutq_lut_gemm_f32(_ptr(X), _ptr(packed), _ptr(Y), M, N, K, flags, _stream(stream)),
           "elutq_lut_gemm_f32")


def elutq_lut_gemm_ws(X, packed, Y, M: int, N: int, K: int, flags: int, workspace, stream=None) -> None:
    _check(lib().elutq_lut_gemm_ws(_ptr(X), _ptr(packed), _ptr(Y), M, N, K, flags, _ptr(workspace),
                                   workspace.numel() * workspace.element_size(), _stream(stream)), "elutq_lut_gemm_ws")


def elutq_lut_gemm_host(X_host, packed, Y_host, M: int, N: int, K: int, stream=None) -> None:
    _check(lib().elutq_lut_gemm_host(_ptr(X_host), _ptr(packed), _ptr(Y_host), M, N, K, _stream(stream)),
           "elutq_lut_gemm_host")


def elutq_takes_tensor_path(M: int, N: int, K: int, G: int = 128, flags: int = 0) -> bool:
    """True when elutq_lut_gemm runs this shape on the tensor-core path (host-only)."""
    return bool(lib().elutq_takes_tensor_path(M, N, K, G, flags))


def elutq_lut_gemm_static(X, packed, Y, M: int, N: int, K: int, stream=None) -> None:
    """elutq_lut_gemm for callers that must not allocate: scratch is a fixed 4 MiB array inside the library."""
    _check(lib().elutq_lut_gemm_static(_ptr(X), _ptr(packed), _ptr(Y), M, N, K, _stream(stream)),
           "elutq_lut_gemm_static")


def elutq_hlq_fit(W, q: int, G: int, t_max: int = 10, trace: bool = False, stream=None):
    """Algorithm 1 on a CUDA fp16 matrix W [N, K] -> (planes uint8 [q,N,K], scales fp16 [N,K/G,q],
    offsets fp16 [N,K/G]) and, with trace=True, the per-group squared error [t_max+1, N*K/G] (fp64)."""
    import torch
    N, K = W.shape
    planes = torch.empty((q, N, K), dtype=torch.uint8, device=W.device)
    scales = torch.empty((N, K // G, q), dtype=torch.float16, device=W.device)
    offsets = torch.empty((N, K // G), dtype=torch.float16, device=W.device)
    tr = torch.empty((t_max + 1, N * (K // G)), dtype=torch.float64, device=W.device) if trace else None
    _check(lib().elutq_hlq_fit(_ptr(W), q, G, N, K, t_max, _ptr(planes), _ptr(scales), _ptr(offsets),
                               _ptr(tr) if trace else None, _stream(stream)), "elutq_hlq_fit")
    return (planes, scales, offsets, tr) if trace else (planes, scales, offsets)


def elutq_device_status(stream=None) -> int:
    """0 unless a kernel gave up on a bounded wait (synchronises the stream)."""
    out = c_int(0)
    _check(lib().elutq_device_status(_stream(stream), ctypes.byref(out)), "elutq_device_status")
    return out.value


def _call_array(calls):
    """calls: sequence of (X, packed, Y, N, K[, flags]) with tensors or raw addresses -> ctypes array."""
    arr = (GemvCall * len(calls))()
    for i, c in enumerate(calls):
        X, packed, Y, N, K = c[:5]
        flags = c[5] if len(c) > 5 else 0
        arr[i] = GemvCall(X if isinstance(X, int) else _ptr(X), packed if isinstance(packed, int) else _ptr(packed),
                          Y if isinstance(Y, int) else _ptr(Y), N, K, flags)
    return arr


def elutq_chain_plan_bytes(calls) -> int:
    out = c_size_t(0)
    _check(lib().elutq_chain_plan_bytes(_call_array(calls), len(calls), ctypes.byref(out)), "elutq_chain_plan_bytes")
    return out.value


def elutq_chain_plan(calls, plan=None, stream=None):
    """Writes the plan of a list of M = 1 calls into a device buffer (allocated here when not given); returns it."""
    import torch
    if plan is None:
        plan = torch.empty(elutq_chain_plan_bytes(calls), dtype=torch.uint8, device="cuda")
    _check(lib().elutq_chain_plan(_call_array(calls), len(calls), _ptr(plan), plan.numel() * plan.element_size(),
                                  _stream(stream)), "elutq_chain_plan")
    return plan


def elutq_chain_run(plan, n_calls: int, stream=None) -> None:
    _check(lib().elutq_chain_run(_ptr(plan), n_calls, _stream(stream)), "elutq_chain_run")


def elutq_chain_run_opts(plan, n_calls: int, wait_limit: int = 0, stream=None) -> None:
    _check(lib().elutq_chain_run_opts(_ptr(plan), n_calls, wait_limit, _stream(stream)), "elutq_chain_run_opts")


def elutq_chain_run_host(plan, n_calls: int, x_dev, x_host, y_dev=None, y_host=None, stream=None) -> None:
    """x_host -> x_dev, the plan's launches, y_dev -> y_host, all on `stream` (whole tensors are copied; a pair that
    is None is not copied: e.g. when the plan's Y pointers name pinned host memory themselves)."""
    xb = 0 if x_host is None else x_host.numel() * x_host.element_size()
    yb = 0 if y_host is None else y_host.numel() * y_host.element_size()
    _check(lib().elutq_chain_run_host(_ptr(plan), n_calls, _ptr(x_dev), _ptr(x_host), xb, _ptr(y_dev), _ptr(y_host), yb,
                                      _stream(stream)), "elutq_chain_run_host")


def elutq_chain_status(plan, stream=None) -> int:
    out = c_int(0)
    _check(lib().elutq_chain_status(_ptr(plan), _stream(stream), ctypes.byref(out)), "elutq_chain_status")
    return out.value


def elutq_chain_forget(plan) -> None:
    _check(lib().elutq_chain_forget(_ptr(plan)), "elutq_chain_forget")


def elutq_chain_shares(N: int, K: int, n_ctas_max: int, cta_first: int = 0, independent: bool = True):
    """(shares, partition): shares[cta] = (first row block, end row block, first chunk, chunks, chunk group);
    partition = (chunks per CTA, row ranges, chunk groups, CTAs with a share).  Host logic only."""
    raw = (c_int * (4 * n_ctas_max))()
    part = (c_int * 4)()
    _check(lib().elutq_chain_shares(N, K, n_ctas_max, cta_first, 1 if independent else 0, raw, part), "elutq_chain_shares")
    shares = [(raw[4 * i], raw[4 * i + 1], raw[4 * i + 2], raw[4 * i + 3] & 0xffff, raw[4 * i + 3] >> 16) for i in range(n_ctas_max)]
    return shares, tuple(part)


def elutq_reserve(M: int, N: int, K: int, stream=None) -> None:
    _check(lib().elutq_reserve(M, N, K, _stream(stream)), "elutq_reserve")


def elutq_scratch_address(kind: int, stream=None):
    """(address or None, bytes) of a library-owned scratch buffer of the stream."""
    ptr, nb = c_void_p(0), c_size_t(0)
    _check(lib().elutq_scratch_address(_stream(stream), kind, ctypes.byref(ptr), ctypes.byref(nb)), "elutq_scratch_address")
    return ptr.value, nb.value


def elutq_test_wait_expiry(X, packed, Y, M: int, N: int, K: int, wait_limit: int, stream=None) -> None:
    _check(lib().elutq_test_wait_expiry(_ptr(X), _ptr(packed), _ptr(Y), M, N, K, wait_limit, _stream(stream)),
           "elutq_test_wait_expiry")
