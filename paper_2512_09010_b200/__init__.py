"""Python binding of the LUVC C-ABI library (``include/luvc.h``).

Argument marshalling only: every step of OIM (Section 3.2 of arXiv 2512.09010) and
SPU (Section 3.3, Algorithm 2) runs inside ``libluvc.so``'s CUDA kernels.  PyTorch
is used for device memory and streams.  There is no CPU fallback: if the shared
library cannot be built or loaded, importing this package fails.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import _build

BF16, F32 = 0, 1
DEFAULT_CUTOFF = 0.125

STATUS_NAMES = {
    0: "LUVC_OK", 1: "LUVC_ERR_NULL", 2: "LUVC_ERR_SHAPE", 3: "LUVC_ERR_TARGET", 4: "LUVC_ERR_KEEP",
    5: "LUVC_ERR_CUTOFF", 6: "LUVC_ERR_ALIGN", 7: "LUVC_ERR_DTYPE", 8: "LUVC_ERR_WORKSPACE",
    9: "LUVC_ERR_CUDA", 10: "LUVC_ERR_TIMEOUT", 11: "LUVC_ERR_INTERNAL",
}

# every symbol include/luvc.h declares
EXPORTS = (
    "luvc_version", "luvc_status_string", "luvc_set_stream", "luvc_shutdown", "luvc_kernel_launches",
    "luvc_profile_enable", "luvc_profile_read", "luvc_check_status", "luvc_read_status", "luvc_debug_wait_probes",
    "luvc_oim_plan", "luvc_oim_plan_anyres", "luvc_oim_workspace_bytes", "luvc_oim_workspace_bytes_ex", "luvc_oim_merge", "luvc_oim_merge_f32", "luvc_oim_merge_ex",
    "luvc_oim_merge_host", "luvc_oim_value_enhance", "luvc_spu_sigma", "luvc_spu_workspace_bytes", "luvc_spu_prune",
    "luvc_spu_prune_f32", "luvc_spu_prune_ex", "luvc_spu_prune_host", "luvc_spu_prune_static", "luvc_spu_static_status",
    "luvc_spu_cascade",
)


class LuvcError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib.luvc_status_string(status).decode()
        super().__init__("%s: %s (%s)" % (where, STATUS_NAMES.get(status, status), msg))


class OimOpts(ctypes.Structure):
    _fields_ = [
        ("dtype", ctypes.c_int), ("stream", ctypes.c_void_p), ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_size_t), ("out_h", ctypes.c_int), ("out_w", ctypes.c_int),
        ("merge_per_step", ctypes.c_int), ("height_first", ctypes.c_int), ("trace", ctypes.c_void_p),
        ("trace_bytes", ctypes.c_size_t), ("out_log_sizes", ctypes.c_void_p), ("matching", ctypes.c_int),
        ("device_status", ctypes.c_void_p), ("merge_per_step_h", ctypes.c_int), ("merge_per_step_w", ctypes.c_int),
    ]


class SpuOpts(ctypes.Structure):
    _fields_ = [
        ("dtype", ctypes.c_int), ("stream", ctypes.c_void_p), ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_size_t), ("no_window", ctypes.c_int), ("out_scores", ctypes.c_void_p),
        ("device_status", ctypes.c_void_p),
    ]


def _load() -> ctypes.CDLL:
    path = _build.LIB
    if _build.is_stale():
        try:
            _build.build()
        except Exception as exc:  # no compiler: a stale or missing library is an error, not a fallback
            if not os.path.exists(path):
                raise ImportError("libluvc.so is missing and could not be built: %s" % exc) from exc
    L = ctypes.CDLL(path)
    i, p, f, sz = ctypes.c_int, ctypes.c_void_p, ctypes.c_float, ctypes.c_size_t
    L.luvc_version.restype = i
    L.luvc_status_string.restype = ctypes.c_char_p
    L.luvc_status_string.argtypes = [i]
    L.luvc_set_stream.argtypes = [p]
    L.luvc_kernel_launches.restype = ctypes.c_longlong
    L.luvc_check_status.argtypes = [p]
    L.luvc_read_status.argtypes = [p, p]
    L.luvc_debug_wait_probes.argtypes = [i, i, p, p]
    L.luvc_spu_static_status.argtypes = [p]
    L.luvc_oim_plan_anyres.argtypes = [i, i, i, i] + [ctypes.POINTER(i)] * 5
    L.luvc_profile_enable.argtypes = [i]
    L.luvc_profile_read.argtypes = [ctypes.POINTER(ctypes.c_float), i]
    L.luvc_oim_plan.argtypes = [i, i, i, i, ctypes.POINTER(i), ctypes.POINTER(i), ctypes.POINTER(i)]
    L.luvc_oim_workspace_bytes.restype = sz
    L.luvc_oim_workspace_bytes.argtypes = [i, i, i, i, i]
    L.luvc_oim_workspace_bytes_ex.restype = sz
    L.luvc_oim_workspace_bytes_ex.argtypes = [i, i, i, i, i, i]
    L.luvc_oim_merge.argtypes = [p, i, i, i, i, i, p, p, p]
    L.luvc_oim_merge_f32.argtypes = [p, i, i, i, i, i, p, p, p]
    L.luvc_oim_merge_ex.argtypes = [p, i, i, i, i, i, p, p, p, ctypes.POINTER(OimOpts)]
    L.luvc_oim_merge_host.argtypes = [p, i, i, i, i, i, i, p, p, p]
    L.luvc_oim_value_enhance.argtypes = [p, p, i, i, i, i, p, p]
    L.luvc_spu_sigma.argtypes = [i, f]
    L.luvc_spu_workspace_bytes.restype = sz
    L.luvc_spu_workspace_bytes.argtypes = [i, i, i, f, i]
    L.luvc_spu_prune.argtypes = [p, i, i, i, f, i, p, p]
    L.luvc_spu_prune_f32.argtypes = [p, i, i, i, f, i, p, p]
    L.luvc_spu_prune_ex.argtypes = [p, i, i, i, f, i, p, p, ctypes.POINTER(SpuOpts)]
    L.luvc_spu_prune_host.argtypes = [p, i, i, i, f, i, i, p, p]
    L.luvc_spu_prune_static.argtypes = [p, i, i, i, f, i, i, p, p, p]
    L.luvc_spu_cascade.argtypes = [p, i, i, i, i, ctypes.POINTER(i), ctypes.POINTER(f), i, p, p, p]
    return L


lib = _load()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise LuvcError(status, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise TypeError("luvc supports bfloat16 and float32 tensors, got %s" % t.dtype)


def _stream_ptr(device) -> int:
    return torch.cuda.current_stream(device).cuda_stream


def version() -> int:
    return lib.luvc_version()


def kernel_launches() -> int:
    return int(lib.luvc_kernel_launches())


def shutdown() -> None:
    _check(lib.luvc_shutdown(), "luvc_shutdown")


def check_status(device=None) -> int:
    """Synchronises the current torch stream and returns (and clears) the device status word."""
    return int(lib.luvc_check_status(_stream_ptr(device)))


PHASES = ("oim_steps", "oim_total", "spu_transform", "spu_select", "spu_gather")


def profile_enable(on: bool) -> None:
    _check(lib.luvc_profile_enable(int(bool(on))), "luvc_profile_enable")


def profile_read() -> dict:
    """Elapsed milliseconds of the phases of the most recent calls (synchronises their events)."""
    buf = (ctypes.c_float * len(PHASES))()
    _check(lib.luvc_profile_read(buf, len(PHASES)), "luvc_profile_read")
    return {name: float(buf[k]) for k, name in enumerate(PHASES)}


def oim_plan(H: int, W: int, target_count: int, merge_per_step: int = 0):
    """(out_h, out_w, n_steps) for a target token count (host only)."""
    h, w, n = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    _check(lib.luvc_oim_plan(H, W, target_count, merge_per_step, ctypes.byref(h), ctypes.byref(w), ctypes.byref(n)),
           "luvc_oim_plan")
    return h.value, w.value, n.value


def oim_plan_anyres(H: int, W: int, n_ops: int, merge_per_step: int = 0):
    """((merge_h, merge_w), (out_h, out_w), n_steps) for a grid whose sides differ (host only)."""
    v = [ctypes.c_int() for _ in range(5)]
    _check(lib.luvc_oim_plan_anyres(H, W, n_ops, merge_per_step, *[ctypes.byref(c) for c in v]), "luvc_oim_plan_anyres")
    return (v[0].value, v[1].value), (v[2].value, v[3].value), v[4].value


def read_status(block: torch.Tensor) -> int:
    """luvc_read_status on a caller-owned status block (int32 tensor of >= 4 words on the device)."""
    return int(lib.luvc_read_status(block.data_ptr(), _stream_ptr(block.device)))


def spu_sigma(N: int, cutoff: float = 0.0) -> int:
    return lib.luvc_spu_sigma(N, float(cutoff))


def oim_merge(tokens: torch.Tensor, target_count: int, *, out_hw=None, merge_per_step: int = 0,
              height_first: bool = False, want_trace: bool = False, workspace: torch.Tensor | None = None,
              want_log_sizes: bool = False, matching: str = "adjacent", merge_per_step_hw=None,
              device_status: torch.Tensor | None = None):
    """luvc_oim_merge_ex on a CUDA tensor [B,H,W,D]; returns (out_tokens [B,T,D], out_sizes [B,T] int32,
    out_map [B,H*W] int32) and, with want_trace, the per-merge decision log [B,H*W-T] int32.
    matching: "adjacent" or "bipartite" (luvc_oim_matching); merge_per_step_hw: (per column in a height
    step, per row in a width step); device_status: a caller-owned status block (see read_status)."""
    if not tokens.is_cuda:
        raise ValueError("tokens must live on a CUDA device; host buffers go through oim_merge_host")
    tokens = tokens.contiguous()
    B, H, W, D = tokens.shape
    T = int(target_count)
    dev = tokens.device
    with torch.cuda.device(dev):
        out_tokens = torch.empty((B, max(T, 0), D), dtype=tokens.dtype, device=dev)
        out_sizes = torch.empty((B, max(T, 0)), dtype=torch.int32, device=dev)
        out_map = torch.empty((B, H * W), dtype=torch.int32, device=dev)
        trace = torch.zeros((B, max(H * W - T, 0)), dtype=torch.int32, device=dev) if want_trace else None
        o = OimOpts()
        o.dtype = _dtype_code(tokens)
        o.stream = _stream_ptr(dev)
        if workspace is not None:
            o.workspace, o.workspace_bytes = workspace.data_ptr(), workspace.numel() * workspace.element_size()
        if out_hw is not None:
            o.out_h, o.out_w = int(out_hw[0]), int(out_hw[1])
        o.merge_per_step = int(merge_per_step)
        o.height_first = int(bool(height_first))
        o.matching = {"adjacent": 0, "bipartite": 1}[matching]
        o.trace = trace.data_ptr() if (trace is not None and trace.numel()) else None
        o.trace_bytes = trace.numel() * 4 if trace is not None else 0
        if merge_per_step_hw is not None:
            o.merge_per_step_h, o.merge_per_step_w = int(merge_per_step_hw[0]), int(merge_per_step_hw[1])
        o.device_status = device_status.data_ptr() if device_status is not None else None
        log_sizes = torch.empty((B, max(T, 0)), dtype=torch.float32, device=dev) if want_log_sizes else None
        o.out_log_sizes = log_sizes.data_ptr() if log_sizes is not None else None
        _check(lib.luvc_oim_merge_ex(tokens.data_ptr(), B, H, W, D, T, out_tokens.data_ptr(), out_sizes.data_ptr(),
                                     out_map.data_ptr(), ctypes.byref(o)), "luvc_oim_merge_ex")
    res = (out_tokens, out_sizes, out_map)
    if want_trace:
        res = res + (trace,)
    if want_log_sizes:
        res = res + (log_sizes,)
    return res


def oim_value_enhance(values: torch.Tensor, sizes: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
    """luvc_oim_value_enhance: values [B,T,D] + log(sizes [B,T]) per row (Eq. 2); `out` may be `values`."""
    values = values.contiguous()
    sizes = sizes.contiguous()
    B, T, D = values.shape
    dev = values.device
    if out is None:
        out = torch.empty_like(values)
    with torch.cuda.device(dev):
        _check(lib.luvc_oim_value_enhance(values.data_ptr(), sizes.data_ptr(), B, T, D, _dtype_code(values),
                                          out.data_ptr(), _stream_ptr(dev)), "luvc_oim_value_enhance")
    return out


def oim_merge_plain(tokens: torch.Tensor, target_count: int):
    """The spec entry points luvc_oim_merge / luvc_oim_merge_f32 on the current torch stream."""
    tokens = tokens.contiguous()
    B, H, W, D = tokens.shape
    T = int(target_count)
    dev = tokens.device
    with torch.cuda.device(dev):
        out_tokens = torch.empty((B, T, D), dtype=tokens.dtype, device=dev)
        out_sizes = torch.empty((B, T), dtype=torch.int32, device=dev)
        out_map = torch.empty((B, H * W), dtype=torch.int32, device=dev)
        _check(lib.luvc_set_stream(_stream_ptr(dev)), "luvc_set_stream")
        fn = lib.luvc_oim_merge if _dtype_code(tokens) == BF16 else lib.luvc_oim_merge_f32
        _check(fn(tokens.data_ptr(), B, H, W, D, T, out_tokens.data_ptr(), out_sizes.data_ptr(), out_map.data_ptr()),
               "luvc_oim_merge")
    return out_tokens, out_sizes, out_map


def spu_prune(hidden: torch.Tensor, keep: int, cutoff: float = 0.0, *, no_window: bool = False,
              want_scores: bool = False, workspace: torch.Tensor | None = None,
              device_status: torch.Tensor | None = None):
    """luvc_spu_prune_ex on a CUDA tensor [B,N,D]; returns (out_idx [B,keep] int32, out_hidden [B,keep,D])
    and, with want_scores, the energies E [B,N] float32."""
    if not hidden.is_cuda:
        raise ValueError("hidden must live on a CUDA device; host buffers go through spu_prune_host")
    hidden = hidden.contiguous()
    B, N, D = hidden.shape
    dev = hidden.device
    k = int(keep)
    with torch.cuda.device(dev):
        out_idx = torch.empty((B, max(k, 0)), dtype=torch.int32, device=dev)
        out_hidden = torch.empty((B, max(k, 0), D), dtype=hidden.dtype, device=dev)
        scores = torch.empty((B, N), dtype=torch.float32, device=dev) if want_scores else None
        o = SpuOpts()
        o.dtype = _dtype_code(hidden)
        o.stream = _stream_ptr(dev)
        if workspace is not None:
            o.workspace, o.workspace_bytes = workspace.data_ptr(), workspace.numel() * workspace.element_size()
        o.no_window = int(bool(no_window))
        o.out_scores = scores.data_ptr() if scores is not None else None
        o.device_status = device_status.data_ptr() if device_status is not None else None
        _check(lib.luvc_spu_prune_ex(hidden.data_ptr(), B, N, D, float(cutoff), k, out_idx.data_ptr(),
                                     out_hidden.data_ptr(), ctypes.byref(o)), "luvc_spu_prune_ex")
    if want_scores:
        return out_idx, out_hidden, scores
    return out_idx, out_hidden


def spu_prune_plain(hidden: torch.Tensor, keep: int, cutoff: float = 0.0):
    """The spec entry points luvc_spu_prune / luvc_spu_prune_f32 on the current torch stream."""
    hidden = hidden.contiguous()
    B, N, D = hidden.shape
    dev = hidden.device
    with torch.cuda.device(dev):
        out_idx = torch.empty((B, keep), dtype=torch.int32, device=dev)
        out_hidden = torch.empty((B, keep, D), dtype=hidden.dtype, device=dev)
        _check(lib.luvc_set_stream(_stream_ptr(dev)), "luvc_set_stream")
        fn = lib.luvc_spu_prune if _dtype_code(hidden) == BF16 else lib.luvc_spu_prune_f32
        _check(fn(hidden.data_ptr(), B, N, D, float(cutoff), int(keep), out_idx.data_ptr(), out_hidden.data_ptr()),
               "luvc_spu_prune")
    return out_idx, out_hidden


def spu_cascade(hidden: torch.Tensor, keeps, cutoffs=None):
    """luvc_spu_cascade: prunes back to back, stage t on the survivors of stage t-1.  Returns
    (out_idx [B, keeps[-1]] int32 into the original sequence, out_hidden [B, keeps[-1], D])."""
    hidden = hidden.contiguous()
    B, N, D = hidden.shape
    dev = hidden.device
    n = len(keeps)
    k_arr = (ctypes.c_int * n)(*[int(k) for k in keeps])
    c_arr = (ctypes.c_float * n)(*[float(c) for c in cutoffs]) if cutoffs is not None else None
    with torch.cuda.device(dev):
        out_idx = torch.empty((B, int(keeps[-1])), dtype=torch.int32, device=dev)
        out_hidden = torch.empty((B, int(keeps[-1]), D), dtype=hidden.dtype, device=dev)
        _check(lib.luvc_spu_cascade(hidden.data_ptr(), B, N, D, n, k_arr, c_arr, _dtype_code(hidden), _stream_ptr(dev),
                                    out_idx.data_ptr(), out_hidden.data_ptr()), "luvc_spu_cascade")
    return out_idx, out_hidden


SPU_STATIC_MAX_BYTES = 32 * 1024 * 1024


def spu_prune_static(hidden: torch.Tensor, keep: int, cutoff: float = 0.0):
    """luvc_spu_prune_static: the prune for callers that cannot allocate device memory.  The library
    call allocates nothing (its workspace is a fixed array inside the library, at most
    SPU_STATIC_MAX_BYTES); this wrapper still creates the two output tensors, which a caller with
    such a constraint would own beforehand.  Returns (out_idx [B,keep] int32, out_hidden [B,keep,D])."""
    if not hidden.is_cuda:
        raise ValueError("hidden must live on a CUDA device")
    hidden = hidden.contiguous()
    B, N, D = hidden.shape
    dev = hidden.device
    with torch.cuda.device(dev):
        out_idx = torch.empty((B, max(int(keep), 0)), dtype=torch.int32, device=dev)
        out_hidden = torch.empty((B, max(int(keep), 0), D), dtype=hidden.dtype, device=dev)
        _check(lib.luvc_spu_prune_static(hidden.data_ptr(), B, N, D, float(cutoff), int(keep), _dtype_code(hidden),
                                         _stream_ptr(dev), out_idx.data_ptr(), out_hidden.data_ptr()),
               "luvc_spu_prune_static")
    return out_idx, out_hidden


def oim_merge_host(tokens: torch.Tensor, target_count: int, out_tokens: torch.Tensor, out_sizes: torch.Tensor,
                   out_map: torch.Tensor) -> None:
    """luvc_oim_merge_host: all four tensors are HOST tensors (pinned recommended); synchronous."""
    B, H, W, D = tokens.shape
    _check(lib.luvc_set_stream(_stream_ptr(None)), "luvc_set_stream")
    _check(lib.luvc_oim_merge_host(tokens.data_ptr(), B, H, W, D, int(target_count), _dtype_code(tokens),
                                   out_tokens.data_ptr(), out_sizes.data_ptr(), out_map.data_ptr()),
           "luvc_oim_merge_host")


def spu_prune_host(hidden: torch.Tensor, keep: int, cutoff: float, out_idx: torch.Tensor,
                   out_hidden: torch.Tensor) -> None:
    """luvc_spu_prune_host: all tensors are HOST tensors (pinned recommended); synchronous."""
    B, N, D = hidden.shape
    _check(lib.luvc_set_stream(_stream_ptr(None)), "luvc_set_stream")
    _check(lib.luvc_spu_prune_host(hidden.data_ptr(), B, N, D, float(cutoff), int(keep), _dtype_code(hidden),
                                   out_idx.data_ptr(), out_hidden.data_ptr()), "luvc_spu_prune_host")
