"""Python face of the CPU oracle (test infrastructure, never part of the product path).

The arithmetic lives in ``luvc_oracle.cpp`` (plain double-precision C++); this
module only builds that file with g++, loads it with ctypes and marshals numpy
arrays.  Nothing here imports the CUDA package, and the CUDA package never
imports this module: only the tests, the smoke check and the CPU-baseline leg
of the benchmark do.

OIM: Section 3.2, Eq. 3 and the appendix on the iterative strategy.
SPU: Eq. 4-8 and Algorithm 2.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "luvc_oracle.cpp")
_LIB = os.path.join(_HERE, "libluvc_oracle.so")
_lock = threading.Lock()
_lib = None

DEFAULT_CUTOFF = 0.125  # this build's choice; the paper never states its cutoff


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than its source."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(
            ["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-pthread", _SRC, "-o", tmp]
        )
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    with _lock:
        if _lib is None:
            build()
            L = ctypes.CDLL(_LIB)
            c_int, c_dbl = ctypes.c_int, ctypes.c_double
            P = ctypes.c_void_p
            L.oracle_oim_final_dims.argtypes = [c_int, c_int, c_int, P, P]
            L.oracle_oim_schedule.argtypes = [c_int] * 7 + [P, P, c_int]
            L.oracle_oim_anyres_plan.argtypes = [c_int] * 4 + [P, P, P, P]
            L.oracle_oim_batch.argtypes = [P] + [c_int] * 10 + [P, P, P, P, c_dbl, P, P, c_int]
            L.oracle_dft_naive.argtypes = [P, c_int, P, P]
            L.oracle_dft_naive.restype = None
            L.oracle_fft.argtypes = [P, P, c_int, c_int, P, P]
            L.oracle_fft.restype = None
            L.oracle_spu_sigma.argtypes = [c_int, c_dbl]
            L.oracle_spu_mask.argtypes = [c_int, c_int, c_int, P]
            L.oracle_spu_mask.restype = None
            L.oracle_spu_scores.argtypes = [P, c_int, c_int, c_int, c_int, c_int, c_int, P]
            L.oracle_spu_scores_at.argtypes = [P, c_int, c_int, c_int, c_int, P, c_int, P]
            L.oracle_spu_select.argtypes = [P, c_int, c_int, P]
            _lib = L
    return _lib


def hardware_threads() -> int:
    return int(lib().oracle_hardware_threads())


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


# --------------------------------------------------------------------------- OIM


def oim_final_dims(H: int, W: int, target: int):
    hf, wf = ctypes.c_int(0), ctypes.c_int(0)
    rc = lib().oracle_oim_final_dims(H, W, target, ctypes.byref(hf), ctypes.byref(wf))
    if rc:
        raise ValueError("target_count %d has no admissible grid inside %dx%d" % (target, H, W))
    return hf.value, wf.value


def _per_axis(r):
    """r is one merge number for both axes, or a pair (r_h, r_w): cells removed per column in a
    height step, per row in a width step."""
    if isinstance(r, (tuple, list)):
        return int(r[0]), int(r[1])
    return int(r), int(r)


def oim_anyres_plan(H: int, W: int, ops: int, r: int = 2):
    """Per-axis merge numbers and final grid for an image whose sides differ (appendix, the variant
    that adjusts the merges to the aspect ratio): ((r_h, r_w), (Hf, Wf))."""
    v = [ctypes.c_int(0) for _ in range(4)]
    rc = lib().oracle_oim_anyres_plan(H, W, ops, r, *[ctypes.byref(c) for c in v])
    if rc:
        raise ValueError("%d operations with merge number %d leave nothing of a %dx%d grid" % (ops, r, H, W))
    return (v[0].value, v[1].value), (v[2].value, v[3].value)


def oim_schedule(H, W, Hf, Wf, r=2, height_first=False):
    """List of (axis, m) steps; axis 0 shrinks the width, axis 1 the height."""
    cap = 2 * (H + W) + 4
    axes = np.zeros(cap, np.int32)
    ms = np.zeros(cap, np.int32)
    r_h, r_w = _per_axis(r)
    n = lib().oracle_oim_schedule(H, W, Hf, Wf, r_w, r_h, int(height_first), _ptr(axes), _ptr(ms), cap)
    if n < 0:
        raise ValueError("grid %dx%d cannot be reduced to %dx%d" % (H, W, Hf, Wf))
    return [(int(axes[i]), int(ms[i])) for i in range(n)]


def oim(tokens, target=None, out_hw=None, r=2, height_first=False, trace=None, tol=1e-4, nthreads=None,
        matching="adjacent"):
    """Run (or, with ``trace``, replay) OIM on tokens [B,H,W,D] (float32-exact values).

    ``matching``: "adjacent" compares every even cell of a line with its one or two
    neighbours; "bipartite" compares it with every odd cell of the line (the reading
    behind the O(n_v^1.5 k) cost stated in Section 3.2).  ``r``: the merge number, or a pair
    (r_h, r_w) for the per-axis numbers of the appendix's aspect-ratio variant.

    Returns a dict: tokens [B,T,D] float64, sizes [B,T] int32, map [B,H*W] int32,
    trace [B,H*W-T] int32, stats [B,4] = (min selection margin, min direction
    margin, violations, deviations), grid (Hf, Wf).
    """
    x = _f32(tokens)
    B, H, W, D = x.shape
    Hf, Wf = out_hw if out_hw is not None else oim_final_dims(H, W, int(target))
    T = Hf * Wf
    out_tokens = np.zeros((B, T, D), np.float64)
    out_sizes = np.zeros((B, T), np.int32)
    out_map = np.full((B, H * W), -1, np.int32)
    trace_out = np.zeros((B, H * W - T), np.int32)
    stats = np.zeros((B, 4), np.float64)
    tin = None
    if trace is not None:
        tin = np.ascontiguousarray(np.asarray(trace, dtype=np.int32)).reshape(B, H * W - T)
    nt = nthreads or hardware_threads()
    r_h, r_w = _per_axis(r)
    rc = lib().oracle_oim_batch(_ptr(x), B, H, W, D, Hf, Wf, r_w, r_h, int(height_first),
                                {"adjacent": 0, "bipartite": 1}[matching], _ptr(out_tokens),
                                _ptr(out_sizes), _ptr(out_map), _ptr(tin), float(tol), _ptr(trace_out),
                                _ptr(stats), nt)
    if rc:
        raise ValueError("oracle OIM rejected the arguments (rc=%d)" % rc)
    return dict(tokens=out_tokens, sizes=out_sizes, map=out_map, trace=trace_out, stats=stats,
                grid=(Hf, Wf), threads=min(nt, B))


def oim_value_enhance(values, sizes):
    """Eq. 2's enhanced values V + log s, in double: values [B,T,D], sizes [B,T]."""
    v = np.asarray(values, dtype=np.float64)
    s = np.asarray(sizes, dtype=np.float64)
    return v + np.log(s)[..., None]


# --------------------------------------------------------------------------- SPU


def dft_naive(x):
    x = np.ascontiguousarray(np.asarray(x, dtype=np.float64))
    N = x.shape[0]
    re, im = np.zeros(N), np.zeros(N)
    lib().oracle_dft_naive(_ptr(x), N, _ptr(re), _ptr(im))
    return re + 1j * im


def fft(x, inverse=False):
    """The oracle's own mixed-radix FFT (inverse: without the 1/N factor)."""
    z = np.asarray(x, dtype=np.complex128)
    re = np.ascontiguousarray(z.real)
    im = np.ascontiguousarray(z.imag)
    N = re.shape[0]
    ore, oim_ = np.zeros(N), np.zeros(N)
    lib().oracle_fft(_ptr(re), _ptr(im), N, +1 if inverse else -1, _ptr(ore), _ptr(oim_))
    return ore + 1j * oim_


def spu_sigma(N: int, cutoff: float) -> int:
    if cutoff is None or cutoff <= 0:
        cutoff = DEFAULT_CUTOFF
    return int(lib().oracle_spu_sigma(N, float(cutoff)))


def spu_mask(N: int, sigma: int, hamming: bool = True):
    M = np.zeros(N, np.float64)
    lib().oracle_spu_mask(N, sigma, int(hamming), _ptr(M))
    return M


def spu_scores(x, sigma: int, hamming: bool = True, method: str = "fft", nthreads=None):
    """E[n] of Eq. 8 for one sequence x [N,D]; method 'naive' is Eq. 4/7 as O(N^2) sums."""
    x = _f32(x)
    N, D = x.shape
    E = np.zeros(N, np.float64)
    nt = nthreads or hardware_threads()
    rc = lib().oracle_spu_scores(_ptr(x), N, D, int(sigma), int(hamming), 0 if method == "naive" else 1, nt, _ptr(E))
    if rc:
        raise ValueError("oracle SPU rejected the arguments")
    return E


def spu_scores_at(x, sigma: int, tokens, hamming: bool = True):
    """Scores of the listed tokens only, by circular convolution with the filter's kernel."""
    x = _f32(x)
    N, D = x.shape
    t = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
    E = np.zeros(t.shape[0], np.float64)
    lib().oracle_spu_scores_at(_ptr(x), N, D, int(sigma), int(hamming), _ptr(t), t.shape[0], _ptr(E))
    return E


def spu_select(E, keep: int):
    E = np.ascontiguousarray(np.asarray(E, dtype=np.float64))
    idx = np.zeros(keep, np.int32)
    rc = lib().oracle_spu_select(_ptr(E), E.shape[0], int(keep), _ptr(idx))
    if rc:
        raise ValueError("keep=%d outside [0, %d]" % (keep, E.shape[0]))
    return idx


def spu(hidden, cutoff=None, keep=None, hamming=True, method="fft", nthreads=None):
    """Algorithm 2 on hidden [B,N,D]: scores, kept indices (ascending) and the kept rows."""
    x = _f32(hidden)
    B, N, D = x.shape
    sigma = spu_sigma(N, cutoff)
    scores = np.stack([spu_scores(x[b], sigma, hamming, method, nthreads) for b in range(B)])
    idx = np.stack([spu_select(scores[b], keep) for b in range(B)])
    kept = np.stack([x[b][idx[b]] for b in range(B)])
    return dict(scores=scores, idx=idx, hidden=kept, sigma=sigma)


def spu_cascade(hidden, keeps, cutoffs=None, hamming=True):
    """Section 3.3's progressive pruning as a plain loop: stage t applies Algorithm 2 to the survivors of
    stage t-1.  Returns per stage the scores and kept indices (in that stage's coordinates) and, at the
    end, the survivors as indices into the original sequence and their rows."""
    x = _f32(hidden)
    B = x.shape[0]
    total = np.tile(np.arange(x.shape[1], dtype=np.int32), (B, 1))
    stages = []
    for t, keep in enumerate(keeps):
        r = spu(x, cutoff=None if cutoffs is None else cutoffs[t], keep=int(keep), hamming=hamming)
        stages.append(r)
        total = np.stack([total[b][r["idx"][b]] for b in range(B)])
        x = r["hidden"]
    return dict(idx=total, hidden=x, stages=stages)
