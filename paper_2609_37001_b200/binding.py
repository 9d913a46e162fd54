"""Thin ctypes binding of libpsa.so: argument marshalling only.

Every step of the path runs inside the CUDA library; torch is used for device memory
and streams.  Importing this module without a built library, or calling it without a
CUDA device, raises -- there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpsa.so")

PSA_OK = 0
PSA_ERR_INVALID_ARG = -1
PSA_ERR_UNSUPPORTED = -2
PSA_ERR_CAPACITY = -3
PSA_ERR_CUDA = -4
PSA_ERR_TIMEOUT = -5
PSA_ERR_INTERNAL = -6


class PsaError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} ({status})")


class HeadParams(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("Tw", "To", "Ts", "Sw", "So", "Ss")]


class Tile(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("bt", "bh", "bw")]


class Problem(ctypes.Structure):
    _fields_ = [("n_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("tile", Tile),
                ("scale", ctypes.c_float), ("stride_head", ctypes.c_int64), ("stride_token", ctypes.c_int64)]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libpsa.so (built by paper_2609_37001_b200.build); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2609_37001_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64p = ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(ctypes.c_int64)
        hp, pp = ctypes.POINTER(HeadParams), ctypes.POINTER(Problem)
        L.psa_status_string.restype = ctypes.c_char_p
        L.psa_status_string.argtypes = [i32]
        L.psa_launch_count.restype = ctypes.c_int64
        L.psa_launch_count.argtypes = []
        L.psa_mask_sizes.argtypes = [hp, pp, i32, i32, i32, i64p, i64p]
        L.psa_mask_build.argtypes = [hp, pp, i32, i32, i32, vp, vp, vp, ctypes.c_int64, vp]
        L.psa_attn_fwd.argtypes = [vp, vp, vp, vp, vp, hp, pp, i32, i32, i32, vp]
        L.psa_attn_fwd_host.argtypes = [vp] * 10 + [hp, pp, i32, i32, i32, vp]
        L.psa_attn_fwd_noalloc.argtypes = [vp, vp, vp, vp, vp, hp, pp, i32, i32, i32, vp, ctypes.POINTER(ctypes.c_int32)]
        L.psa_attn_fwd_noalloc.restype = ctypes.c_int
        L.psa_attn_fwd_batched.argtypes = [vp, vp, vp, vp, vp, hp, pp, i32, ctypes.c_int64, i32, i32, i32, vp]
        L.psa_attn_fwd_joint.argtypes = [vp, vp, vp, vp, vp, hp, pp, ctypes.c_int64, i32, i32, i32, vp]
        L.psa_search_scratch_bytes.argtypes = [i32, i32, i32, i32]
        L.psa_search_scratch_bytes.restype = ctypes.c_int64
        L.psa_search_losses.argtypes = [vp, vp, vp, hp, i32, pp, i32, i32, i32, vp, vp, vp]
        L.psa_search_losses.restype = ctypes.c_int
        L.psa_search_select.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float), i32, ctypes.c_float]
        L.psa_search_select.restype = ctypes.c_int
        L.psa_search_select_at_sparsity.argtypes = L.psa_search_select.argtypes
        L.psa_search_select_at_sparsity.restype = ctypes.c_int
        L.psa_last_device_status.argtypes = [ctypes.POINTER(ctypes.c_int32)]
        L.psa_shutdown.argtypes = []
        L.psa_selftest_wait_timeout.argtypes = [i32, vp]
        L.psa_selftest_wait_timeout.restype = ctypes.c_int
        L.psa_profile_events.argtypes = [vp, vp]
        L.psa_profile_events.restype = ctypes.c_int
        for f in (L.psa_mask_sizes, L.psa_mask_build, L.psa_attn_fwd, L.psa_attn_fwd_host,
                  L.psa_last_device_status, L.psa_shutdown):
            f.restype = ctypes.c_int
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().psa_status_string(int(status)).decode()


def _check(status: int, what: str) -> None:
    if status != PSA_OK:
        raise PsaError(status, what)


_PARAMS_CACHE: dict = {}


def _params_array(head_params: Sequence[Sequence[int]]):
    """ctypes array of the per-head parameters (memoised: repeated calls with the same heads are common)."""
    key = tuple(tuple(int(x) for x in p) for p in head_params)
    arr = _PARAMS_CACHE.get(key)
    if arr is None:
        arr = (HeadParams * len(key))()
        for i, p in enumerate(key):
            arr[i] = HeadParams(*p)
        if len(_PARAMS_CACHE) > 64:
            _PARAMS_CACHE.clear()
        _PARAMS_CACHE[key] = arr
    return arr


def make_problem(n_heads: int, tile: Sequence[int], scale: float, stride_head: int, stride_token: int,
                 head_dim: int = 128) -> Problem:
    return Problem(int(n_heads), int(head_dim), Tile(*[int(x) for x in tile]), float(scale),
                   int(stride_head), int(stride_token))


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def _require_cuda(*tensors: torch.Tensor) -> None:
    for t in tensors:
        if not t.is_cuda:
            raise ValueError("device tensors required")


def psa_mask_sizes(head_params, grid: Sequence[int], tile: Sequence[int]) -> Tuple[int, int]:
    """(NB, nnz) for psa_mask_build's outputs.  Host arithmetic only."""
    prob = make_problem(len(head_params), tile, 1.0, 0, 128)
    nb, nnz = ctypes.c_int64(0), ctypes.c_int64(0)
    T, H, W = (int(x) for x in grid)
    _check(lib().psa_mask_sizes(_params_array(head_params), ctypes.byref(prob), T, H, W,
                                ctypes.byref(nb), ctypes.byref(nnz)), "psa_mask_sizes")
    return nb.value, nnz.value


def psa_mask_build(head_params, grid: Sequence[int], tile: Sequence[int], device="cuda",
                   out: Optional[Tuple[torch.Tensor, torch.Tensor, torch.Tensor]] = None,
                   stream: Optional[torch.cuda.Stream] = None):
    """Block mask uint8[heads, NB, NB], row_ptr int32[heads*NB+1], col_idx int32[nnz] on the device."""
    nh = len(head_params)
    T, H, W = (int(x) for x in grid)
    if out is None:
        nb, nnz = psa_mask_sizes(head_params, grid, tile)
        mask = torch.empty((nh, nb, nb), dtype=torch.uint8, device=device)
        row_ptr = torch.empty(nh * nb + 1, dtype=torch.int32, device=device)
        col_idx = torch.empty(max(nnz, 1), dtype=torch.int32, device=device)
    else:
        mask, row_ptr, col_idx = out
        nnz = None
    _require_cuda(mask, row_ptr, col_idx)
    prob = make_problem(nh, tile, 1.0, 0, 128)
    _check(lib().psa_mask_build(_params_array(head_params), ctypes.byref(prob), T, H, W, mask.data_ptr(),
                                row_ptr.data_ptr(), col_idx.data_ptr(), col_idx.numel(), _stream_ptr(stream)),
           "psa_mask_build")
    if nnz is not None:
        col_idx = col_idx[:nnz]
    return mask, row_ptr, col_idx


def psa_attn_fwd(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, head_params, grid: Sequence[int],
                 tile: Sequence[int], scale: float, out: Optional[torch.Tensor] = None,
                 lse: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """q, k, v: bf16 device tensors [heads, L, 128] (any head/token strides, last dim contiguous,
    shared by all three).  Returns (out bf16 like q, lse fp32 [heads, L])."""
    _require_cuda(q, k, v)
    if q.dtype != torch.bfloat16 or k.dtype != torch.bfloat16 or v.dtype != torch.bfloat16:
        raise ValueError("bf16 tensors required")
    nh, L, d = q.shape
    T, H, W = (int(x) for x in grid)
    if L != T * H * W or k.shape != q.shape or v.shape != q.shape:
        raise ValueError("shape mismatch")
    if q.stride() != k.stride() or q.stride() != v.stride() or q.stride(2) != 1:
        raise ValueError("q, k, v must share strides with a contiguous last dimension")
    if out is None:
        out = torch.empty_strided(q.shape, q.stride(), dtype=q.dtype, device=q.device)
    if lse is None:
        lse = torch.empty((nh, L), dtype=torch.float32, device=q.device)
    if out.stride() != q.stride() or not lse.is_contiguous():
        raise ValueError("out must share q's strides; lse must be contiguous")
    prob = make_problem(nh, tile, scale, q.stride(0), q.stride(1), d)
    _check(lib().psa_attn_fwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), lse.data_ptr(),
                              _params_array(head_params), ctypes.byref(prob), T, H, W, _stream_ptr(stream)),
           "psa_attn_fwd")
    return out, lse


def psa_attn_fwd_batched(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, head_params, grid: Sequence[int],
                         tile: Sequence[int], scale: float, out: Optional[torch.Tensor] = None,
                         lse: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """Batched call: q, k, v are bf16 device tensors [batch, heads, L, 128] sharing strides (last dim
    contiguous); every sample uses the same per-head masks.  Returns (out like q, lse fp32
    [batch, heads, L])."""
    _require_cuda(q, k, v)
    if q.dtype != torch.bfloat16 or k.dtype != torch.bfloat16 or v.dtype != torch.bfloat16:
        raise ValueError("bf16 tensors required")
    nb, nh, L, d = q.shape
    T, H, W = (int(x) for x in grid)
    if L != T * H * W or k.shape != q.shape or v.shape != q.shape or len(head_params) != nh:
        raise ValueError("shape mismatch")
    if q.stride() != k.stride() or q.stride() != v.stride() or q.stride(3) != 1:
        raise ValueError("q, k, v must share strides with a contiguous last dimension")
    if out is None:
        out = torch.empty_strided(q.shape, q.stride(), dtype=q.dtype, device=q.device)
    if lse is None:
        lse = torch.empty((nb, nh, L), dtype=torch.float32, device=q.device)
    if out.stride() != q.stride() or not lse.is_contiguous():
        raise ValueError("out must share q's strides; lse must be contiguous")
    prob = make_problem(nh, tile, scale, q.stride(1), q.stride(2), d)
    _check(lib().psa_attn_fwd_batched(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), lse.data_ptr(),
                                      _params_array(head_params), ctypes.byref(prob), nb, q.stride(0), T, H, W,
                                      _stream_ptr(stream)), "psa_attn_fwd_batched")
    return out, lse


def psa_attn_fwd_joint(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, head_params, grid: Sequence[int],
                       tile: Sequence[int], scale: float, n_text: int, out: Optional[torch.Tensor] = None,
                       lse: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None):
    """Joint video + text sequence: q, k, v are bf16 device tensors [heads, L + n_text, 128] with the
    video tokens first.  The stripe mask applies between video tokens; text keys are attended by every
    query and text queries attend every key.  Returns (out like q, lse fp32 [heads, L + n_text])."""
    _require_cuda(q, k, v)
    if q.dtype != torch.bfloat16 or k.dtype != torch.bfloat16 or v.dtype != torch.bfloat16:
        raise ValueError("bf16 tensors required")
    nh, Lt, d = q.shape
    T, H, W = (int(x) for x in grid)
    if Lt != T * H * W + int(n_text) or k.shape != q.shape or v.shape != q.shape:
        raise ValueError("shape mismatch")
    if q.stride() != k.stride() or q.stride() != v.stride() or q.stride(2) != 1:
        raise ValueError("q, k, v must share strides with a contiguous last dimension")
    if out is None:
        out = torch.empty_strided(q.shape, q.stride(), dtype=q.dtype, device=q.device)
    if lse is None:
        lse = torch.empty((nh, Lt), dtype=torch.float32, device=q.device)
    if out.stride() != q.stride() or not lse.is_contiguous():
        raise ValueError("out must share q's strides; lse must be contiguous")
    prob = make_problem(nh, tile, scale, q.stride(0), q.stride(1), d)
    _check(lib().psa_attn_fwd_joint(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), lse.data_ptr(),
                                    _params_array(head_params), ctypes.byref(prob), int(n_text), T, H, W,
                                    _stream_ptr(stream)), "psa_attn_fwd_joint")
    return out, lse


def psa_attn_fwd_noalloc(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: torch.Tensor, lse: torch.Tensor,
                         head_params, grid: Sequence[int], tile: Sequence[int], scale: float,
                         stream: Optional[torch.cuda.Stream] = None, check: bool = True) -> int:
    """psa_attn_fwd through the entry point that never allocates device memory: for callers whose device
    memory is owned by someone else's pool, or who cannot afford the device-wide synchronisation of
    cudaMalloc.  The caller supplies ``out`` and ``lse`` (nothing is allocated here either); the library's
    scratch is a fixed array inside the library image, so the problem must fit its limits (see psa.h).
    With ``check`` the call synchronises the stream and raises on a device-side timeout; it returns the
    diagnostic word."""
    _require_cuda(q, k, v, out, lse)
    nh, L, d = q.shape
    T, H, W = (int(x) for x in grid)
    if L != T * H * W or k.shape != q.shape or v.shape != q.shape or out.shape != q.shape:
        raise ValueError("shape mismatch")
    if q.stride() != k.stride() or q.stride() != v.stride() or q.stride() != out.stride() or q.stride(2) != 1:
        raise ValueError("q, k, v, out must share strides with a contiguous last dimension")
    if not lse.is_contiguous() or tuple(lse.shape) != (nh, L):
        raise ValueError("lse must be a contiguous [heads, L] tensor")
    prob = make_problem(nh, tile, scale, q.stride(0), q.stride(1), d)
    detail = ctypes.c_int32(0)
    _check(lib().psa_attn_fwd_noalloc(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), lse.data_ptr(),
                                      _params_array(head_params), ctypes.byref(prob), T, H, W, _stream_ptr(stream),
                                      ctypes.byref(detail) if check else None), "psa_attn_fwd_noalloc")
    return detail.value


def psa_attn_fwd_host(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: torch.Tensor, lse: torch.Tensor,
                      staging: Sequence[torch.Tensor], head_params, grid: Sequence[int], tile: Sequence[int],
                      scale: float, stream: Optional[torch.cuda.Stream] = None) -> None:
    """Host-tensor variant: q, k, v, out (bf16 [heads, L, 128], contiguous) and lse (fp32 [heads, L])
    live in host memory; ``staging`` = (d_q, d_k, d_v, d_out, d_lse) are device buffers of the same
    shapes.  Copies in, runs, copies out and synchronises the stream."""
    d_q, d_k, d_v, d_out, d_lse = staging
    _require_cuda(d_q, d_k, d_v, d_out, d_lse)
    for t in (q, k, v, out, lse):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("contiguous host tensors required")
    nh, L, d = q.shape
    T, H, W = (int(x) for x in grid)
    prob = make_problem(nh, tile, scale, q.stride(0), q.stride(1), d)
    _check(lib().psa_attn_fwd_host(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), lse.data_ptr(),
                                   d_q.data_ptr(), d_k.data_ptr(), d_v.data_ptr(), d_out.data_ptr(),
                                   d_lse.data_ptr(), _params_array(head_params), ctypes.byref(prob), T, H, W,
                                   _stream_ptr(stream)), "psa_attn_fwd_host")


def psa_search_scratch_bytes(n_cand: int, grid: Sequence[int]) -> int:
    """Bytes of device scratch psa_search_losses needs for ``n_cand`` candidates on this token grid."""
    T, H, W = (int(x) for x in grid)
    n = int(lib().psa_search_scratch_bytes(int(n_cand), T, H, W))
    if n < 0:
        _check(n, "psa_search_scratch_bytes")
    return n


def psa_search_losses(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, candidates, grid: Sequence[int],
                      tile: Sequence[int], scale: float, scratch: Optional[torch.Tensor] = None,
                      stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Inner loop of PSA-Search for one head (Algorithm 3): q, k, v are bf16 [L, 128] device tensors of
    that head, ``candidates`` a sequence of six-integer masks.  Returns the fp32 loss of every candidate
    against full attention (device tensor).  ``scratch`` (uint8, psa_search_scratch_bytes long) is
    allocated when not given."""
    _require_cuda(q, k, v)
    L, d = q.shape
    T, H, W = (int(x) for x in grid)
    if L != T * H * W or k.shape != q.shape or v.shape != q.shape:
        raise ValueError("shape mismatch")
    if q.stride() != k.stride() or q.stride() != v.stride() or q.stride(1) != 1:
        raise ValueError("q, k, v must share strides with a contiguous last dimension")
    n_cand = len(candidates)
    need = psa_search_scratch_bytes(n_cand, grid)
    if scratch is None:
        scratch = torch.empty(need, dtype=torch.uint8, device=q.device)
    if scratch.numel() * scratch.element_size() < need or not scratch.is_contiguous():
        raise ValueError("scratch too small")
    losses = torch.empty(n_cand, dtype=torch.float32, device=q.device)
    prob = make_problem(1, tile, scale, 0, q.stride(0), d)
    _check(lib().psa_search_losses(q.data_ptr(), k.data_ptr(), v.data_ptr(), _params_array(candidates), n_cand,
                                   ctypes.byref(prob), T, H, W, scratch.data_ptr(), losses.data_ptr(),
                                   _stream_ptr(stream)), "psa_search_losses")
    return losses


def psa_search_select(losses: Sequence[float], sparsity: Sequence[float], alpha: float) -> int:
    """Selection step of PSA-Search (Algorithm 3) on host arrays; returns the chosen candidate's index."""
    n = len(losses)
    if len(sparsity) != n:
        raise ValueError("losses and sparsity differ in length")
    la = (ctypes.c_float * n)(*[float(x) for x in losses])
    sa = (ctypes.c_float * n)(*[float(x) for x in sparsity])
    r = int(lib().psa_search_select(la, sa, n, float(alpha)))
    if r < 0:
        _check(r, "psa_search_select")
    return r


def psa_search_select_at_sparsity(losses: Sequence[float], sparsity: Sequence[float], target: float) -> int:
    """Second interface of PSA-Search: minimal-loss candidate among those at least ``target`` sparse;
    -1 when none is."""
    n = len(losses)
    if len(sparsity) != n:
        raise ValueError("losses and sparsity differ in length")
    la = (ctypes.c_float * n)(*[float(x) for x in losses])
    sa = (ctypes.c_float * n)(*[float(x) for x in sparsity])
    r = int(lib().psa_search_select_at_sparsity(la, sa, n, float(target)))
    if r == -3:  # PSA_ERR_CAPACITY: no candidate reaches the target
        return -1
    if r < 0:
        _check(r, "psa_search_select_at_sparsity")
    return r


def psa_last_device_status() -> Tuple[int, int]:
    """Synchronises the device; returns (status, detail) left by the last psa_attn_fwd."""
    detail = ctypes.c_int32(0)
    st = lib().psa_last_device_status(ctypes.byref(detail))
    return st, detail.value


def psa_profile_events(start: Optional[torch.cuda.Event], stop: Optional[torch.cuda.Event]) -> None:
    """Record ``start``/``stop`` around the attention kernel of every later psa_attn_fwd (None, None: off).
    The events must have been created with enable_timing=True and recorded once (so that they exist)."""
    a = None if start is None else ctypes.c_void_p(start.cuda_event)
    b = None if stop is None else ctypes.c_void_p(stop.cuda_event)
    _check(lib().psa_profile_events(a, b), "psa_profile_events")


def psa_selftest_wait_timeout(limit_ms: int = 20, stream: Optional[torch.cuda.Stream] = None) -> None:
    """Launches the bounded-wait self-test kernel (see psa.h); read the outcome with psa_last_device_status()."""
    _check(lib().psa_selftest_wait_timeout(int(limit_ms), _stream_ptr(stream)), "psa_selftest_wait_timeout")


def psa_launch_count() -> int:
    return int(lib().psa_launch_count())


def psa_shutdown() -> None:
    _check(lib().psa_shutdown(), "psa_shutdown")
