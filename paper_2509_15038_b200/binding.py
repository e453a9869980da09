"""Thin ctypes binding of ``libcurdkv.so`` (declared in ``include/curdkv.h``).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  torch supplies device memory and the current stream.  There is no
CPU or eager fallback: if the library is missing or a call fails, an exception
is raised.
"""
from __future__ import annotations

import ctypes
from pathlib import Path
from typing import Optional

import torch

_LIB_PATH = Path(__file__).resolve().parent / "libcurdkv.so"
_lib = None

STATUS_OK = 0
DEV_TIMEOUT = 0x1
DEV_BAD_INDEX = 0x2
DEV_CACHE_FULL = 0x4
DEV_NOT_SPD = 0x8

EXPORTS = (
    "curdkv_workspace_bytes", "curdkv_score", "curdkv_select", "curdkv_compact",
    "curdkv_gqa_map", "curdkv_device_status", "curdkv_launch_count", "curdkv_status_string",
    "curdkv_score_static", "curdkv_host_arena_bytes", "curdkv_compress_host",
    "curdkv_profile_next_score", "curdkv_cache_workspace_bytes", "curdkv_cache_append",
    "curdkv_cache_compress", "curdkv_attention_workspace_bytes", "curdkv_attention_out",
    "curdkv_eviction_loss", "curdkv_gqa_expand", "curdkv_cache_compress_inplace",
    "curdkv_selftest_bounded_wait", "curdkv_selftest_gather_wait", "curdkv_compress", "curdkv_cache_step",
)


class CurdkvError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {status_string(code)} (status {code})")
        self.code = code


class Desc(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32), ("kv_heads", ctypes.c_int32), ("q_heads", ctypes.c_int32),
        ("n_max", ctypes.c_int32), ("d", ctypes.c_int32), ("r", ctypes.c_int32),
        ("k_stride_b", ctypes.c_int64), ("k_stride_h", ctypes.c_int64), ("k_stride_n", ctypes.c_int64),
        ("v_stride_b", ctypes.c_int64), ("v_stride_h", ctypes.c_int64), ("v_stride_n", ctypes.c_int64),
        ("seqlens", ctypes.c_void_p),
        ("score_mode", ctypes.c_int32), ("use_projection", ctypes.c_int32),
        ("raw_scores", ctypes.c_int32), ("whiten", ctypes.c_int32), ("ridge", ctypes.c_double),
    ]


class Cache(ctypes.Structure):
    """``curdkv_cache``: device pointers of one layer's generation-phase cache."""

    _fields_ = [
        ("K", ctypes.c_void_p), ("V", ctypes.c_void_p), ("raw", ctypes.c_void_p),
        ("pos", ctypes.c_void_p), ("count", ctypes.c_void_p), ("total", ctypes.c_void_p),
        ("capacity", ctypes.c_int32),
    ]


def load():
    """Load the CUDA library, compiling it first with nvcc if it is missing or older than its
    sources (a fresh checkout has no binary).  There is no other implementation to fall back to:
    if the build fails, this raises."""
    global _lib
    if _lib is not None:
        return _lib
    from . import build as _build

    try:
        _build.build_library()
    except Exception as exc:
        if not _LIB_PATH.exists():
            raise RuntimeError(f"{_LIB_PATH} is missing and could not be built: {exc} "
                               "(there is no fallback path)") from exc
    lib = ctypes.CDLL(str(_LIB_PATH))
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    dp = ctypes.POINTER(Desc)
    lib.curdkv_workspace_bytes.restype = ctypes.c_size_t
    lib.curdkv_workspace_bytes.argtypes = [dp, i32, i32]
    lib.curdkv_score.restype = ctypes.c_int
    lib.curdkv_score.argtypes = [vp, vp, vp, i32, dp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.curdkv_score_static.restype = ctypes.c_int
    lib.curdkv_score_static.argtypes = [vp, vp, vp, i32, dp, vp, vp, vp, vp]
    lib.curdkv_select.restype = ctypes.c_int
    lib.curdkv_select.argtypes = [vp, dp, i32, vp, i32, i32, i32, ctypes.c_double, vp, vp, vp, vp,
                                  ctypes.c_size_t, vp]
    lib.curdkv_compact.restype = ctypes.c_int
    lib.curdkv_compact.argtypes = [vp, vp, dp, vp, i64, vp, vp, vp, vp, i64, vp, vp]
    lib.curdkv_compress.restype = ctypes.c_int
    lib.curdkv_compress.argtypes = [vp, vp, vp, i32, dp, i32, vp, i32, i32, i32, ctypes.c_double,
                                    vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.curdkv_host_arena_bytes.restype = ctypes.c_size_t
    lib.curdkv_host_arena_bytes.argtypes = [dp, i32, i32, i32]
    lib.curdkv_compress_host.restype = ctypes.c_int
    lib.curdkv_compress_host.argtypes = [vp, vp, vp, i32, dp, i32, i32, i32, i32, ctypes.c_double,
                                         vp, vp, vp, vp, vp, vp, ctypes.c_size_t, i32,
                                         ctypes.POINTER(ctypes.c_uint32)]
    lib.curdkv_gqa_map.restype = ctypes.c_int
    lib.curdkv_gqa_map.argtypes = [dp, vp, vp]
    lib.curdkv_gqa_expand.restype = ctypes.c_int
    lib.curdkv_gqa_expand.argtypes = [dp, vp, vp, i32, vp, vp, vp]
    lib.curdkv_device_status.restype = ctypes.c_int
    lib.curdkv_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32), vp]
    cp = ctypes.POINTER(Cache)
    lib.curdkv_cache_workspace_bytes.restype = ctypes.c_size_t
    lib.curdkv_cache_workspace_bytes.argtypes = [i32, i32, i32, i32, i32]
    lib.curdkv_cache_append.restype = ctypes.c_int
    lib.curdkv_cache_append.argtypes = [cp, vp, vp, vp, i32, dp, vp, ctypes.c_size_t, vp]
    lib.curdkv_cache_compress.restype = ctypes.c_int
    lib.curdkv_cache_compress.argtypes = [cp, cp, dp, i32, i32, i32, vp, ctypes.c_size_t, vp]
    lib.curdkv_cache_compress_inplace.restype = ctypes.c_int
    lib.curdkv_cache_compress_inplace.argtypes = [cp, dp, i32, i32, i32, vp, ctypes.c_size_t, vp]
    lib.curdkv_cache_step.restype = ctypes.c_int
    lib.curdkv_cache_step.argtypes = [cp, vp, vp, vp, i32, dp, i32, i32, i32, vp, ctypes.c_size_t, vp]
    lib.curdkv_attention_workspace_bytes.restype = ctypes.c_size_t
    lib.curdkv_attention_workspace_bytes.argtypes = [dp]
    lib.curdkv_attention_out.restype = ctypes.c_int
    lib.curdkv_attention_out.argtypes = [vp, i32, i64, i64, i64, vp, vp, dp, vp, vp, i64, vp,
                                         ctypes.c_float, i32, vp, vp, ctypes.c_size_t, vp]
    lib.curdkv_eviction_loss.restype = ctypes.c_int
    lib.curdkv_eviction_loss.argtypes = [vp, vp, i32, i64, vp, vp, vp]
    lib.curdkv_selftest_bounded_wait.restype = ctypes.c_int
    lib.curdkv_selftest_bounded_wait.argtypes = [ctypes.c_uint64, vp, vp]
    lib.curdkv_selftest_gather_wait.restype = ctypes.c_int
    lib.curdkv_selftest_gather_wait.argtypes = [ctypes.c_uint64, vp, vp]
    lib.curdkv_profile_next_score.restype = ctypes.c_int
    lib.curdkv_profile_next_score.argtypes = [vp, vp]
    lib.curdkv_launch_count.restype = ctypes.c_uint64
    lib.curdkv_launch_count.argtypes = []
    lib.curdkv_status_string.restype = ctypes.c_char_p
    lib.curdkv_status_string.argtypes = [ctypes.c_int]
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load().curdkv_status_string(int(code)).decode()


def launch_count() -> int:
    return int(load().curdkv_launch_count())


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    # an empty view of a live allocation still has a valid base address
    return ctypes.c_void_p(t.data_ptr() if t.numel() else t.untyped_storage().data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(code: int, what: str):
    if code != STATUS_OK:
        raise CurdkvError(code, what)


def make_desc(K: torch.Tensor, V: torch.Tensor, r: int, *, q_heads: Optional[int] = None,
              seqlens: Optional[torch.Tensor] = None, score_mode: int = 0,
              use_projection: int = 1, raw_scores: int = 0, whiten: int = 0,
              ridge: float = 0.0) -> Desc:
    """Descriptor of bf16 K, V ``[B, Hkv, n_max, d]`` (any strides with d contiguous)."""
    if K.dtype != torch.bfloat16 or V.dtype != torch.bfloat16:
        raise TypeError("K and V must be bf16")
    if K.dim() != 4 or K.shape != V.shape or K.stride(3) != 1 or V.stride(3) != 1:
        raise ValueError("K and V must be [B, Hkv, n, d] with a contiguous last axis")
    if seqlens is not None and (seqlens.dtype != torch.int32 or seqlens.numel() != K.shape[0]
                                or not seqlens.is_contiguous()):
        raise ValueError("seqlens must be a contiguous int32 tensor of length B")
    B, H, n, d = K.shape
    return Desc(B, H, q_heads or H, n, d, int(r),
                K.stride(0), K.stride(1), K.stride(2), V.stride(0), V.stride(1), V.stride(2),
                seqlens.data_ptr() if seqlens is not None else None,
                int(score_mode), int(use_projection), int(raw_scores), int(whiten), float(ridge))


def workspace_bytes(desc: Desc, max_budget: int = 0, adaptive: bool = False) -> int:
    return int(load().curdkv_workspace_bytes(ctypes.byref(desc), int(max_budget), int(adaptive)))


def alloc_workspace(desc: Desc, max_budget: int = 1, adaptive: bool = False, device=None) -> torch.Tensor:
    nbytes = workspace_bytes(desc, max_budget, adaptive)
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device or "cuda")


def curdkv_score(K, V, G, desc: Desc, workspace: torch.Tensor, scores=None, head_sums=None):
    """Alg. 1 (scoring steps).  G: fp32 device tensor [d, r] or [Hkv, d, r].  Returns (scores, head_sums)."""
    dev = K.device
    if scores is None:
        scores = torch.empty((desc.batch, desc.kv_heads, desc.n_max), dtype=torch.float32, device=dev)
    if head_sums is None:
        head_sums = torch.empty((desc.batch, desc.kv_heads), dtype=torch.float32, device=dev)
    g_per_head = int(G is not None and G.dim() == 3)
    if G is not None and (G.dtype != torch.float32 or not G.is_contiguous()):
        raise TypeError("G must be a contiguous fp32 tensor")
    code = load().curdkv_score(_ptr(K), _ptr(V), _ptr(G), g_per_head, ctypes.byref(desc),
                               _ptr(scores), _ptr(head_sums), _ptr(workspace),
                               workspace.numel(), _stream())
    _check(code, "curdkv_score")
    return scores, head_sums


def curdkv_score_static(K, V, G, desc: Desc, scores=None, head_sums=None, status_flags=None):
    """curdkv_score for callers that may not allocate device memory: the library's built-in
    scratch array stands in for the workspace (see the header for its limit and sharing rules).
    Output tensors are still the caller's; pass them in to keep this call allocation-free."""
    dev = K.device
    if scores is None:
        scores = torch.empty((desc.batch, desc.kv_heads, desc.n_max), dtype=torch.float32, device=dev)
    if head_sums is None:
        head_sums = torch.empty((desc.batch, desc.kv_heads), dtype=torch.float32, device=dev)
    g_per_head = int(G is not None and G.dim() == 3)
    code = load().curdkv_score_static(_ptr(K), _ptr(V), _ptr(G), g_per_head, ctypes.byref(desc),
                                      _ptr(scores), _ptr(head_sums), _ptr(status_flags), _stream())
    _check(code, "curdkv_score_static")
    return scores, head_sums


def curdkv_select(scores, desc: Desc, budget: int, *, num_sink: int = 0, window: int = 0,
                  head_budgets=None, adaptive: bool = False, alpha: float = 0.2,
                  workspace: Optional[torch.Tensor] = None, idx=None, head_counts=None,
                  head_offsets=None):
    """Alg. 1 (sinks, top-k, union) / AdaCurDKV.  Returns (idx, head_counts, head_offsets)."""
    dev = scores.device
    P = desc.batch * desc.kv_heads
    if idx is None:
        if adaptive:
            idx = torch.empty((P * max(min(budget, desc.n_max), 0) + 1,), dtype=torch.int32, device=dev)[:-1]
        else:
            idx = torch.empty((P * max(budget, 0) + 1,), dtype=torch.int32, device=dev)
            idx = idx[: P * max(budget, 0)].view(desc.batch, desc.kv_heads, max(budget, 0))
    if head_counts is None:
        head_counts = torch.empty((desc.batch, desc.kv_heads), dtype=torch.int32, device=dev)
    if head_offsets is None:
        head_offsets = torch.empty((P + 1,), dtype=torch.int32, device=dev)
    code = load().curdkv_select(_ptr(scores), ctypes.byref(desc), int(budget), _ptr(head_budgets),
                                int(num_sink), int(window), int(adaptive), float(alpha),
                                _ptr(idx), _ptr(head_counts), _ptr(head_offsets), _ptr(workspace),
                                0 if workspace is None else workspace.numel(), _stream())
    _check(code, "curdkv_select")
    return idx, head_counts, head_offsets


def curdkv_compact(K, V, desc: Desc, idx, head_counts, head_offsets=None, *, packed: bool = False,
                   K_out=None, V_out=None, workspace: Optional[torch.Tensor] = None):
    """Alg. 1 (gather step).  Fixed layout -> [B, Hkv, budget, d]; packed -> [capacity, d]."""
    dev = K.device
    if packed:
        rows = idx.numel()
        shape, out_stride_h, idx_stride = (rows, desc.d), 0, 0
    else:
        budget = idx.shape[-1]
        shape, out_stride_h, idx_stride = (desc.batch, desc.kv_heads, budget, desc.d), budget, budget
    if K_out is None:
        K_out = torch.zeros(shape, dtype=torch.bfloat16, device=dev)
    if V_out is None:
        V_out = torch.zeros(shape, dtype=torch.bfloat16, device=dev)
    if not packed and out_stride_h == 0:
        return K_out, V_out
    code = load().curdkv_compact(_ptr(K), _ptr(V), ctypes.byref(desc), _ptr(idx), idx_stride,
                                 _ptr(head_counts), _ptr(head_offsets), _ptr(K_out), _ptr(V_out),
                                 out_stride_h, _ptr(workspace), _stream())
    _check(code, "curdkv_compact")
    return K_out, V_out


def curdkv_compress(K, V, G, desc: Desc, budget: int, workspace: torch.Tensor, *, num_sink: int = 0,
                    window: int = 0, head_budgets=None, adaptive: bool = False, alpha: float = 0.2,
                    scores=None, head_sums=None, idx=None, head_counts=None, head_offsets=None,
                    K_out=None, V_out=None):
    """Alg. 1 (all steps) (or AdaCurDKV) in one call; the workspace must come from
    ``alloc_workspace(desc, budget, adaptive)``.  Returns (scores, head_sums, idx, head_counts,
    head_offsets, K_out, V_out) with the layouts of the three separate calls."""
    dev = K.device
    P, b = desc.batch * desc.kv_heads, max(budget, 0)
    if scores is None:
        scores = torch.empty((desc.batch, desc.kv_heads, desc.n_max), dtype=torch.float32, device=dev)
    if head_sums is None:
        head_sums = torch.empty((desc.batch, desc.kv_heads), dtype=torch.float32, device=dev)
    rows = P * (min(b, desc.n_max) if adaptive else b)
    if idx is None:
        idx = torch.empty((rows + 1,), dtype=torch.int32, device=dev)[:rows]
        if not adaptive:
            idx = idx.view(desc.batch, desc.kv_heads, b)
    if head_counts is None:
        head_counts = torch.empty((desc.batch, desc.kv_heads), dtype=torch.int32, device=dev)
    if head_offsets is None:
        head_offsets = torch.empty((P + 1,), dtype=torch.int32, device=dev)
    shape = (rows, desc.d) if adaptive else (desc.batch, desc.kv_heads, b, desc.d)
    if K_out is None:
        K_out = torch.zeros(shape, dtype=torch.bfloat16, device=dev)
    if V_out is None:
        V_out = torch.zeros(shape, dtype=torch.bfloat16, device=dev)
    g_per_head = int(G is not None and G.dim() == 3)
    code = load().curdkv_compress(_ptr(K), _ptr(V), _ptr(G), g_per_head, ctypes.byref(desc), int(budget),
                                  _ptr(head_budgets), int(num_sink), int(window), int(adaptive), float(alpha),
                                  _ptr(scores), _ptr(head_sums), _ptr(idx), _ptr(head_counts),
                                  _ptr(head_offsets), _ptr(K_out), _ptr(V_out), _ptr(workspace),
                                  workspace.numel(), _stream())
    _check(code, "curdkv_compress")
    return scores, head_sums, idx, head_counts, head_offsets, K_out, V_out


class HostBuffers:
    """Pinned host outputs and the device arena of :func:`curdkv_compress_host`."""

    def __init__(self, desc: Desc, budget: int, adaptive: bool, chunk_batch: int, device="cuda"):
        P = desc.batch * desc.kv_heads
        rows = P * (min(budget, desc.n_max) if adaptive else budget)
        pin = dict(pin_memory=True)
        self.idx = torch.empty((max(rows, 1),), dtype=torch.int32, **pin)[:rows]
        self.K_out = torch.empty((max(rows, 1), desc.d), dtype=torch.bfloat16, **pin)[:rows]
        self.V_out = torch.empty((max(rows, 1), desc.d), dtype=torch.bfloat16, **pin)[:rows]
        self.counts = torch.empty((desc.batch, desc.kv_heads), dtype=torch.int32, **pin)
        self.offsets = torch.empty((P + 1,), dtype=torch.int32, **pin)
        nbytes = int(load().curdkv_host_arena_bytes(ctypes.byref(desc), int(budget), int(adaptive),
                                                    int(chunk_batch)))
        if nbytes == 0:
            raise ValueError("invalid shape for curdkv_compress_host")
        self.arena = torch.empty((nbytes,), dtype=torch.uint8, device=device)
        self.chunk_batch = int(chunk_batch)
        if not adaptive:
            self.idx = self.idx.view(desc.batch, desc.kv_heads, budget)
            self.K_out = self.K_out.view(desc.batch, desc.kv_heads, budget, desc.d)
            self.V_out = self.V_out.view(desc.batch, desc.kv_heads, budget, desc.d)


def curdkv_compress_host(K_host, V_host, G_host, desc: Desc, budget: int, buffers: HostBuffers, *,
                         num_sink: int = 0, window: int = 0, adaptive: bool = False,
                         alpha: float = 0.2) -> int:
    """Whole path on host-resident K, V (CPU tensors, ideally pinned); ``desc`` must describe the
    host tensors (``desc.seqlens`` = address of a host int32 array or None).  Results land in
    ``buffers``; returns the device status flags."""
    for t in (K_host, V_host):
        if t.device.type != "cpu" or not t.is_contiguous():
            raise ValueError("host tensors must be contiguous CPU tensors")
    flags = ctypes.c_uint32(0)
    g_per_head = int(G_host is not None and G_host.dim() == 3)
    code = load().curdkv_compress_host(
        _ptr(K_host), _ptr(V_host), _ptr(G_host), g_per_head, ctypes.byref(desc), int(budget),
        int(num_sink), int(window), int(adaptive), float(alpha), _ptr(buffers.K_out),
        _ptr(buffers.V_out), _ptr(buffers.idx), _ptr(buffers.counts), _ptr(buffers.offsets),
        _ptr(buffers.arena), buffers.arena.numel(), buffers.chunk_batch, ctypes.byref(flags))
    _check(code, "curdkv_compress_host")
    return int(flags.value)


class DeviceCache:
    """Torch-owned buffers of one generation-phase cache plus the ``curdkv_cache`` view of them."""

    def __init__(self, batch: int, kv_heads: int, capacity: int, d: int, device="cuda"):
        self.batch, self.kv_heads, self.capacity, self.d = batch, kv_heads, capacity, d
        self.K = torch.zeros((batch, kv_heads, capacity, d), dtype=torch.bfloat16, device=device)
        self.V = torch.zeros_like(self.K)
        self.raw = torch.zeros((batch, kv_heads, capacity), dtype=torch.float32, device=device)
        self.pos = torch.full((batch, kv_heads, capacity), -1, dtype=torch.int32, device=device)
        self.count = torch.zeros((batch,), dtype=torch.int32, device=device)
        self.total = torch.zeros((batch,), dtype=torch.int32, device=device)
        self.c = Cache(self.K.data_ptr(), self.V.data_ptr(), self.raw.data_ptr(), self.pos.data_ptr(),
                       self.count.data_ptr(), self.total.data_ptr(), capacity)


def cache_workspace(batch: int, kv_heads: int, t_max: int, capacity: int, budget: int,
                    device="cuda") -> torch.Tensor:
    nbytes = int(load().curdkv_cache_workspace_bytes(batch, kv_heads, t_max, capacity, budget))
    if nbytes == 0:
        raise ValueError("invalid shape for the generation-phase cache")
    return torch.zeros((nbytes,), dtype=torch.uint8, device=device)


def curdkv_cache_append(cache: DeviceCache, K_new, V_new, G, workspace: torch.Tensor, *,
                        t_new: Optional[torch.Tensor] = None) -> None:
    """Sec. 3.2, generation phase: score K_new, V_new ``[B, Hkv, t, d]`` and append them."""
    desc = make_desc(K_new, V_new, G.shape[-1], seqlens=t_new)
    code = load().curdkv_cache_append(ctypes.byref(cache.c), _ptr(K_new), _ptr(V_new), _ptr(G),
                                      int(G.dim() == 3), ctypes.byref(desc), _ptr(workspace),
                                      workspace.numel(), _stream())
    _check(code, "curdkv_cache_append")


def curdkv_cache_compress(src: DeviceCache, dst: DeviceCache, budget: int, workspace: torch.Tensor, *,
                          num_sink: int = 0, window: int = 0) -> None:
    """Alg. 1 (normalisation, selection, gather) on the rows held in ``src``; survivors go to ``dst``."""
    desc = Desc(src.batch, src.kv_heads, src.kv_heads, src.capacity, src.d, 1)
    desc.use_projection = 1
    code = load().curdkv_cache_compress(ctypes.byref(src.c), ctypes.byref(dst.c), ctypes.byref(desc),
                                        int(budget), int(num_sink), int(window), _ptr(workspace),
                                        workspace.numel(), _stream())
    _check(code, "curdkv_cache_compress")


def curdkv_cache_compress_inplace(cache: DeviceCache, budget: int, workspace: torch.Tensor, *,
                                  num_sink: int = 0, window: int = 0) -> None:
    """Alg. 1 (normalisation, selection, gather) on the rows held in ``cache``, in place (the row order is given up)."""
    desc = Desc(cache.batch, cache.kv_heads, cache.kv_heads, cache.capacity, cache.d, 1)
    desc.use_projection = 1
    code = load().curdkv_cache_compress_inplace(ctypes.byref(cache.c), ctypes.byref(desc), int(budget),
                                                int(num_sink), int(window), _ptr(workspace),
                                                workspace.numel(), _stream())
    _check(code, "curdkv_cache_compress_inplace")


def curdkv_cache_step(cache: DeviceCache, K_new, V_new, G, budget: int, workspace: torch.Tensor, *,
                      num_sink: int = 0, window: int = 0, t_new: Optional[torch.Tensor] = None) -> None:
    """One generation step: append K_new, V_new ``[B, Hkv, t, d]`` and compress in place to ``budget``."""
    desc = make_desc(K_new, V_new, G.shape[-1], seqlens=t_new)
    code = load().curdkv_cache_step(ctypes.byref(cache.c), _ptr(K_new), _ptr(V_new), _ptr(G), int(G.dim() == 3),
                                    ctypes.byref(desc), int(budget), int(num_sink), int(window),
                                    _ptr(workspace), workspace.numel(), _stream())
    _check(code, "curdkv_cache_step")


def curdkv_attention_out(Q, K, V, desc: Desc, *, scale: float = 1.0, head_rows=None, head_offsets=None,
                         extra_zero_keys=None, O=None, workspace: Optional[torch.Tensor] = None,
                         weight_split: bool = True):
    """O = softmax(scale Q K^T) V per (b, h).  Q bf16 ``[B, Hkv, m, 128]``; K, V as described by
    ``desc``, or packed ``[rows, 128]`` arrays when ``head_offsets`` is given."""
    if Q.dtype != torch.bfloat16 or Q.dim() != 4 or Q.stride(3) != 1:
        raise ValueError("Q must be bf16 [B, Hkv, m, d] with a contiguous last axis")
    B, H, m, d = Q.shape
    if O is None:
        O = torch.empty((B, H, m, d), dtype=torch.float32, device=Q.device)
    if workspace is None:
        nbytes = int(load().curdkv_attention_workspace_bytes(ctypes.byref(desc)))
        workspace = torch.empty((max(nbytes, 256),), dtype=torch.uint8, device=Q.device)
    packed_rows = K.shape[0] if head_offsets is not None else 0
    code = load().curdkv_attention_out(_ptr(Q), m, Q.stride(0), Q.stride(1), Q.stride(2), _ptr(K), _ptr(V),
                                       ctypes.byref(desc), _ptr(head_rows), _ptr(head_offsets),
                                       packed_rows, _ptr(extra_zero_keys), float(scale), int(weight_split),
                                       _ptr(O), _ptr(workspace), workspace.numel(), _stream())
    _check(code, "curdkv_attention_out")
    return O, workspace


def curdkv_eviction_loss(O_full, O_comp):
    """(||O - O'||_F, ||O||_F) per (b, h) for fp32 ``[B, Hkv, m, d]`` outputs."""
    B, H = O_full.shape[:2]
    loss = torch.empty((B, H), dtype=torch.float32, device=O_full.device)
    ref = torch.empty_like(loss)
    code = load().curdkv_eviction_loss(_ptr(O_full), _ptr(O_comp), B * H, O_full[0, 0].numel(), _ptr(loss),
                                       _ptr(ref), _stream())
    _check(code, "curdkv_eviction_loss")
    return loss, ref


def curdkv_profile_next_score(start: torch.cuda.Event, stop: torch.cuda.Event) -> None:
    """Have the next curdkv_score call of this thread record ``start`` / ``stop`` (timing events
    that have been recorded at least once, so that their handles exist) around its sketch kernel."""
    _check(load().curdkv_profile_next_score(ctypes.c_void_p(start.cuda_event),
                                            ctypes.c_void_p(stop.cuda_event)),
           "curdkv_profile_next_score")


def curdkv_selftest_bounded_wait(limit_ns: int, workspace: torch.Tensor) -> None:
    """Runs the kernels' bounded wait on a barrier nobody completes; leaves DEV_TIMEOUT in the status word."""
    _check(load().curdkv_selftest_bounded_wait(int(limit_ns), _ptr(workspace), _stream()),
           "curdkv_selftest_bounded_wait")


def curdkv_selftest_gather_wait(limit_ns: int, workspace: torch.Tensor) -> None:
    """Runs the gather's bounded wait for a head that is never announced; leaves DEV_TIMEOUT in the status word."""
    _check(load().curdkv_selftest_gather_wait(int(limit_ns), _ptr(workspace), _stream()),
           "curdkv_selftest_gather_wait")


def curdkv_gqa_map(desc: Desc, device="cuda") -> torch.Tensor:
    out = torch.empty((desc.q_heads,), dtype=torch.int32, device=device)
    _check(load().curdkv_gqa_map(ctypes.byref(desc), _ptr(out), _stream()), "curdkv_gqa_map")
    return out


def curdkv_gqa_expand(desc: Desc, idx: torch.Tensor, head_counts: torch.Tensor):
    """Per-query-head copies of a fixed-layout selection: (idx_q [B, Hq, budget], counts_q [B, Hq])."""
    budget = idx.shape[-1]
    idx_q = torch.empty((desc.batch, desc.q_heads, budget), dtype=torch.int32, device=idx.device)
    counts_q = torch.empty((desc.batch, desc.q_heads), dtype=torch.int32, device=idx.device)
    _check(load().curdkv_gqa_expand(ctypes.byref(desc), _ptr(idx), _ptr(head_counts), budget, _ptr(idx_q),
                                    _ptr(counts_q), _stream()), "curdkv_gqa_expand")
    return idx_q, counts_q


def curdkv_device_status(workspace: torch.Tensor, with_code: bool = False):
    """Synchronises the current stream and returns the device status flags (with_code: the pair
    (return code, flags); the code is 5, CURDKV_ERR_TIMEOUT, when the timeout bit is set)."""
    flags = ctypes.c_uint32(0)
    code = load().curdkv_device_status(_ptr(workspace), ctypes.byref(flags), _stream())
    if code not in (STATUS_OK, 5):
        raise CurdkvError(code, "curdkv_device_status")
    return (int(code), int(flags.value)) if with_code else int(flags.value)
