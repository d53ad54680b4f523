"""ctypes binding of the kvc C ABI (include/kvc.h).

Argument marshalling only: every step of the hot path runs in the CUDA library.  PyTorch is used
for device memory and stream handles.  There is no CPU fallback: if the shared library is missing
the import of this module fails, and every call needs a CUDA device.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

from . import build as _build

KVC_OK, KVC_EINVAL, KVC_ESTATE, KVC_ECUDA, KVC_ETIMEOUT = 0, -1, -2, -3, -4
KVC_F32, KVC_BF16 = 0, 1
KVC_SCORE_ATTN, KVC_SCORE_KEYDIFF = 0, 1
KVC_FLAG_CUDA_CORES = 1
KVC_FLAG_ASYNC_COMPRESS = 16

EXPORTS = [
    "kvc_create", "kvc_destroy", "kvc_cache_nbytes", "kvc_workspace_init", "kvc_reset",
    "kvc_prefill_chunk", "kvc_prefill_chunk_layers", "kvc_staging_nbytes", "kvc_prefill_chunk_host", "kvc_host_flush",
    "kvc_prefill_chunk_static", "kvc_status_static", "kvc_prefill_chunk_proxy",
    "kvc_join", "kvc_cache_view", "kvc_workspace_view", "kvc_move_counts", "kvc_status", "kvc_kv_bytes", "kvc_profile_enable",
    "kvc_profile_read", "kvc_launch_count", "kvc_last_error", "kvc_set_wait_limit", "kvc_selftest_wait_timeout",
    "kvc_profile_device", "kvc_profile_device_read",
]


class KvcConfig(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int), ("n_q_heads", ctypes.c_int), ("n_kv_heads", ctypes.c_int),
                ("head_dim", ctypes.c_int), ("dtype", ctypes.c_int), ("budget", ctypes.c_int),
                ("max_chunk", ctypes.c_int), ("obs_window", ctypes.c_int), ("policy", ctypes.c_int),
                ("softmax_scale", ctypes.c_float), ("device", ctypes.c_int), ("flags", ctypes.c_uint)]


class KvcView(ctypes.Structure):
    _fields_ = [("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("pos", ctypes.c_void_p),
                ("len", ctypes.c_int), ("cap", ctypes.c_int), ("n_kv_heads", ctypes.c_int),
                ("head_dim", ctypes.c_int), ("dtype", ctypes.c_int)]


def lib_path() -> str:
    return _build.LIB


def load_library() -> ctypes.CDLL:
    """Loads libkvc.so (building it first if nvcc is available and it is stale)."""
    path = _build.build(force=bool(os.environ.get("KVC_REBUILD")))
    lib = ctypes.CDLL(path)
    vp, i, ll, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_longlong, ctypes.c_size_t
    psz = ctypes.POINTER(ctypes.c_size_t)
    lib.kvc_create.argtypes = [ctypes.POINTER(KvcConfig), ctypes.POINTER(vp)]
    lib.kvc_destroy.argtypes = [vp]
    lib.kvc_cache_nbytes.argtypes = [vp, psz, psz]
    lib.kvc_workspace_init.argtypes = [vp, vp, vp]
    lib.kvc_reset.argtypes = [vp, i, i, vp, sz, vp]
    lib.kvc_prefill_chunk.argtypes = [vp, i, vp, vp, vp, i, ll, vp, vp, vp, vp]
    lib.kvc_prefill_chunk_proxy.argtypes = [vp, i, vp, vp, vp, i, i, ll, vp, vp, vp, vp]
    lib.kvc_prefill_chunk_layers.argtypes = [vp, i, i, vp, ll, vp, vp, ll, i, ll, vp, sz, vp, vp, ll, vp]
    lib.kvc_staging_nbytes.argtypes = [vp, psz]
    lib.kvc_prefill_chunk_host.argtypes = [vp, i, vp, vp, vp, i, ll, vp, vp, vp, vp, vp]
    lib.kvc_host_flush.argtypes = [vp, vp]
    lib.kvc_prefill_chunk_static.argtypes = [vp, i, vp, vp, vp, i, ll, vp, vp, vp]
    lib.kvc_status_static.argtypes = [vp, vp]
    lib.kvc_cache_view.argtypes = [vp, i, vp, ctypes.POINTER(KvcView)]
    lib.kvc_workspace_view.argtypes = [vp, vp, i, ctypes.POINTER(vp), ctypes.POINTER(vp)]
    lib.kvc_move_counts.argtypes = [vp, vp, i, ctypes.POINTER(vp)]
    lib.kvc_status.argtypes = [vp, vp, vp]
    lib.kvc_join.argtypes = [vp, vp]
    lib.kvc_set_wait_limit.argtypes = [vp, ll]
    lib.kvc_selftest_wait_timeout.argtypes = [vp, vp, vp]
    lib.kvc_kv_bytes.argtypes = [vp, ll, psz, psz, psz]
    lib.kvc_profile_enable.argtypes = [vp, i]
    lib.kvc_profile_read.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ll)]
    lib.kvc_profile_device.argtypes = [vp, vp, ll, vp]
    lib.kvc_profile_device_read.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ll), ctypes.POINTER(ctypes.c_double)]
    lib.kvc_launch_count.argtypes = [vp]
    lib.kvc_launch_count.restype = ll
    lib.kvc_last_error.argtypes = [vp]
    lib.kvc_last_error.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name not in ("kvc_launch_count", "kvc_last_error"):
            getattr(lib, name).restype = i
    return lib


_LIB: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    global _LIB
    if _LIB is None:
        _LIB = load_library()
    return _LIB


class KvcError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"kvc error {code}: {msg}")
        self.code = code


def _ptr(t: Optional[torch.Tensor]) -> int:
    return 0 if t is None else t.data_ptr()


class Kvc:
    """One kvc context plus the device buffers it needs (allocated here with torch).

    Mirrors the C ABI one to one: ``prefill_chunk``, ``prefill_chunk_layers``,
    ``prefill_chunk_host``, ``cache_view``, ``reset``, ``status``.
    """

    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, dtype: torch.dtype,
                 budget: int, max_chunk: int, obs_window: int = 0, softmax_scale: float = 0.0,
                 device: int = 0, flags: int = 0, allocate: bool = True, policy: int = KVC_SCORE_ATTN):
        if not torch.cuda.is_available():
            raise RuntimeError("kvc needs a CUDA device: there is no CPU implementation of the hot path")
        self._lib = lib()
        self.dtype = dtype
        self.device = torch.device("cuda", device)
        code = {torch.float32: KVC_F32, torch.bfloat16: KVC_BF16}[dtype]
        self.cfg = KvcConfig(n_layers, n_q_heads, n_kv_heads, head_dim, code, budget, max_chunk, obs_window,
                             policy, softmax_scale, device, flags)
        h = ctypes.c_void_p()
        rc = self._lib.kvc_create(ctypes.byref(self.cfg), ctypes.byref(h))
        if rc != KVC_OK:
            raise KvcError(rc, "kvc_create rejected the configuration")
        self._h = h
        a, b = ctypes.c_size_t(), ctypes.c_size_t()
        self._check(self._lib.kvc_cache_nbytes(self._h, ctypes.byref(a), ctypes.byref(b)))
        self.blob_bytes, self.ws_bytes = a.value, b.value
        s = ctypes.c_size_t()
        self._check(self._lib.kvc_staging_nbytes(self._h, ctypes.byref(s)))
        self.staging_bytes = s.value
        self.cache = self.workspace = self.staging = None
        if allocate:
            with torch.cuda.device(self.device):
                self.cache = torch.empty(n_layers, self.blob_bytes, dtype=torch.uint8, device=self.device)
                self.workspace = torch.empty(self.ws_bytes, dtype=torch.uint8, device=self.device)
                self._check(self._lib.kvc_workspace_init(self._h, self.workspace.data_ptr(), self._stream()))
                self.reset()

    # -- helpers ---------------------------------------------------------------------------------
    def _stream(self) -> int:
        return torch.cuda.current_stream(self.device).cuda_stream

    def _check(self, rc: int):
        if rc != KVC_OK:
            raise KvcError(rc, self._lib.kvc_last_error(self._h).decode())

    def close(self):
        if getattr(self, "_h", None):
            self._lib.kvc_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- C ABI mirrors ---------------------------------------------------------------------------
    def reset(self, layer: int = 0, n_layers: Optional[int] = None):
        n_layers = self.cfg.n_layers - layer if n_layers is None else n_layers
        self._check(self._lib.kvc_reset(self._h, layer, n_layers, self.cache[layer].data_ptr(),
                                        self.cache.stride(0), self._stream()))

    def prefill_chunk(self, layer: int, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, pos0: int,
                      out: Optional[torch.Tensor] = None) -> torch.Tensor:
        n = q.shape[0]
        if out is None:
            out = torch.empty_like(q)
        assert q.is_contiguous() and k.is_contiguous() and v.is_contiguous() and out.is_contiguous()
        assert q.dtype == self.dtype and k.dtype == self.dtype and v.dtype == self.dtype
        self._check(self._lib.kvc_prefill_chunk(self._h, layer, _ptr(q), _ptr(k), _ptr(v), n, pos0,
                                                self.cache[layer].data_ptr(), self.workspace.data_ptr(),
                                                _ptr(out), self._stream()))
        return out

    def prefill_chunk_proxy(self, layer: int, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, n_proxy: int, pos0: int,
                            out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """prefill_chunk whose last ``n_proxy`` rows are proxy query tokens: observers that are never cached."""
        if out is None:
            out = torch.empty_like(q)
        assert q.is_contiguous() and k.is_contiguous() and v.is_contiguous() and out.is_contiguous()
        self._check(self._lib.kvc_prefill_chunk_proxy(self._h, layer, _ptr(q), _ptr(k), _ptr(v), q.shape[0], n_proxy, pos0,
                                                      self.cache[layer].data_ptr(), self.workspace.data_ptr(),
                                                      _ptr(out), self._stream()))
        return out

    def prefill_chunk_layers(self, layer0: int, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, pos0: int,
                             out: torch.Tensor) -> torch.Tensor:
        """q/out: [nl][n][Hq][d] views (token dimension may be a slice of a longer buffer), k/v likewise."""
        nl, n = q.shape[0], q.shape[1]
        for t in (q, k, v, out):
            assert t.stride(-1) == 1 and t.stride(-2) == t.shape[-1] and t.stride(1) == t.shape[-1] * t.shape[-2]
        self._check(self._lib.kvc_prefill_chunk_layers(
            self._h, layer0, nl, _ptr(q), q.stride(0), _ptr(k), _ptr(v), k.stride(0), n, pos0,
            self.cache[layer0].data_ptr(), self.cache.stride(0), self.workspace.data_ptr(), _ptr(out), out.stride(0),
            self._stream()))
        return out

    def prefill_chunk_host(self, layer: int, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, pos0: int,
                           out: torch.Tensor) -> torch.Tensor:
        """q/k/v/out are HOST tensors (pinned for asynchronous copies).  ``out`` is complete once the stream has run
        the next call of this method or ``host_flush``."""
        if self.staging is None:
            self.staging = torch.empty(self.staging_bytes, dtype=torch.uint8, device=self.device)
        assert not q.is_cuda and not out.is_cuda
        self._check(self._lib.kvc_prefill_chunk_host(self._h, layer, _ptr(q), _ptr(k), _ptr(v), q.shape[0], pos0,
                                                     self.cache[layer].data_ptr(), self.workspace.data_ptr(),
                                                     self.staging.data_ptr(), _ptr(out), self._stream()))
        return out

    def host_flush(self) -> None:
        """The current stream waits for the copies of every ``out`` of ``prefill_chunk_host`` so far."""
        self._check(self._lib.kvc_host_flush(self._h, self._stream()))

    def prefill_chunk_static(self, layer: int, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, pos0: int,
                             out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """prefill_chunk with the library's built-in scratch array instead of ``self.workspace``:
        for callers that cannot allocate device memory.  One stream at a time per device."""
        if out is None:
            out = torch.empty_like(q)
        assert q.is_contiguous() and k.is_contiguous() and v.is_contiguous() and out.is_contiguous()
        self._check(self._lib.kvc_prefill_chunk_static(self._h, layer, _ptr(q), _ptr(k), _ptr(v), q.shape[0], pos0,
                                                       self.cache[layer].data_ptr(), _ptr(out), self._stream()))
        return out

    def status_static(self) -> int:
        return self._lib.kvc_status_static(self._h, self._stream())

    def cache_view(self, layer: int) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor, int]:
        """(K [Hkv][cap][d], V [Hkv][cap][d], pos [Hkv][cap], len): tensors alias the cache blob."""
        view = KvcView()
        self._check(self._lib.kvc_cache_view(self._h, layer, self.cache[layer].data_ptr(), ctypes.byref(view)))
        blob = self.cache[layer]
        hkv, cap, d = view.n_kv_heads, view.cap, view.head_dim
        esz = 4 if self.dtype == torch.float32 else 2
        kvb = hkv * cap * d * esz
        base = blob.data_ptr()
        assert view.k == base and view.v == base + kvb and view.pos == base + 2 * kvb
        K = blob[:kvb].view(self.dtype).view(hkv, cap, d)
        V = blob[kvb:2 * kvb].view(self.dtype).view(hkv, cap, d)
        pos = blob[2 * kvb:2 * kvb + hkv * cap * 4].view(torch.int32).view(hkv, cap)
        return K, V, pos, view.len

    def slot_of(self, layer: int) -> int:
        """Workspace slot of a single-layer call: the layer itself while compress runs on the side stream, else 0."""
        side = (self.cfg.flags & KVC_FLAG_ASYNC_COMPRESS) and self.dtype == torch.bfloat16 \
            and not (self.cfg.flags & KVC_FLAG_CUDA_CORES)
        return layer if side else 0

    def workspace_view(self, slot: int = 0) -> Tuple[torch.Tensor, torch.Tensor]:
        """(lse [max(max_chunk, B)][Hq] fp32, score [Hkv][cap] fp32) of the most recent call, aliasing the workspace."""
        a, b = ctypes.c_void_p(), ctypes.c_void_p()
        self._check(self._lib.kvc_workspace_view(self._h, self.workspace.data_ptr(), slot, ctypes.byref(a),
                                                 ctypes.byref(b)))
        base = self.workspace.data_ptr()
        cap = (self.cfg.budget + self.cfg.max_chunk + 127) // 128 * 128
        lo = a.value - base
        rows = max(self.cfg.max_chunk, self.cfg.budget)
        lse = self.workspace[lo:lo + rows * self.cfg.n_q_heads * 4].view(torch.float32)
        so = b.value - base
        score = self.workspace[so:so + self.cfg.n_kv_heads * cap * 4].view(torch.float32)
        return lse.view(rows, self.cfg.n_q_heads), score.view(self.cfg.n_kv_heads, cap)

    def move_counts(self, slot: int = 0) -> torch.Tensor:
        """int32 [Hkv]: entries moved per kv-head by the most recent compaction of this slot."""
        a = ctypes.c_void_p()
        self._check(self._lib.kvc_move_counts(self._h, self.workspace.data_ptr(), slot, ctypes.byref(a)))
        off = a.value - self.workspace.data_ptr()
        return self.workspace[off:off + 4 * self.cfg.n_kv_heads].view(torch.int32)

    def join(self) -> None:
        """Orders the current stream after compress kernels still pending on the context's side stream."""
        self._check(self._lib.kvc_join(self._h, self._stream()))

    def status(self) -> int:
        return self._lib.kvc_status(self._h, self.workspace.data_ptr(), self._stream())

    def set_wait_limit(self, cycles: int) -> None:
        self._check(self._lib.kvc_set_wait_limit(self._h, cycles))

    def selftest_wait_timeout(self) -> None:
        """Enqueues the kernel whose only wait has no producer; ``status()`` then returns KVC_ETIMEOUT."""
        self._check(self._lib.kvc_selftest_wait_timeout(self._h, self.workspace.data_ptr(), self._stream()))

    def workspace_init(self) -> None:
        self._check(self._lib.kvc_workspace_init(self._h, self.workspace.data_ptr(), self._stream()))

    def kv_bytes(self, seq_len: int) -> Tuple[int, int, int]:
        a, b, c = ctypes.c_size_t(), ctypes.c_size_t(), ctypes.c_size_t()
        self._check(self._lib.kvc_kv_bytes(self._h, seq_len, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)))
        return a.value, b.value, c.value

    def profile_enable(self, on: bool):
        self._check(self._lib.kvc_profile_enable(self._h, int(on)))

    def profile_read(self):
        """({step: milliseconds}, {step: launches}) accumulated since profiling was enabled / last read."""
        ms = (ctypes.c_double * 5)()
        cnt = (ctypes.c_longlong * 5)()
        self._check(self._lib.kvc_profile_read(self._h, ms, cnt))
        names = ("append", "attention", "score", "compress", "unused")
        return dict(zip(names, list(ms))), dict(zip(names, list(cnt)))

    def profile_device(self, capacity: int) -> None:
        """Starts device-side time stamps for the next ``capacity`` launches (0 stops them)."""
        if capacity <= 0:
            self._stamps = None
            self._check(self._lib.kvc_profile_device(self._h, None, 0, self._stream()))
            return
        self._stamps = torch.empty(capacity * 2, dtype=torch.int64, device=self.device)
        self._check(self._lib.kvc_profile_device(self._h, self._stamps.data_ptr(), capacity, self._stream()))

    def profile_device_read(self):
        """({step: milliseconds}, {step: launches}, span in ms) of the launches stamped since profile_device()."""
        torch.cuda.synchronize(self.device)
        host = self._stamps.cpu()
        ms = (ctypes.c_double * 5)()
        cnt = (ctypes.c_longlong * 5)()
        span = ctypes.c_double()
        self._check(self._lib.kvc_profile_device_read(self._h, host.data_ptr(), ms, cnt, ctypes.byref(span)))
        names = ("append", "attention", "score", "compress", "unused")
        return dict(zip(names, list(ms))), dict(zip(names, list(cnt))), span.value

    def launch_count(self) -> int:
        return self._lib.kvc_launch_count(self._h)

    def last_error(self) -> str:
        return self._lib.kvc_last_error(self._h).decode()
