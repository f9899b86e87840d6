"""ctypes binding of the ckv C ABI (include/ckv.h): argument marshalling only.

Every function takes torch tensors that live on the GPU, passes their pointers to the
library and returns; all arithmetic runs in the CUDA kernels.  There is no CPU fallback:
if libckv.so is missing or cannot be loaded the import of this module fails.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

from . import build as _build

F32, BF16 = 0, 1
SELECT_GLOBAL, SELECT_CHUNK = 0, 1
OK = 0

EXPORTS = ["ckv_compress_plan", "ckv_workspace_bytes", "ckv_compress_prefill", "ckv_compress_append", "ckv_compress_append_batch",
           "ckv_decode_workspace_bytes", "ckv_decode_attn", "ckv_status_string", "ckv_workspace_status",
           "ckv_decode_attn_static", "ckv_compress_append_recluster", "ckv_decode_attn_paged", "ckv_pages_gather",
           "ckv_pages_scatter", "ckv_pages_plan", "ckv_paged_workspace_bytes", "ckv_compress_paged",
           "ckv_decode_append_attn_paged"]


class CkvPagePool(C.Structure):
    _fields_ = [("k_pages", C.c_void_p), ("v_pages", C.c_void_p), ("deg_pages", C.c_void_p), ("logdeg_pages", C.c_void_p)]


class CkvCache(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("deg", C.c_void_p), ("logdeg", C.c_void_p),
                ("L", C.c_int32), ("H", C.c_int32), ("D", C.c_int32), ("dtype", C.c_int32),
                ("cap", C.c_int64), ("len", C.c_int64), ("pending", C.c_int64)]


class CkvParams(C.Structure):
    _fields_ = [("chunk", C.c_int32), ("n_sink", C.c_int32), ("n_recent", C.c_int32), ("n_rounds_max", C.c_int32),
                ("r_init", C.c_float), ("r_decay", C.c_float), ("r_min", C.c_float), ("select", C.c_int32),
                ("budget", C.c_int64)]


class CkvLayerView(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("logdeg", C.c_void_p), ("len", C.c_int64), ("cap", C.c_int64)]


def _load():
    path = _build.LIB
    if not os.path.exists(path):
        path = _build.build()
    lib = C.CDLL(path)
    lib.ckv_status_string.restype = C.c_char_p
    lib.ckv_status_string.argtypes = [C.c_int]
    lib.ckv_compress_plan.restype = C.c_int
    lib.ckv_compress_plan.argtypes = [C.c_int64, C.POINTER(CkvParams), C.POINTER(C.c_int64), C.POINTER(C.c_int64),
                                      C.POINTER(C.c_int64)]
    lib.ckv_workspace_bytes.restype = C.c_size_t
    lib.ckv_workspace_bytes.argtypes = [C.POINTER(CkvCache), C.POINTER(CkvParams)]
    lib.ckv_compress_prefill.restype = C.c_int
    lib.ckv_compress_prefill.argtypes = [C.POINTER(CkvCache), C.POINTER(CkvCache), C.POINTER(CkvParams), C.c_void_p,
                                         C.c_void_p, C.c_size_t, C.c_void_p, C.POINTER(C.c_int64)]
    lib.ckv_compress_append.restype = C.c_int
    lib.ckv_compress_append.argtypes = [C.POINTER(CkvCache), C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(CkvParams),
                                        C.c_void_p, C.c_size_t, C.c_void_p]
    lib.ckv_compress_append_batch.restype = C.c_int
    lib.ckv_compress_append_batch.argtypes = [C.POINTER(CkvCache), C.c_int32, C.c_void_p, C.c_void_p, C.POINTER(CkvParams),
                                              C.c_void_p, C.c_size_t, C.c_void_p]
    lib.ckv_compress_append_recluster.restype = C.c_int
    lib.ckv_compress_append_recluster.argtypes = [C.POINTER(CkvCache), C.POINTER(CkvCache), C.c_void_p, C.c_void_p, C.c_int32,
                                                  C.POINTER(CkvParams), C.c_int32, C.c_void_p, C.c_size_t, C.c_void_p,
                                                  C.POINTER(C.c_int64)]
    lib.ckv_decode_attn_paged.restype = C.c_int
    lib.ckv_decode_attn_paged.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                          C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_float, C.c_int64, C.c_void_p, C.c_size_t,
                                          C.c_void_p]
    lib.ckv_pages_gather.restype = C.c_int
    lib.ckv_pages_gather.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                     C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
    lib.ckv_pages_scatter.restype = C.c_int
    lib.ckv_pages_scatter.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_int32,
                                      C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.ckv_decode_append_attn_paged.restype = C.c_int
    lib.ckv_decode_append_attn_paged.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                                 C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_float,
                                                 C.c_int64, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.ckv_pages_plan.restype = C.c_int
    lib.ckv_pages_plan.argtypes = [C.c_int64, C.POINTER(CkvParams), C.c_int32, C.POINTER(C.c_int64), C.POINTER(C.c_int64),
                                   C.POINTER(C.c_int64), C.POINTER(C.c_int32), C.POINTER(C.c_int64)]
    lib.ckv_paged_workspace_bytes.restype = C.c_size_t
    lib.ckv_paged_workspace_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int64, C.POINTER(CkvParams)]
    lib.ckv_compress_paged.restype = C.c_int
    lib.ckv_compress_paged.argtypes = [C.POINTER(CkvPagePool), C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                                       C.c_int64, C.c_int32, C.c_void_p, C.c_int64, C.POINTER(CkvParams), C.c_void_p, C.c_size_t,
                                       C.c_void_p, C.POINTER(C.c_int64), C.POINTER(C.c_int32)]
    lib.ckv_workspace_status.restype = C.c_int
    lib.ckv_workspace_status.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_int32)]
    lib.ckv_decode_workspace_bytes.restype = C.c_size_t
    lib.ckv_decode_workspace_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int64]
    lib.ckv_decode_attn.restype = C.c_int
    lib.ckv_decode_attn.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                                    C.c_void_p, C.c_float, C.c_int64, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.ckv_decode_attn_static.restype = C.c_int
    lib.ckv_decode_attn_static.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                                           C.c_void_p, C.c_float, C.c_int64, C.c_void_p]
    return lib


lib = _load()


class CkvError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        super().__init__(f"ckv status {status}: {lib.ckv_status_string(status).decode()}")


def _check(status: int):
    if status != OK:
        raise CkvError(status)


def dtype_code(t: torch.dtype) -> int:
    return {torch.float32: F32, torch.bfloat16: BF16}[t]


@dataclass
class Params:
    """Mirror of ckv_params.  Ratios are stored as float32, like the C struct."""
    chunk: int = 256
    n_sink: int = 16
    n_recent: int = 64
    n_rounds_max: int = 8
    r_init: float = 0.8
    r_decay: float = 0.2
    r_min: float = 0.2
    select: int = SELECT_GLOBAL
    budget: int = 0

    def c(self) -> CkvParams:
        return CkvParams(self.chunk, self.n_sink, self.n_recent, self.n_rounds_max, self.r_init, self.r_decay,
                         self.r_min, self.select, self.budget)

    def as_float32(self):
        """(r_init, r_decay, r_min) as the float32 values the library sees."""
        p = self.c()
        return float(p.r_init), float(p.r_decay), float(p.r_min)


def compress_plan(length: int, params: Params):
    """ckv_compress_plan: (final length, rounds, destination capacity needed).  Host only."""
    out_len, rounds, cap = C.c_int64(), C.c_int64(), C.c_int64()
    _check(lib.ckv_compress_plan(length, C.byref(params.c()), C.byref(out_len), C.byref(rounds), C.byref(cap)))
    return out_len.value, rounds.value, cap.value


class Cache:
    """One sequence's cache on the GPU: k, v [L, H, cap, D]; deg int32 and logdeg fp32 [L, H, cap]."""

    def __init__(self, k: torch.Tensor, v: torch.Tensor, deg: torch.Tensor | None, logdeg: torch.Tensor | None,
                 length: int, pending: int = 0):
        assert k.is_contiguous() and v.is_contiguous() and k.shape == v.shape and k.dim() == 4
        self.k, self.v, self.deg, self.logdeg = k, v, deg, logdeg
        self.len, self.pending = length, pending

    @classmethod
    def empty(cls, L, H, cap, D, dtype, device="cuda", with_logdeg=True):
        k = torch.empty((L, H, cap, D), dtype=dtype, device=device)
        v = torch.empty_like(k)
        deg = torch.zeros((L, H, cap), dtype=torch.int32, device=device)
        logdeg = torch.zeros((L, H, cap), dtype=torch.float32, device=device) if with_logdeg else None
        return cls(k, v, deg, logdeg, 0)

    @property
    def cap(self):
        return self.k.shape[2]

    def c(self) -> CkvCache:
        L, H, cap, D = self.k.shape
        return CkvCache(self.k.data_ptr(), self.v.data_ptr(),
                        self.deg.data_ptr() if self.deg is not None else None,
                        self.logdeg.data_ptr() if self.logdeg is not None else None,
                        L, H, D, dtype_code(self.k.dtype), cap, self.len, self.pending)


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream_ptr():
    """The current CUDA stream as a pointer (the raw-handle query is several times cheaper than building a Stream object,
    which matters for calls that take ten microseconds on the GPU)."""
    if _raw_stream is not None:
        return C.c_void_p(_raw_stream(torch.cuda.current_device()))
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def workspace_bytes(cache: Cache, params: Params) -> int:
    return lib.ckv_workspace_bytes(C.byref(cache.c()), C.byref(params.c()))


def compress_prefill(src: Cache, dst: Cache, params: Params, workspace: torch.Tensor, assign: torch.Tensor | None = None):
    """ckv_compress_prefill on the current stream.  Returns the number of rounds; dst.len is updated."""
    cs, cd, rounds = src.c(), dst.c(), C.c_int64()
    _check(lib.ckv_compress_prefill(C.byref(cs), C.byref(cd), C.byref(params.c()),
                                    assign.data_ptr() if assign is not None else None,
                                    workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream_ptr(),
                                    C.byref(rounds)))
    dst.len, dst.pending = cd.len, cd.pending
    return rounds.value


def compress_append(cache: Cache, k_new: torch.Tensor, v_new: torch.Tensor, params: Params, workspace: torch.Tensor):
    """ckv_compress_append on the current stream; cache.len / cache.pending are updated."""
    assert k_new.is_contiguous() and v_new.is_contiguous() and k_new.shape == v_new.shape
    cc = cache.c()
    _check(lib.ckv_compress_append(C.byref(cc), k_new.data_ptr(), v_new.data_ptr(), k_new.shape[2], C.byref(params.c()),
                                   workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream_ptr()))
    cache.len, cache.pending = cc.len, cc.pending


def compress_append_batch(caches, k_new: torch.Tensor, v_new: torch.Tensor, params: Params, workspace: torch.Tensor):
    """ckv_compress_append_batch on the current stream: one new token for each cache of the list (k_new, v_new:
    [L, H, len(caches), D]); every cache's len / pending are updated."""
    assert k_new.is_contiguous() and v_new.is_contiguous() and k_new.shape == v_new.shape and k_new.shape[2] == len(caches)
    arr = (CkvCache * len(caches))(*[c.c() for c in caches])
    _check(lib.ckv_compress_append_batch(arr, len(caches), k_new.data_ptr(), v_new.data_ptr(), C.byref(params.c()),
                                         workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream_ptr()))
    for c, cc in zip(caches, arr):
        c.len, c.pending = cc.len, cc.pending


def compress_append_recluster(cache: Cache, spare: Cache, k_new: torch.Tensor, v_new: torch.Tensor, params: Params,
                              interval: int, workspace: torch.Tensor) -> int:
    """ckv_compress_append_recluster on the current stream: append, and one clustering round over the whole cache
    whenever it reaches budget + interval tokens.  The two Cache objects trade tensors like the C structs trade
    buffers, so `cache` always holds the live cache.  Returns the number of re-clusterings."""
    assert k_new.is_contiguous() and v_new.is_contiguous() and k_new.shape == v_new.shape
    cc, cs, calls = cache.c(), spare.c(), C.c_int64()
    live_before = cc.k
    _check(lib.ckv_compress_append_recluster(C.byref(cc), C.byref(cs), k_new.data_ptr(), v_new.data_ptr(), k_new.shape[2],
                                             C.byref(params.c()), interval, workspace.data_ptr(),
                                             workspace.numel() * workspace.element_size(), _stream_ptr(), C.byref(calls)))
    if cc.k != live_before:   # an odd number of rounds ran: the tensors trade places
        cache.k, spare.k = spare.k, cache.k
        cache.v, spare.v = spare.v, cache.v
        cache.deg, spare.deg = spare.deg, cache.deg
        cache.logdeg, spare.logdeg = spare.logdeg, cache.logdeg
    cache.len, cache.pending = cc.len, cc.pending
    return calls.value


def workspace_status(workspace: torch.Tensor) -> int:
    """ckv_workspace_status: synchronises the current stream and returns the device status word (0 = fine)."""
    st = C.c_int32(-1)
    _check(lib.ckv_workspace_status(workspace.data_ptr(), _stream_ptr(), C.byref(st)))
    return st.value


def layer_views(caches, layer: int, device="cuda") -> torch.Tensor:
    """Device array of ckv_layer_view for one layer of a batch of caches (as an int64 tensor of 5 words each)."""
    rows = []
    for c in caches:
        L, H, cap, D = c.k.shape
        es = c.k.element_size()
        off = layer * H * cap
        rows.append([c.k.data_ptr() + off * D * es, c.v.data_ptr() + off * D * es,
                     (c.logdeg.data_ptr() + off * 4) if c.logdeg is not None else 0, c.len, cap])
    return torch.tensor(rows, dtype=torch.int64).to(device)


def pages_plan(length: int, params: Params, page_tokens: int):
    """ckv_pages_plan: (final length, rounds, scratch pages needed, result in scratch?, pages kept).  Host only."""
    out_len, rounds, scratch, kept, in_scratch = C.c_int64(), C.c_int64(), C.c_int64(), C.c_int64(), C.c_int32()
    _check(lib.ckv_pages_plan(length, C.byref(params.c()), page_tokens, C.byref(out_len), C.byref(rounds), C.byref(scratch),
                              C.byref(in_scratch), C.byref(kept)))
    return out_len.value, rounds.value, scratch.value, bool(in_scratch.value), kept.value


def paged_workspace_bytes(L: int, H: int, D: int, dtype: torch.dtype, length: int, params: Params) -> int:
    return lib.ckv_paged_workspace_bytes(L, H, D, dtype_code(dtype), length, C.byref(params.c()))


def compress_paged(pools, block_table: torch.Tensor, length: int, has_deg: bool, scratch_table: torch.Tensor, params: Params,
                   workspace: torch.Tensor):
    """ckv_compress_paged on the current stream.  pools: one (k_pages, v_pages, deg_pages, logdeg_pages or None) per layer,
    k_pages [n_pages, H, page_tokens, D].  Returns (final length, result in the scratch table's pages?)."""
    kp = pools[0][0]
    n_pages, H, P, D = kp.shape
    arr = (CkvPagePool * len(pools))(*[CkvPagePool(k.data_ptr(), v.data_ptr(), d.data_ptr(), lg.data_ptr() if lg is not None else None)
                                       for k, v, d, lg in pools])
    out_len, in_scratch = C.c_int64(), C.c_int32()
    _check(lib.ckv_compress_paged(arr, len(pools), H, D, dtype_code(kp.dtype), P, block_table.data_ptr(), length, int(has_deg),
                                  scratch_table.data_ptr() if scratch_table is not None else None,
                                  scratch_table.numel() if scratch_table is not None else 0, C.byref(params.c()),
                                  workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream_ptr(),
                                  C.byref(out_len), C.byref(in_scratch)))
    return out_len.value, bool(in_scratch.value)


def layer_views_all(caches, device="cuda") -> torch.Tensor:
    """[L, Bz, 5] int64: the ckv_layer_view arrays of every layer of a batch of caches, built and copied to the device
    in one go (views[l] is the argument of ckv_decode_attn for layer l)."""
    L = caches[0].k.shape[0]
    base = []
    for c in caches:
        _, H, cap, D = c.k.shape
        base.append([c.k.data_ptr(), c.v.data_ptr(), c.logdeg.data_ptr() if c.logdeg is not None else 0, c.len, cap,
                     H * cap * D * c.k.element_size(), H * cap * 4])
    t = torch.tensor(base, dtype=torch.int64)                       # [Bz, 7]
    lay = torch.arange(L, dtype=torch.int64).view(L, 1)
    out = torch.empty((L, len(caches), 5), dtype=torch.int64)
    out[:, :, 0] = t[:, 0] + lay * t[:, 5]
    out[:, :, 1] = t[:, 1] + lay * t[:, 5]
    out[:, :, 2] = torch.where(t[:, 2] != 0, t[:, 2] + lay * t[:, 6], torch.zeros_like(t[:, 2]))
    out[:, :, 3] = t[:, 3]
    out[:, :, 4] = t[:, 4]
    return out.to(device)


def decode_workspace_bytes(Bz, H, G, D, max_len) -> int:
    return lib.ckv_decode_workspace_bytes(Bz, H, G, D, max_len)


def decode_attn(views: torch.Tensor, H: int, G: int, q: torch.Tensor, out: torch.Tensor, scale: float, max_len: int,
                workspace: torch.Tensor):
    """ckv_decode_attn on the current stream.  views: layer_views(...); q, out: [Bz, H*G, D]."""
    Bz, HG, D = q.shape
    assert HG == H * G and q.is_contiguous() and out.is_contiguous()
    _check(lib.ckv_decode_attn(views.data_ptr(), Bz, H, G, D, dtype_code(q.dtype), q.data_ptr(), out.data_ptr(), scale,
                               max_len, workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream_ptr()))


def decode_attn_static(views: torch.Tensor, H: int, G: int, q: torch.Tensor, out: torch.Tensor, scale: float, max_len: int):
    """ckv_decode_attn_static on the current stream: decode attention without a caller workspace, for callers
    that cannot allocate device memory; the split partials use a fixed 4 MiB array inside the library."""
    Bz, HG, D = q.shape
    assert HG == H * G and q.is_contiguous() and out.is_contiguous()
    _check(lib.ckv_decode_attn_static(views.data_ptr(), Bz, H, G, D, dtype_code(q.dtype), q.data_ptr(), out.data_ptr(),
                                      scale, max_len, _stream_ptr()))


# ---- paged cache: one layer's pool k_pages, v_pages [n_pages, H, P, D], deg_pages int32 / logdeg_pages fp32 [n_pages, H, P]

def _ptr(t):
    return t.data_ptr() if t is not None else None


def paged_views(block_tables, lens, device="cuda") -> torch.Tensor:
    """Device array of ckv_paged_view (two int64 words each) from per-sequence block-table tensors on the GPU."""
    return torch.tensor([[t.data_ptr(), n] for t, n in zip(block_tables, lens)], dtype=torch.int64).to(device)


def decode_attn_paged(views: torch.Tensor, k_pages, v_pages, logdeg_pages, H: int, G: int, q, out, scale: float, max_len: int,
                      workspace: torch.Tensor):
    """ckv_decode_attn_paged on the current stream."""
    Bz, HG, D = q.shape
    assert HG == H * G and q.is_contiguous() and out.is_contiguous() and k_pages.is_contiguous() and v_pages.is_contiguous()
    _check(lib.ckv_decode_attn_paged(views.data_ptr(), k_pages.data_ptr(), v_pages.data_ptr(), _ptr(logdeg_pages), k_pages.shape[2],
                                     Bz, H, G, D, dtype_code(q.dtype), q.data_ptr(), out.data_ptr(), scale, max_len,
                                     workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream_ptr()))


def decode_append_attn_paged(views: torch.Tensor, k_pages, v_pages, deg_pages, logdeg_pages, H: int, G: int, k_new, v_new, q, out,
                             scale: float, max_len: int, workspace: torch.Tensor):
    """ckv_decode_append_attn_paged on the current stream: k_new, v_new [Bz, H, D] are written to slot views[b].len of
    every sequence's pages and attended to in the same launch; max_len bounds every len + 1."""
    Bz, HG, D = q.shape
    assert HG == H * G and q.is_contiguous() and out.is_contiguous() and k_new.is_contiguous() and v_new.is_contiguous()
    assert k_new.shape == (Bz, H, D) and v_new.shape == (Bz, H, D)
    _check(lib.ckv_decode_append_attn_paged(views.data_ptr(), k_pages.data_ptr(), v_pages.data_ptr(), deg_pages.data_ptr(),
                                            _ptr(logdeg_pages), k_pages.shape[2], Bz, H, G, D, dtype_code(q.dtype), k_new.data_ptr(),
                                            v_new.data_ptr(), q.data_ptr(), out.data_ptr(), scale, max_len, workspace.data_ptr(),
                                            workspace.numel() * workspace.element_size(), _stream_ptr()))


def pages_gather(block_table, length, k_pages, v_pages, deg_pages, k, v, deg, logdeg=None):
    """ckv_pages_gather: pages -> contiguous slab k, v [H, cap, D], deg [H, cap] of one layer."""
    _, H, P, D = k_pages.shape
    _check(lib.ckv_pages_gather(block_table.data_ptr(), length, k_pages.data_ptr(), v_pages.data_ptr(), _ptr(deg_pages), P, H, D,
                                dtype_code(k_pages.dtype), k.data_ptr(), v.data_ptr(), _ptr(deg), _ptr(logdeg), k.shape[1], _stream_ptr()))


def pages_scatter(block_table, length, k, v, deg, k_pages, v_pages, deg_pages, logdeg_pages):
    """ckv_pages_scatter: contiguous slab -> pages (degrees and log-degrees included)."""
    _, H, P, D = k_pages.shape
    _check(lib.ckv_pages_scatter(block_table.data_ptr(), length, k.data_ptr(), v.data_ptr(), _ptr(deg), k.shape[1], P, H, D,
                                 dtype_code(k_pages.dtype), k_pages.data_ptr(), v_pages.data_ptr(), _ptr(deg_pages),
                                 _ptr(logdeg_pages), _stream_ptr()))

