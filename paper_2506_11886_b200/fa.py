"""Thin ctypes binding of the C ABI in ``include/fa.h`` (same names, argument
marshalling only: every step of the path runs in the CUDA kernels of
``csrc/libfa.so``).  PyTorch is used for device memory and streams.

There is no CPU fallback: if the library has not been built, or a call returns
a non-zero status, this module raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "csrc", "libfa.so")

FA_OK, FA_ERR_INVALID_ARG, FA_ERR_UNSUPPORTED, FA_ERR_CAPACITY = 0, 1, 2, 3
FA_ERR_WORKSPACE, FA_ERR_CUDA, FA_ERR_TIMEOUT, FA_ERR_INDEX = 4, 5, 6, 7
FA_F32, FA_BF16 = 0, 1
FA_NORM_ORTHO, FA_NORM_PAPER = 0, 1
FA_DECODE_AUTO, FA_DECODE_DIRECT, FA_DECODE_FFT, FA_DECODE_FFT_SPLIT = 0, 1, 2, 3
FA_COMPRESS_ORDERED, FA_COMPRESS_FFT = 1, 2


class fa_layout(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "batch", "n_q_heads", "n_kv_heads", "head_dim", "n_full_k", "n_full_v", "n_coef", "period",
        "l_init", "l_local", "max_mid", "mid_classes", "kv_dtype", "norm", "decode_algo")] + [("softmax_scale", C.c_float)]


_CACHE_FIELDS = ("idx_full_k", "idx_comp_k", "idx_full_v", "idx_comp_v", "k_init", "v_init", "k_local", "v_local",
                 "k_mid", "v_mid", "coef_k", "coef_v", "state", "status")


class fa_cache(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _CACHE_FIELDS]


class fa_cache_sizes(C.Structure):
    _fields_ = [(n, C.c_size_t) for n in _CACHE_FIELDS]


class FaError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: fa_status {status} ({status_string(status)})")


_lib = None


def lib() -> C.CDLL:
    """Loads csrc/libfa.so; raises if it has not been built (no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2506_11886_b200.build` "
                "(there is no CPU or PyTorch fallback for this path)")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
        lp, cp = C.POINTER(fa_layout), C.POINTER(fa_cache)
        L.fa_cache_sizes_of.argtypes = [lp, C.POINTER(fa_cache_sizes)]
        L.fa_workspace_bytes.argtypes = [lp, C.POINTER(sz)]
        L.fa_cache_reset.argtypes = [lp, cp, vp]
        L.fa_workspace_init.argtypes = [vp, sz, vp]
        L.fa_validate.argtypes = [lp, cp, vp]
        L.fa_compress.argtypes = [lp, cp, vp, vp, i64, i64, i64, i32, vp, sz, vp]
        L.fa_compress_ex.argtypes = [lp, cp, vp, vp, i64, i64, i64, i32, C.c_uint32, vp, sz, vp]
        L.fa_compress_ex.restype = C.c_int
        L.fa_compress_layers.argtypes = [i32, lp, cp, C.POINTER(vp), C.POINTER(vp), i64, i64, i64, i32, C.c_uint32, vp, sz, vp]
        L.fa_compress_layers.restype = C.c_int
        L.fa_append.argtypes = [lp, cp, vp, vp, vp]
        L.fa_compress_ragged.argtypes = [lp, cp, vp, vp, i64, i64, i64, C.POINTER(C.c_int32), vp, sz, vp]
        L.fa_decode_attention.argtypes = [lp, cp, vp, vp, vp, sz, vp]
        L.fa_poll_status.argtypes = [cp, vp]
        L.fa_decode_step_host.argtypes = [lp, cp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.fa_decode_step.argtypes = [lp, cp, vp, vp, vp, vp, vp, sz, vp]
        L.fa_decode_step_layers.argtypes = [i32, lp, cp, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), vp, sz, vp]
        L.fa_decode_step_layers.restype = C.c_int
        L.fa_select_workspace_bytes.argtypes = [lp, C.POINTER(sz)]
        L.fa_select_dims.argtypes = [lp, vp, vp, i64, i64, i64, i32, vp, vp, vp, vp, vp, vp, sz, vp]
        L.fa_step_staging_bytes.argtypes = [lp]
        L.fa_step_staging_bytes.restype = sz
        L.fa_launch_count.argtypes = [lp, C.c_int]
        L.fa_status_string.argtypes = [C.c_int]
        L.fa_status_string.restype = C.c_char_p
        for name in ("fa_cache_sizes_of", "fa_workspace_bytes", "fa_cache_reset", "fa_validate", "fa_compress",
                     "fa_append", "fa_decode_attention", "fa_poll_status", "fa_launch_count", "fa_version",
                     "fa_decode_step_host", "fa_decode_step", "fa_select_workspace_bytes", "fa_select_dims", "fa_compress_ragged", "fa_workspace_init"):
            getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().fa_status_string(int(status)).decode()


def _check(status: int, what: str) -> None:
    if status != FA_OK:
        raise FaError(status, what)


def _stream(stream) -> C.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _ptr(t) -> C.c_void_p:
    return C.c_void_p(0 if t is None or t.numel() == 0 else t.data_ptr())


@dataclass
class Layout:
    """Python mirror of ``fa_layout`` (field meanings: include/fa.h)."""
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_full_k: int
    n_full_v: int
    n_coef: int
    period: int
    l_init: int
    l_local: int
    max_mid: int
    mid_classes: int = 1
    kv_dtype: int = FA_BF16
    norm: int = FA_NORM_ORTHO
    decode_algo: int = FA_DECODE_AUTO
    softmax_scale: float = 1.0

    def c(self) -> fa_layout:
        return fa_layout(self.batch, self.n_q_heads, self.n_kv_heads, self.head_dim, self.n_full_k, self.n_full_v,
                         self.n_coef, self.period, self.l_init, self.l_local, self.max_mid, self.mid_classes,
                         self.kv_dtype, self.norm, self.decode_algo, float(self.softmax_scale))

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.kv_dtype == FA_BF16 else torch.float32

    @property
    def slots(self) -> int:
        return (self.max_mid + self.mid_classes - 1) // self.mid_classes


def fa_cache_sizes_of(layout: Layout) -> dict:
    out = fa_cache_sizes()
    _check(lib().fa_cache_sizes_of(C.byref(layout.c()), C.byref(out)), "fa_cache_sizes_of")
    return {n: int(getattr(out, n)) for n in _CACHE_FIELDS}


def fa_workspace_bytes(layout: Layout) -> int:
    out = C.c_size_t(0)
    _check(lib().fa_workspace_bytes(C.byref(layout.c()), C.byref(out)), "fa_workspace_bytes")
    return int(out.value)


class Cache:
    """Caller-owned device buffers of one layer's cache, allocated with torch and
    sized by ``fa_cache_sizes_of``.  Typed views: ``k_mid`` is
    [B][H_kv][P][slots][n_full_k], ``coef_k`` is [B][H_kv][M][d - n_full_k], ..."""

    def __init__(self, layout: Layout, idx_full_k: torch.Tensor, idx_full_v: torch.Tensor, device="cuda"):
        self.layout = layout
        self.device = torch.device(device)
        sizes = fa_cache_sizes_of(layout)
        L, dt = layout, layout.torch_dtype
        B, H, d = L.batch, L.n_kv_heads, L.head_dim

        def comp(idx_full):
            rows = []
            for h in range(H):
                keep = torch.zeros(d, dtype=torch.bool)
                keep[idx_full[h].long()] = True
                rows.append(torch.nonzero(~keep).flatten().to(torch.int32))
            return torch.stack(rows) if rows else torch.zeros((0, 0), dtype=torch.int32)

        idx_full_k = idx_full_k.to(torch.int32).cpu().reshape(H, L.n_full_k)
        idx_full_v = idx_full_v.to(torch.int32).cpu().reshape(H, L.n_full_v)
        dev = self.device
        self.idx_full_k = idx_full_k.contiguous().to(dev)
        self.idx_full_v = idx_full_v.contiguous().to(dev)
        self.idx_comp_k = comp(idx_full_k).contiguous().to(dev)
        self.idx_comp_v = comp(idx_full_v).contiguous().to(dev)
        z = lambda shape, dtype: torch.zeros(shape, dtype=dtype, device=dev)
        self.k_init, self.v_init = z((B, H, L.l_init, d), dt), z((B, H, L.l_init, d), dt)
        self.k_local, self.v_local = z((B, H, L.l_local, d), dt), z((B, H, L.l_local, d), dt)
        self.k_mid = z((B, H, L.mid_classes, L.slots, L.n_full_k), dt)
        self.v_mid = z((B, H, L.mid_classes, L.slots, L.n_full_v), dt)
        self.coef_k = z((B, H, L.n_coef, d - L.n_full_k), torch.float32)
        self.coef_v = z((B, H, L.n_coef, d - L.n_full_v), torch.float32)
        self.state = z((B, 8), torch.int32)
        self.status = z((4,), torch.int32)
        for n in _CACHE_FIELDS:
            t = getattr(self, n)
            assert t.numel() * t.element_size() == sizes[n], (n, t.shape, sizes[n])
        self._c = fa_cache(*[_ptr(getattr(self, n)).value for n in _CACHE_FIELDS])

    def c(self) -> fa_cache:
        return self._c

    def bytes(self) -> int:
        return sum(getattr(self, n).numel() * getattr(self, n).element_size() for n in _CACHE_FIELDS)


def new_workspace(layout: Layout, device="cuda") -> torch.Tensor:
    """A zero-filled workspace (its first 4 KiB are barrier counters that must start at zero)."""
    return torch.zeros(max(4096, fa_workspace_bytes(layout)), dtype=torch.uint8, device=device)


def fa_workspace_init(ws: torch.Tensor, stream=None) -> None:
    """Re-zeroes the barrier counters of a workspace (after FA_ERR_TIMEOUT, or for a buffer not made by new_workspace)."""
    _check(lib().fa_workspace_init(_ptr(ws), ws.numel(), _stream(stream)), "fa_workspace_init")


def fa_cache_reset(layout: Layout, cache: Cache, stream=None) -> None:
    _check(lib().fa_cache_reset(C.byref(layout.c()), C.byref(cache.c()), _stream(stream)), "fa_cache_reset")


def fa_validate(layout: Layout, cache: Cache, stream=None) -> None:
    _check(lib().fa_validate(C.byref(layout.c()), C.byref(cache.c()), _stream(stream)), "fa_validate")


def fa_compress(layout: Layout, cache: Cache, K: torch.Tensor, V: torch.Tensor, ws: torch.Tensor, stream=None, flags: int = 0) -> None:
    """K, V: [B][L][H_kv][d] (any strides with unit stride on d) in the layout's dtype.
    flags: 0, or FA_COMPRESS_ORDERED / FA_COMPRESS_FFT (fa_compress_ex)."""
    assert K.dtype == layout.torch_dtype and V.dtype == K.dtype and K.shape == V.shape and K.stride() == V.stride()
    assert K.is_cuda and V.is_cuda and (K.shape[1] == 0 or K.stride(3) == 1)
    L = K.shape[1]
    sb, st, sh = (K.stride(0), K.stride(1), K.stride(2)) if L > 0 else (0, layout.head_dim * layout.n_kv_heads, layout.head_dim)
    if K.shape[0] == 1:
        sb = 0
    if flags:
        _check(lib().fa_compress_ex(C.byref(layout.c()), C.byref(cache.c()), _ptr(K), _ptr(V), sb, st, sh, L, int(flags),
                                    _ptr(ws), ws.numel(), _stream(stream)), "fa_compress_ex")
        return
    _check(lib().fa_compress(C.byref(layout.c()), C.byref(cache.c()), _ptr(K), _ptr(V), sb, st, sh, L,
                             _ptr(ws), ws.numel(), _stream(stream)), "fa_compress")


def fa_compress_layers(layouts, caches, Ks, Vs, ws: torch.Tensor, stream=None, flags: int = 0) -> None:
    """Compression of the prefill of several layers in one call: Ks[i], Vs[i] are layer i's [B][L][H_kv][d] tensors
    (same shape and strides for all layers), caches[i] its cache (no two layers share one)."""
    n = len(layouts)
    assert n == len(caches) == len(Ks) == len(Vs) and n > 0
    K0 = Ks[0]
    for lay, K, V in zip(layouts, Ks, Vs):
        assert K.dtype == lay.torch_dtype and V.dtype == K.dtype and K.shape == K0.shape and V.shape == K0.shape
        assert K.stride() == K0.stride() and V.stride() == K0.stride() and K.is_cuda and V.is_cuda
        assert K.shape[1] == 0 or K.stride(3) == 1
    L = K0.shape[1]
    lay0 = layouts[0]
    sb, st, sh = (K0.stride(0), K0.stride(1), K0.stride(2)) if L > 0 else (0, lay0.head_dim * lay0.n_kv_heads, lay0.head_dim)
    if K0.shape[0] == 1:
        sb = 0
    c_layouts = (fa_layout * n)(*[l.c() for l in layouts])
    c_caches = (fa_cache * n)(*[c.c() for c in caches])
    arr = lambda ts: (C.c_void_p * n)(*[t.data_ptr() for t in ts])
    _check(lib().fa_compress_layers(n, c_layouts, c_caches, arr(Ks), arr(Vs), sb, st, sh, L, int(flags), _ptr(ws), ws.numel(),
                                    _stream(stream)), "fa_compress_layers")


def fa_compress_ragged(layout: Layout, cache: Cache, K: torch.Tensor, V: torch.Tensor, lengths, ws: torch.Tensor,
                       stream=None) -> None:
    """fa_compress with a prompt length per batch row (lengths: B ints, each <= K.shape[1])."""
    assert K.is_cuda and V.is_cuda and K.dtype == layout.torch_dtype and K.shape == V.shape and K.stride() == V.stride()
    assert K.stride(3) == 1 and len(lengths) == layout.batch and max(lengths) <= K.shape[1]
    arr = (C.c_int32 * layout.batch)(*[int(x) for x in lengths])
    _check(lib().fa_compress_ragged(C.byref(layout.c()), C.byref(cache.c()), _ptr(K), _ptr(V), K.stride(0), K.stride(1),
                                    K.stride(2), arr, _ptr(ws), ws.numel(), _stream(stream)), "fa_compress_ragged")


def fa_append(layout: Layout, cache: Cache, k_new: torch.Tensor, v_new: torch.Tensor, stream=None) -> None:
    """k_new, v_new: contiguous [B][H_kv][d]."""
    assert k_new.is_contiguous() and v_new.is_contiguous() and k_new.dtype == layout.torch_dtype and k_new.is_cuda
    _check(lib().fa_append(C.byref(layout.c()), C.byref(cache.c()), _ptr(k_new), _ptr(v_new), _stream(stream)), "fa_append")


def fa_decode_attention(layout: Layout, cache: Cache, q: torch.Tensor, out: torch.Tensor, ws: torch.Tensor, stream=None) -> None:
    """q, out: contiguous [B][H_q][d]."""
    assert q.is_contiguous() and out.is_contiguous() and q.dtype == layout.torch_dtype and out.dtype == q.dtype
    assert q.is_cuda and out.is_cuda
    _check(lib().fa_decode_attention(C.byref(layout.c()), C.byref(cache.c()), _ptr(q), _ptr(out), _ptr(ws), ws.numel(),
                                     _stream(stream)), "fa_decode_attention")


def fa_step_staging_bytes(layout: Layout) -> int:
    return int(lib().fa_step_staging_bytes(C.byref(layout.c())))


def fa_select_dims(layout: Layout, K: torch.Tensor, V: torch.Tensor, stream=None):
    """Sec. 3.4: index sets (idx_full_k, idx_comp_k, idx_full_v, idx_comp_v) [H_kv][...] int32 on the
    device of K, and the per-row mean squared reconstruction errors [B][H_kv][2][d]."""
    assert K.is_cuda and V.is_cuda and K.dtype == layout.torch_dtype and K.shape == V.shape and K.stride() == V.stride()
    B, L, H, d = K.shape
    assert K.stride(3) == 1
    out = C.c_size_t(0)
    _check(lib().fa_select_workspace_bytes(C.byref(layout.c()), C.byref(out)), "fa_select_workspace_bytes")
    ws = torch.zeros(max(256, out.value), dtype=torch.uint8, device=K.device)
    dev = K.device
    idx = [torch.zeros((H, n), dtype=torch.int32, device=dev) for n in
           (layout.n_full_k, d - layout.n_full_k, layout.n_full_v, d - layout.n_full_v)]
    mse = torch.zeros((B, H, 2, d), dtype=torch.float32, device=dev)
    _check(lib().fa_select_dims(C.byref(layout.c()), _ptr(K), _ptr(V), K.stride(0), K.stride(1), K.stride(2), L,
                                *[_ptr(t) if t.numel() else None for t in idx], _ptr(mse), _ptr(ws), ws.numel(),
                                _stream(stream)), "fa_select_dims")
    return (*idx, mse)


def fa_decode_step(layout: Layout, cache: Cache, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor,
                   out: torch.Tensor, ws: torch.Tensor, stream=None) -> None:
    """fa_append(k_new, v_new) then fa_decode_attention(q) as one step (device tensors)."""
    for t in (q, k_new, v_new, out):
        assert t.is_cuda and t.is_contiguous() and t.dtype == layout.torch_dtype
    _check(lib().fa_decode_step(C.byref(layout.c()), C.byref(cache.c()), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out),
                                _ptr(ws), ws.numel(), _stream(stream)), "fa_decode_step")


class LayerStep:
    """Marshalled arguments of ``fa_decode_step_layers`` for a fixed set of layers and tensors (built
    once, so that the per-token call is one C call)."""

    def __init__(self, layouts, caches, qs, k_news, v_news, outs):
        n = len(layouts)
        assert n == len(caches) == len(qs) == len(k_news) == len(v_news) == len(outs)
        for lay, q, k, v, o in zip(layouts, qs, k_news, v_news, outs):
            for t in (q, k, v, o):
                assert t.is_cuda and t.is_contiguous() and t.dtype == lay.torch_dtype
        self.n = n
        self.layouts = (fa_layout * n)(*[l.c() for l in layouts])
        self.caches = (fa_cache * n)(*[c.c() for c in caches])
        arr = lambda ts: (C.c_void_p * n)(*[t.data_ptr() for t in ts])
        self.q, self.k, self.v, self.o = arr(qs), arr(k_news), arr(v_news), arr(outs)
        self._keep = (list(qs), list(k_news), list(v_news), list(outs), list(caches))


def fa_decode_step_layers(args: LayerStep, ws: torch.Tensor, stream=None) -> None:
    """One decoded token across all layers of ``args`` (fa_decode_step per layer, in order)."""
    _check(lib().fa_decode_step_layers(args.n, args.layouts, args.caches, args.q, args.k, args.v, args.o, _ptr(ws),
                                       ws.numel(), _stream(stream)), "fa_decode_step_layers")


def fa_decode_step_host(layout: Layout, cache: Cache, q_host: torch.Tensor, k_new_host, v_new_host,
                        out_host: torch.Tensor, staging: torch.Tensor, ws: torch.Tensor, stream=None) -> None:
    """Host-buffer decode step: q_host / out_host [B][H_q][d], k_new_host / v_new_host [B][H_kv][d]
    (or None to skip the append) are CPU tensors, pinned for asynchronous copies."""
    for t in (q_host, out_host, k_new_host, v_new_host):
        assert t is None or (not t.is_cuda and t.is_contiguous() and t.dtype == layout.torch_dtype)
    assert staging.is_cuda and staging.numel() * staging.element_size() >= fa_step_staging_bytes(layout)
    _check(lib().fa_decode_step_host(C.byref(layout.c()), C.byref(cache.c()), _ptr(q_host), _ptr(k_new_host),
                                     _ptr(v_new_host), _ptr(out_host), _ptr(staging), _ptr(ws), ws.numel(),
                                     _stream(stream)), "fa_decode_step_host")


def fa_poll_status(cache: Cache, stream=None) -> int:
    return int(lib().fa_poll_status(C.byref(cache.c()), _stream(stream)))


def fa_launch_count(layout: Layout, what: int) -> int:
    return int(lib().fa_launch_count(C.byref(layout.c()), int(what)))


def fa_version() -> int:
    return int(lib().fa_version())


def fa_static_workspace_limit() -> int:
    f = lib().fa_static_workspace_limit
    f.restype, f.argtypes = C.c_size_t, []
    return int(f())


def fa_decode_attention_static(layout: Layout, cache: Cache, q: torch.Tensor, out: torch.Tensor, stream=None) -> None:
    """``fa_decode_attention`` for callers that cannot allocate device memory (an engine
    whose memory is all spoken for, a loop in which cudaMalloc is not allowed): the scratch
    is the library's own fixed 8 MiB array, so no workspace is passed.  Layouts that need
    more scratch raise FA_ERR_WORKSPACE.  Calls on one GPU share that array: do not overlap
    them, and make the first call on a device outside any stream capture."""
    assert q.is_contiguous() and out.is_contiguous() and q.dtype == layout.torch_dtype and out.dtype == q.dtype
    assert q.is_cuda and out.is_cuda
    f = lib().fa_decode_attention_static
    f.restype = C.c_int
    f.argtypes = [C.POINTER(fa_layout), C.POINTER(fa_cache), C.c_void_p, C.c_void_p, C.c_void_p]
    _check(f(C.byref(layout.c()), C.byref(cache.c()), _ptr(q), _ptr(out), _stream(stream)), "fa_decode_attention_static")
