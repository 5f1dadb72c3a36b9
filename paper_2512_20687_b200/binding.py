"""Thin ctypes binding of libphoton.so: same names as include/photon.h,
argument marshalling only.  Tensors are torch CUDA tensors (bf16 data held as
torch.bfloat16 or as raw int16/uint16 bits; int32 index arrays); the binding
passes their data pointers and the current (or a given) CUDA stream.  Every
step of the path runs in the library's kernels; there is no fallback: if the
shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_float, c_int32, c_int64, c_size_t, c_void_p

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libphoton.so")

PHOTON_OK, PHOTON_ERR_INVALID_ARG, PHOTON_ERR_UNSUPPORTED, PHOTON_ERR_CUDA, PHOTON_ERR_WORKSPACE = range(5)
PHOTON_DEV_CAPACITY, PHOTON_DEV_BAD_INDEX, PHOTON_DEV_TIMEOUT = 1, 2, 4
PHOTON_W_IN_MAJOR, PHOTON_W_OUT_MAJOR = 0, 1


class PhotonError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {photon_status_str(code)} (status {code})")


class photon_config(Structure):
    _fields_ = [(n, c_int32) for n in ("Hq", "Hkv", "dh", "D", "P", "C", "max_queries", "max_splits")]


class photon_kv(Structure):
    _fields_ = [
        ("k", c_void_p), ("v", c_void_p), ("len", c_void_p),
        ("n_units", c_int32), ("cap", c_int32), ("max_len", c_int32),
        ("k_shared", c_void_p), ("v_shared", c_void_p),
        ("shared_len", c_void_p), ("shared_id", c_void_p),
        ("n_shared", c_int32), ("cap_shared", c_int32), ("max_shared_len", c_int32),
        ("page_table", c_void_p), ("page_rows", c_int32), ("pages_per_unit", c_int32), ("n_pages", c_int32),
    ]


class photon_step_args(Structure):
    _fields_ = [
        ("coarse", POINTER(photon_kv)),
        ("k_new", c_void_p), ("v_new", c_void_p), ("q_coarse", c_void_p),
        ("out_coarse", c_void_p), ("lse_coarse", c_void_p), ("scale_coarse", c_float),
        ("x", c_void_p), ("w", c_void_p), ("bias", c_void_p), ("w_layout", c_int32),
        ("U", c_void_p), ("B", c_int32),
        ("chunks", POINTER(photon_kv)),
        ("q_chunk", c_void_p), ("slot", c_void_p), ("out_chunk", c_void_p),
        ("Nc", c_int32), ("scale_chunk", c_float),
        ("ev_attn_begin", c_void_p), ("ev_attn_end", c_void_p),
    ]


class photon_layer(Structure):
    _fields_ = [(n, c_void_p) for n in ("g1", "wqkv", "wo", "g2", "wgu", "wdown")] + [
        ("w_layout", c_int32), ("F", c_int32), ("eps", c_float), ("theta", c_float)]


class photon_layer_scratch(Structure):
    _fields_ = [(n, c_void_p) for n in ("n", "qkv", "q", "k_new", "v_new", "att", "h", "gu", "act")]


_lib = None


def load() -> ctypes.CDLL:
    """Loads libphoton.so (built in-tree by paper_2512_20687_b200.build).  Raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} not found: build it with `python -m paper_2512_20687_b200.build`; "
            "there is no CPU fallback")
    lib = ctypes.CDLL(LIB_PATH)
    st = c_int32
    lib.photon_create.restype = st
    lib.photon_create.argtypes = [POINTER(c_void_p), POINTER(photon_config)]
    lib.photon_destroy.restype = st
    lib.photon_destroy.argtypes = [c_void_p]
    lib.photon_kv_append.restype = st
    lib.photon_kv_append.argtypes = [c_void_p, POINTER(photon_kv), c_void_p, c_void_p, c_void_p,
                                     c_int32, c_int32, c_void_p]
    for name in ("photon_coarse_attn", "photon_flat_attn"):
        f = getattr(lib, name)
        f.restype = st
        f.argtypes = [c_void_p, POINTER(photon_kv), c_void_p, c_void_p, c_void_p, c_float, c_void_p]
    lib.photon_coarse_attn_noalloc.restype = st
    lib.photon_coarse_attn_noalloc.argtypes = [POINTER(photon_config), POINTER(photon_kv), c_void_p, c_void_p,
                                               c_void_p, c_float, c_void_p, c_void_p]
    lib.photon_converter.restype = st
    lib.photon_converter.argtypes = [c_void_p, c_void_p, c_void_p, c_int32, c_void_p, c_void_p,
                                     c_int32, c_void_p]
    lib.photon_chunk_attn.restype = st
    lib.photon_chunk_attn.argtypes = [c_void_p, POINTER(photon_kv), c_void_p, c_void_p, c_void_p,
                                      c_int32, c_float, c_void_p]
    lib.photon_decoder_prefill.restype = st
    lib.photon_decoder_prefill.argtypes = [c_void_p, POINTER(photon_layer), POINTER(photon_layer_scratch), c_void_p,
                                           POINTER(photon_kv), c_void_p, c_int32, c_void_p, c_float, c_void_p]
    lib.photon_chunk_causal_attn.restype = st
    lib.photon_chunk_causal_attn.argtypes = [c_void_p, POINTER(photon_kv), c_void_p, c_void_p, c_void_p,
                                             c_int32, c_int32, c_int32, c_float, c_void_p]
    lib.photon_rmsnorm.restype = st
    lib.photon_rmsnorm.argtypes = [c_void_p, c_void_p, c_void_p, c_float, c_void_p, c_int32, c_int32, c_void_p]
    lib.photon_linear.restype = st
    lib.photon_linear.argtypes = [c_void_p, c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_void_p, c_int32,
                                  c_int32, c_int32, c_void_p]
    lib.photon_rope_split.restype = st
    lib.photon_rope_split.argtypes = [c_void_p, c_void_p, c_void_p, c_int32, c_float, c_void_p, c_void_p,
                                      c_void_p, c_void_p]
    lib.photon_swiglu.restype = st
    lib.photon_swiglu.argtypes = [c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_void_p]
    for f in (lib.photon_encoder_step, lib.photon_decoder_step):
        f.restype = st
        f.argtypes = [c_void_p, POINTER(photon_layer), POINTER(photon_layer_scratch), c_void_p,
                      POINTER(photon_kv), c_void_p, c_float, c_void_p]
    lib.photon_decode_step.restype = st
    lib.photon_decode_step.argtypes = [c_void_p, POINTER(photon_step_args), c_void_p]
    lib.photon_decode_step_host.restype = st
    lib.photon_decode_step_host.argtypes = [c_void_p, POINTER(photon_step_args), c_void_p, c_void_p, c_size_t, c_size_t,
                                            c_void_p, c_void_p, c_size_t, c_size_t, c_void_p]
    lib.photon_device_status.restype = st
    lib.photon_device_status.argtypes = [c_void_p, POINTER(c_int32), c_int32]
    lib.photon_set_attention_ctas.restype = st
    lib.photon_set_attention_ctas.argtypes = [c_void_p, c_int32]
    lib.photon_read_probe.restype = st
    lib.photon_read_probe.argtypes = [c_void_p, c_void_p, c_size_t, c_int32, c_void_p, c_void_p]
    lib.photon_wait_probe.restype = st
    lib.photon_wait_probe.argtypes = [c_void_p, c_int64, c_void_p]
    lib.photon_set_host_step_tuning.restype = st
    lib.photon_set_host_step_tuning.argtypes = [c_void_p, c_int64, c_int64]
    lib.photon_launch_count.restype = c_int64
    lib.photon_launch_count.argtypes = [c_void_p]
    lib.photon_status_str.restype = c_char_p
    lib.photon_status_str.argtypes = [c_int32]
    _lib = lib
    return lib


def _ptr(t) -> c_void_p:
    """Device pointer of a tensor (None -> NULL, int -> as is)."""
    if t is None:
        return c_void_p(0)
    if isinstance(t, int):
        return c_void_p(t)
    if not t.is_cuda:
        raise ValueError("libphoton takes device tensors")
    if not t.is_contiguous():
        raise ValueError("libphoton takes contiguous tensors")
    return c_void_p(t.data_ptr())


def _stream(stream) -> c_void_p:
    if stream is None:
        import torch
        return c_void_p(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return c_void_p(stream)
    return c_void_p(stream.cuda_stream)


def _check(code: int, where: str) -> None:
    if code != PHOTON_OK:
        raise PhotonError(code, where)


def photon_status_str(code: int) -> str:
    return load().photon_status_str(int(code)).decode()


def make_kv(k, v, length, max_len: int = 0, k_shared=None, v_shared=None, shared_len=None,
            shared_id=None, max_shared_len: int = 0, page_table=None) -> photon_kv:
    """Fills a photon_kv from tensors k, v [n_units, Hkv, cap, dh], length [n_units]
    (and the optional shared-prefix tensors).  With page_table [n_units, pages_per_unit]
    k and v are pools [n_pages, Hkv, page_rows, dh].  The struct keeps the tensors alive."""
    kv = photon_kv()
    kv.k, kv.v, kv.len = _ptr(k), _ptr(v), _ptr(length)
    kv.n_units, kv.cap, kv.max_len = k.shape[0], k.shape[2], max_len
    if page_table is not None:
        kv.page_table = _ptr(page_table)
        kv.n_pages, kv.page_rows = k.shape[0], k.shape[2]
        kv.n_units, kv.pages_per_unit = page_table.shape
        kv.cap = kv.page_rows * kv.pages_per_unit
    kv._pages = page_table
    if k_shared is not None:
        kv.k_shared, kv.v_shared = _ptr(k_shared), _ptr(v_shared)
        kv.shared_len, kv.shared_id = _ptr(shared_len), _ptr(shared_id)
        kv.n_shared, kv.cap_shared, kv.max_shared_len = k_shared.shape[0], k_shared.shape[2], max_shared_len
    kv._keep = (k, v, length, k_shared, v_shared, shared_len, shared_id)
    return kv


def photon_create(Hq, Hkv, dh, D, P, C, max_queries, max_splits=0) -> c_void_p:
    cfg = photon_config(Hq, Hkv, dh, D, P, C, max_queries, max_splits)
    ctx = c_void_p(0)
    _check(load().photon_create(byref(ctx), byref(cfg)), "photon_create")
    return ctx


def photon_destroy(ctx) -> None:
    _check(load().photon_destroy(ctx), "photon_destroy")


def photon_kv_append(ctx, cache: photon_kv, k_new, v_new, unit_ids=None, n=None, n_rows=1,
                     stream=None) -> None:
    if n is None:
        n = k_new.shape[0]
    _check(load().photon_kv_append(ctx, byref(cache), _ptr(k_new), _ptr(v_new), _ptr(unit_ids),
                                   int(n), int(n_rows), _stream(stream)), "photon_kv_append")


def photon_coarse_attn(ctx, cache: photon_kv, q, out, lse=None, scale=1.0, stream=None) -> None:
    _check(load().photon_coarse_attn(ctx, byref(cache), _ptr(q), _ptr(out), _ptr(lse),
                                     c_float(scale), _stream(stream)), "photon_coarse_attn")


def photon_coarse_attn_noalloc(Hq, Hkv, dh, cache: photon_kv, q, out, lse=None, scale=1.0, dev_status=None,
                               stream=None) -> None:
    """photon_coarse_attn without a context and without any device allocation (see photon.h);
    dev_status: optional device int32 tensor that receives PHOTON_DEV_* bits."""
    cfg = photon_config(Hq, Hkv, dh, Hq * dh, 1, 1, 1, 0)
    _check(load().photon_coarse_attn_noalloc(byref(cfg), byref(cache), _ptr(q), _ptr(out), _ptr(lse),
                                             c_float(scale), _ptr(dev_status), _stream(stream)),
           "photon_coarse_attn_noalloc")


def photon_flat_attn(ctx, cache: photon_kv, q, out, lse=None, scale=1.0, stream=None) -> None:
    _check(load().photon_flat_attn(ctx, byref(cache), _ptr(q), _ptr(out), _ptr(lse),
                                   c_float(scale), _stream(stream)), "photon_flat_attn")


def photon_converter(ctx, x, w, w_layout, bias, U, B=None, stream=None) -> None:
    if B is None:
        B = x.shape[0]
    _check(load().photon_converter(ctx, _ptr(x), _ptr(w), int(w_layout), _ptr(bias), _ptr(U), int(B),
                                   _stream(stream)), "photon_converter")


def photon_rmsnorm(ctx, x, gamma, eps, out, rows=None, cols=None, stream=None) -> None:
    rows = x.shape[0] if rows is None else rows
    cols = x.shape[1] if cols is None else cols
    _check(load().photon_rmsnorm(ctx, _ptr(x), _ptr(gamma), c_float(eps), _ptr(out), int(rows), int(cols),
                                 _stream(stream)), "photon_rmsnorm")


def photon_linear(ctx, x, w, w_layout, bias, y, B=None, K=None, N=None, residual=None, stream=None) -> None:
    B = x.shape[0] if B is None else B
    K = x.shape[1] if K is None else K
    N = y.shape[1] if N is None else N
    _check(load().photon_linear(ctx, _ptr(x), _ptr(w), int(w_layout), _ptr(bias), _ptr(residual), _ptr(y), int(B),
                                int(K), int(N), _stream(stream)), "photon_linear")


def photon_rope_split(ctx, qkv, pos, q, k, v, theta=10000.0, n=None, stream=None) -> None:
    n = qkv.shape[0] if n is None else n
    _check(load().photon_rope_split(ctx, _ptr(qkv), _ptr(pos), int(n), c_float(theta), _ptr(q), _ptr(k), _ptr(v),
                                    _stream(stream)), "photon_rope_split")


def photon_swiglu(ctx, gu, out, n=None, F=None, stream=None) -> None:
    n = gu.shape[0] if n is None else n
    F = gu.shape[1] // 2 if F is None else F
    _check(load().photon_swiglu(ctx, _ptr(gu), _ptr(out), int(n), int(F), _stream(stream)), "photon_swiglu")


def make_layer(g1, wqkv, wo, g2, wgu, wdown, w_layout, F, eps=1e-5, theta=10000.0) -> photon_layer:
    L = photon_layer()
    L.g1, L.wqkv, L.wo, L.g2, L.wgu, L.wdown = (_ptr(t) for t in (g1, wqkv, wo, g2, wgu, wdown))
    L.w_layout, L.F, L.eps, L.theta = int(w_layout), int(F), eps, theta
    L._keep = (g1, wqkv, wo, g2, wgu, wdown)
    return L


def make_layer_scratch(B, Hq, Hkv, dh, F, device, dtype) -> photon_layer_scratch:
    """Allocates the intermediates of photon_encoder_step with torch (the caller owns them)."""
    import torch
    D = Hq * dh
    shapes = {"n": (B, D), "qkv": (B, (Hq + 2 * Hkv) * dh), "q": (B, Hq, dh), "k_new": (B, Hkv, dh),
              "v_new": (B, Hkv, dh), "att": (B, Hq, dh), "h": (B, D), "gu": (B, 2 * F), "act": (B, F)}
    sc = photon_layer_scratch()
    sc.tensors = {k: torch.empty(v, dtype=dtype, device=device) for k, v in shapes.items()}
    for k, t in sc.tensors.items():
        setattr(sc, k, _ptr(t))
    return sc


def photon_decoder_prefill(ctx, layer: photon_layer, scratch: photon_layer_scratch, U, chunks: photon_kv, unit_ids, y,
                           n=None, scale=1.0, stream=None) -> None:
    n = U.shape[0] if n is None else n
    _check(load().photon_decoder_prefill(ctx, byref(layer), byref(scratch), _ptr(U), byref(chunks), _ptr(unit_ids),
                                         int(n), _ptr(y), c_float(scale), _stream(stream)), "photon_decoder_prefill")


def photon_decoder_step(ctx, layer: photon_layer, scratch: photon_layer_scratch, x, chunks: photon_kv, y,
                        scale=1.0, stream=None) -> None:
    _check(load().photon_decoder_step(ctx, byref(layer), byref(scratch), _ptr(x), byref(chunks), _ptr(y),
                                      c_float(scale), _stream(stream)), "photon_decoder_step")


def photon_encoder_step(ctx, layer: photon_layer, scratch: photon_layer_scratch, x, cache: photon_kv, y,
                        scale=1.0, stream=None) -> None:
    _check(load().photon_encoder_step(ctx, byref(layer), byref(scratch), _ptr(x), byref(cache), _ptr(y),
                                      c_float(scale), _stream(stream)), "photon_encoder_step")


def photon_chunk_causal_attn(ctx, chunks: photon_kv, q, slot, out, Nc=None, row0=0, rows=None,
                             scale=1.0, stream=None) -> None:
    if Nc is None:
        Nc = q.shape[0]
    if rows is None:
        rows = q.shape[1]
    _check(load().photon_chunk_causal_attn(ctx, byref(chunks), _ptr(q), _ptr(slot), _ptr(out), int(Nc),
                                           int(row0), int(rows), c_float(scale), _stream(stream)),
           "photon_chunk_causal_attn")


def photon_chunk_attn(ctx, chunks: photon_kv, q, slot, out, Nc=None, scale=1.0, stream=None) -> None:
    if Nc is None:
        Nc = q.shape[0]
    _check(load().photon_chunk_attn(ctx, byref(chunks), _ptr(q), _ptr(slot), _ptr(out), int(Nc),
                                    c_float(scale), _stream(stream)), "photon_chunk_attn")


def make_step_args(coarse: photon_kv, k_new, v_new, q_coarse, out_coarse, scale_coarse, w, w_layout,
                   U, B, chunks: photon_kv | None = None, q_chunk=None, out_chunk=None, Nc=0,
                   scale_chunk=1.0, x=None, bias=None, lse_coarse=None, slot=None,
                   ev_attn_begin=None, ev_attn_end=None) -> photon_step_args:
    a = photon_step_args()
    a.coarse = ctypes.pointer(coarse)
    a.k_new, a.v_new, a.q_coarse = _ptr(k_new), _ptr(v_new), _ptr(q_coarse)
    a.out_coarse, a.lse_coarse, a.scale_coarse = _ptr(out_coarse), _ptr(lse_coarse), scale_coarse
    a.x, a.w, a.bias, a.w_layout = _ptr(x), _ptr(w), _ptr(bias), int(w_layout)
    a.U, a.B = _ptr(U), int(B)
    if chunks is not None:
        a.chunks = ctypes.pointer(chunks)
    a.q_chunk, a.slot, a.out_chunk = _ptr(q_chunk), _ptr(slot), _ptr(out_chunk)
    a.Nc, a.scale_chunk = int(Nc), scale_chunk
    a.ev_attn_begin = c_void_p(ev_attn_begin.cuda_event if ev_attn_begin is not None else 0)
    a.ev_attn_end = c_void_p(ev_attn_end.cuda_event if ev_attn_end is not None else 0)
    a._keep = (coarse, chunks, k_new, v_new, q_coarse, out_coarse, lse_coarse, x, w, bias, U,
               q_chunk, slot, out_chunk, ev_attn_begin, ev_attn_end)
    return a


def photon_decode_step(ctx, args: photon_step_args, stream=None) -> None:
    _check(load().photon_decode_step(ctx, byref(args), _stream(stream)), "photon_decode_step")


class HostIO:
    """The four buffers of photon_decode_step_host, checked once: host_in / host_out are CPU uint8
    tensors (pinned for asynchronous copies), dev_in / dev_out the device staging tensors that the
    pointers of the step's arguments look into; `stream` is looked up once, here (None: the
    stream that is current now).  in_split / out_split: the leading bytes that belong to the coarse
    part of the step, the rest being the chunk attention's (None: no split, everything is copied
    before and after the step).  Keeps the tensors alive."""

    def __init__(self, host_in, dev_in, dev_out, host_out, stream=None, in_split=None, out_split=None):
        for h, d in ((host_in, dev_in), (host_out, dev_out)):
            if h.is_cuda or not d.is_cuda or not h.is_contiguous() or not d.is_contiguous():
                raise ValueError("host tensors on the CPU, staging tensors on the device, both contiguous")
            if h.numel() * h.element_size() != d.numel() * d.element_size():
                raise ValueError("a host buffer and its staging area differ in size")
        self._keep = (host_in, dev_in, dev_out, host_out)
        n_in, n_out = host_in.numel() * host_in.element_size(), host_out.numel() * host_out.element_size()
        self.argv = (c_void_p(host_in.data_ptr()), c_void_p(dev_in.data_ptr()), c_size_t(n_in),
                     c_size_t(n_in if in_split is None else in_split), c_void_p(dev_out.data_ptr()),
                     c_void_p(host_out.data_ptr()), c_size_t(n_out), c_size_t(n_out if out_split is None else out_split),
                     _stream(stream))
        self._call = load().photon_decode_step_host


def photon_decode_step_host(ctx, args: photon_step_args, io: HostIO) -> None:
    """Copy in, decode step, copy out on io's stream; returns once io's host_out holds the results.
    Nothing is looked up per call: the host's time before the first copy is enqueued is the step's latency."""
    rc = io._call(ctx, byref(args), *io.argv)
    if rc != PHOTON_OK:
        _check(rc, "photon_decode_step_host")


def photon_device_status(ctx, clear=True) -> int:
    bits = c_int32(0)
    _check(load().photon_device_status(ctx, byref(bits), int(bool(clear))), "photon_device_status")
    return bits.value


def photon_set_attention_ctas(ctx, n: int) -> None:
    _check(load().photon_set_attention_ctas(ctx, int(n)), "photon_set_attention_ctas")


def photon_read_probe(ctx, src, nbytes=None, ctas=0, sum_out=None, stream=None) -> None:
    """Streams the first nbytes of the device tensor src through the attention kernels' kind of ring (see photon.h)."""
    if nbytes is None:
        nbytes = src.numel() * src.element_size()
    _check(load().photon_read_probe(ctx, _ptr(src), c_size_t(int(nbytes)), int(ctas), _ptr(sum_out), _stream(stream)),
           "photon_read_probe")


def photon_wait_probe(ctx, limit_ns=1_000_000, stream=None) -> None:
    _check(load().photon_wait_probe(ctx, c_int64(int(limit_ns)), _stream(stream)), "photon_wait_probe")


def photon_set_host_step_tuning(ctx, pause_ns: int = 1500, poll_us: int = 2000) -> None:
    _check(load().photon_set_host_step_tuning(ctx, c_int64(int(pause_ns)), c_int64(int(poll_us))),
           "photon_set_host_step_tuning")


def photon_launch_count(ctx) -> int:
    return int(load().photon_launch_count(ctx))
