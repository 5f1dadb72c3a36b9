"""ctypes front end of the CPU oracle (oracle/photon_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg; never by the product package.  Arrays are numpy:
bf16 tensors as raw uint16 bits, results as float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "photon_oracle.cpp")
_LIB = os.path.join(_HERE, "libphoton_oracle.so")

DEV_CAPACITY = 1
DEV_BAD_INDEX = 2


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (plain -O2, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread",
                               "-o", _LIB, _SRC])
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_kv_append.restype = ctypes.c_int
        _lib.oracle_attention.restype = ctypes.c_int
        _lib.oracle_chunk_causal_attention.restype = ctypes.c_int
        _lib.oracle_hardware_threads.restype = ctypes.c_int
    return _lib


def _p(a):
    if a is None:
        return ctypes.c_void_p(0)
    assert a.flags["C_CONTIGUOUS"], "oracle arrays must be C-contiguous"
    return ctypes.c_void_p(a.ctypes.data)


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16
    return a


def _i32(a):
    if a is None:
        return None
    a = np.ascontiguousarray(a)
    assert a.dtype == np.int32
    return a


def hardware_threads() -> int:
    return lib().oracle_hardware_threads()


def kv_append(k, v, length, k_new, v_new, unit_ids=None, n_rows=1) -> int:
    """In-place append (Eq. 12 / Eq. 13, cache half).  k, v: [n_units, Hkv, cap, dh]
    uint16; length: [n_units] int32; k_new, v_new: [n, n_rows, Hkv, dh] (or
    [n, Hkv, dh] when n_rows == 1).  Returns device-style flag bits."""
    n_units, Hkv, cap, dh = k.shape
    assert k.dtype == np.uint16 and v.dtype == np.uint16 and length.dtype == np.int32
    assert k.flags["C_CONTIGUOUS"] and v.flags["C_CONTIGUOUS"] and length.flags["C_CONTIGUOUS"]
    k_new, v_new = _u16(k_new), _u16(v_new)
    n = k_new.shape[0]
    assert k_new.size == n * n_rows * Hkv * dh and v_new.size == k_new.size
    unit_ids = _i32(unit_ids)
    return lib().oracle_kv_append(_p(k), _p(v), _p(length), n_units, Hkv, cap, dh,
                                  _p(k_new), _p(v_new), _p(unit_ids), n, n_rows)


def attention(q, k, v, length, scale, slot=None, shared=None, n_threads=1, want_flags=False):
    """Softmax attention of each query over the valid rows of its cache unit
    (and, when `shared` is given, its shared prefix first).  q: [n_q, Hq, dh];
    k, v: [n_units, Hkv, cap, dh]; length: [n_units].  shared = dict(k, v,
    len, id) with k, v: [n_shared, Hkv, cap_sh, dh].  Returns (out, lse) as
    float64 [n_q, Hq, dh] and [n_q, Hq]."""
    q, k, v = _u16(q), _u16(k), _u16(v)
    length = _i32(length)
    n_q, Hq, dh = q.shape
    n_units, Hkv, cap, dh2 = k.shape
    assert dh == dh2 and Hq % Hkv == 0 and v.shape == k.shape
    slot = _i32(slot)
    if slot is None:
        assert n_q == n_units
    ks = vs = sl = sid = None
    n_sh = cap_sh = 0
    if shared is not None:
        ks, vs = _u16(shared["k"]), _u16(shared["v"])
        sl, sid = _i32(shared["len"]), _i32(shared["id"])
        n_sh, _, cap_sh, _ = ks.shape
    out = np.empty((n_q, Hq, dh), dtype=np.float64)
    lse = np.empty((n_q, Hq), dtype=np.float64)
    flags = lib().oracle_attention(_p(q), n_q, _p(slot), _p(k), _p(v), _p(length),
                                   n_units, Hq, Hkv, cap, dh, _p(ks), _p(vs), _p(sl), _p(sid),
                                   n_sh, cap_sh, ctypes.c_double(scale), _p(out), _p(lse),
                                   int(n_threads))
    return (out, lse, flags) if want_flags else (out, lse)


def chunk_attention(q, kc, vc, length, scale, slot=None, n_threads=1):
    """Bounded attention of the local decoders (Eq. 6-7): query c attends rows
    [0, length[c]) of its own chunk buffer only (P prefix rows then the
    in-chunk rows)."""
    return attention(q, kc, vc, length, scale, slot=slot, n_threads=n_threads)


def chunk_causal_attention(q, kc, vc, length, scale, row0=0, slot=None, n_threads=1,
                           want_flags=False):
    """The local decoder at R positions of every chunk at once (teacher-forced form
    of Eq. 6 under the causal mask below Eq. 7).  q: [n, R, Hq, dh]; query t stands
    at row row0 + t of its chunk buffer (kc, vc: [n_units, Hkv, cap, dh]) and attends
    rows 0 .. row0 + t; positions >= length[u] give zero rows.  Returns float64
    [n, R, Hq, dh]."""
    q, kc, vc = _u16(q), _u16(kc), _u16(vc)
    length = _i32(length)
    n, R, Hq, dh = q.shape
    n_units, Hkv, cap, dh2 = kc.shape
    assert dh == dh2 and Hq % Hkv == 0 and vc.shape == kc.shape
    slot = _i32(slot)
    if slot is None:
        assert n == n_units
    out = np.empty((n, R, Hq, dh), dtype=np.float64)
    flags = lib().oracle_chunk_causal_attention(_p(q), n, R, int(row0), _p(slot), _p(kc), _p(vc),
                                                _p(length), n_units, Hq, Hkv, cap, dh,
                                                ctypes.c_double(scale), _p(out), int(n_threads))
    return (out, flags) if want_flags else out


def attn_range(q_vec, k_rows, v_rows, r0, r1, scale):
    """One query vector over rows [r0, r1) of k_rows, v_rows: [rows, dh]."""
    q_vec, k_rows, v_rows = _u16(q_vec), _u16(k_rows), _u16(v_rows)
    dh = q_vec.shape[-1]
    o = np.empty(dh, dtype=np.float64)
    lse = ctypes.c_double(0.0)
    lib().oracle_attn_range(_p(q_vec), _p(k_rows), _p(v_rows), int(r0), int(r1), dh,
                            ctypes.c_double(scale), _p(o), ctypes.byref(lse))
    return o, lse.value


def lse_merge(o_parts, lse_parts):
    """Log-sum-exp combination of partial attentions: o_parts [n, dh], lse_parts [n]."""
    o_parts = np.ascontiguousarray(o_parts, dtype=np.float64)
    lse_parts = np.ascontiguousarray(lse_parts, dtype=np.float64)
    n, dh = o_parts.shape
    o = np.empty(dh, dtype=np.float64)
    lse = ctypes.c_double(0.0)
    lib().oracle_lse_merge(n, dh, _p(o_parts), _p(lse_parts), _p(o), ctypes.byref(lse))
    return o, lse.value


def converter(x, w, bias=None, w_out_major=False, n_threads=1):
    """Context converter (Section 2.1.2): U[b, r, :] = x[b, :] . W[:, r*D:(r+1)*D] + bias.
    x: [B, D]; w: [D, P*D] (or [P*D, D] when w_out_major).  Returns float64 [B, P, D]."""
    x, w = _u16(x), _u16(w)
    B, D = x.shape
    if w_out_major:
        N, D2 = w.shape
    else:
        D2, N = w.shape
    assert D2 == D and N % D == 0
    P = N // D
    bias = None if bias is None else _u16(bias)
    out = np.empty((B, P, D), dtype=np.float64)
    lib().oracle_converter(_p(x), _p(w), int(bool(w_out_major)), _p(bias), B, D, P, _p(out),
                           int(n_threads))
    return out


def rmsnorm(x, gamma=None, eps=0.0):
    """Root-mean-square normalisation of each row of x [rows, cols] with an optional
    per-column scale (first half of the context chunker).  Returns float64."""
    x = _u16(x)
    rows, cols = x.shape
    gamma = None if gamma is None else _u16(gamma)
    out = np.empty((rows, cols), dtype=np.float64)
    lib().oracle_rmsnorm(_p(x), _p(gamma), ctypes.c_double(eps), rows, cols, _p(out))
    return out


def linear(x, w, bias=None, w_out_major=False, n_threads=1):
    """y = x W + b.  x: [B, K]; w: [K, N] (or [N, K] when w_out_major).  Returns float64 [B, N]."""
    x, w = _u16(x), _u16(w)
    B, K = x.shape
    N = w.shape[0] if w_out_major else w.shape[1]
    assert (w.shape[1] if w_out_major else w.shape[0]) == K
    bias = None if bias is None else _u16(bias)
    out = np.empty((B, N), dtype=np.float64)
    lib().oracle_linear(_p(x), _p(w), int(bool(w_out_major)), _p(bias), B, K, N, _p(out), int(n_threads))
    return out


def chunker(x, gamma, eps, w, bias=None, w_out_major=False, n_threads=1):
    """Level-L context chunker (Section 2.1.1; step (ii) of Section 2.3.3): the C_L
    reconstructed lower-level latents of a meta-context, concatenated (x: [B, C*D]),
    normalised with a learned scale, rounded to bf16 (what the linear part reads),
    then mapped to D_L.  Returns (normalised bf16 bits [B, C*D], float64 [B, N])."""
    xn = round_bf16(rmsnorm(x, gamma, eps))
    return xn, linear(xn, w, bias, w_out_major=w_out_major, n_threads=n_threads)


def rope_split(qkv, pos, Hq, Hkv, dh, theta=10000.0):
    """Split a fused projection [n, (Hq + 2 Hkv) dh] into q, k, v and rotate q and k
    by the item's position (half-split pairing, base theta).  Returns float64
    (q [n, Hq, dh], k [n, Hkv, dh], v [n, Hkv, dh])."""
    qkv, pos = _u16(qkv), _i32(pos)
    n = qkv.shape[0]
    assert qkv.shape[1] == (Hq + 2 * Hkv) * dh and dh % 2 == 0
    q = np.empty((n, Hq, dh)); k = np.empty((n, Hkv, dh)); v = np.empty((n, Hkv, dh))
    lib().oracle_rope_split(_p(qkv), _p(pos), n, Hq, Hkv, dh, ctypes.c_double(theta), _p(q), _p(k), _p(v))
    return q, k, v


def swiglu(gu):
    """silu(gate) * up for gu [n, 2F] = [gate | up].  Returns float64 [n, F]."""
    gu = _u16(gu)
    n, F2 = gu.shape
    out = np.empty((n, F2 // 2))
    lib().oracle_swiglu(_p(gu), n, F2 // 2, _p(out))
    return out


def encoder_step(x, lw, cache, scale, eps=1e-5, theta=10000.0, n_threads=1):
    """STEP of one LLaMA layer of the top-level context encoder for the newest
    latent of every sequence (Eq. 12 / Eq. 13 with the layer written out): x [B, D]
    -> normalise -> fused q/k/v projection -> rotary encoding at position len[b]
    -> append k, v -> attention over the grown cache -> output projection + residual
    -> normalise -> gate/up projection -> silu(g) * u -> down projection + residual.
    Every intermediate is rounded to bf16 where the next part reads it.  lw: dict of
    bf16 weights g1 [D], wqkv [D, (Hq+2Hkv) dh], wo [Hq dh, D], g2 [D], wgu [D, 2F],
    wdown [F, D] (all in-major).  cache: dict k, v [B, Hkv, cap, dh], len [B] (grown
    in place).  Returns dict of the bf16 intermediates and y (float64 [B, D])."""
    B, D = x.shape
    Hkv, dh = cache["k"].shape[1], cache["k"].shape[3]
    Hq = lw["wo"].shape[0] // dh
    n1 = round_bf16(rmsnorm(x, lw["g1"], eps))
    qkv = round_bf16(linear(n1, lw["wqkv"], n_threads=n_threads))
    q, k_new, v_new = (round_bf16(t) for t in rope_split(qkv, cache["len"], Hq, Hkv, dh, theta))
    flags = kv_append(cache["k"], cache["v"], cache["len"], k_new, v_new)
    att, _ = attention(q, cache["k"], cache["v"], cache["len"], scale, n_threads=n_threads)
    att = round_bf16(att).reshape(B, Hq * dh)
    h = round_bf16(linear(att, lw["wo"], n_threads=n_threads) + widen_bf16(x))
    n2 = round_bf16(rmsnorm(h, lw["g2"], eps))
    gu = round_bf16(linear(n2, lw["wgu"], n_threads=n_threads))
    act = round_bf16(swiglu(gu))
    y = linear(act, lw["wdown"], n_threads=n_threads) + widen_bf16(h)
    return {"n1": n1, "qkv": qkv, "q": q, "k_new": k_new, "v_new": v_new, "att": att, "h": h, "n2": n2,
            "gu": gu, "act": act, "y": y, "flags": flags}


def decoder_prefill(U, lw, chunks, scale, unit_ids=None, eps=1e-5, theta=10000.0, n_threads=1):
    """The pass of one local-decoder layer over a fresh converter prefix (the first R_l
    positions of the sequence [U ; X_<j] of Eq. 6, before any in-chunk position exists):
    U [n, P, D] -> normalise -> fused q/k/v projection -> rotary encoding at positions
    0..P-1 -> the P key/value rows become rows 0..P-1 of the chunk buffers unit_ids[i]
    (which must be empty) -> causal attention among the P rows -> output projection +
    residual -> MLP + residual.  Intermediates are rounded to bf16 as in encoder_step.
    chunks: dict k, v [n_units, Hkv, cap, dh], len [n_units] (grown in place).
    Returns dict with y (float64 [n, P, D]) and the bf16 intermediates."""
    n, P, D = U.shape
    Hkv, dh = chunks["k"].shape[1], chunks["k"].shape[3]
    Hq = lw["wo"].shape[0] // dh
    x = np.ascontiguousarray(U).reshape(n * P, D)
    pos = np.tile(np.arange(P, dtype=np.int32), n)
    n1 = round_bf16(rmsnorm(x, lw["g1"], eps))
    qkv = round_bf16(linear(n1, lw["wqkv"], n_threads=n_threads))
    q, k_new, v_new = (round_bf16(t) for t in rope_split(qkv, pos, Hq, Hkv, dh, theta))
    flags = kv_append(chunks["k"], chunks["v"], chunks["len"], k_new.reshape(n, P, Hkv, dh),
                      v_new.reshape(n, P, Hkv, dh), unit_ids=unit_ids, n_rows=P)
    att = chunk_causal_attention(q.reshape(n, P, Hq, dh), chunks["k"], chunks["v"], chunks["len"], scale,
                                 slot=unit_ids, n_threads=n_threads)
    att = round_bf16(att).reshape(n * P, Hq * dh)
    h = round_bf16(linear(att, lw["wo"], n_threads=n_threads) + widen_bf16(x))
    n2 = round_bf16(rmsnorm(h, lw["g2"], eps))
    gu = round_bf16(linear(n2, lw["wgu"], n_threads=n_threads))
    act = round_bf16(swiglu(gu))
    y = linear(act, lw["wdown"], n_threads=n_threads) + widen_bf16(h)
    return {"qkv": qkv, "q": q, "k_new": k_new, "v_new": v_new, "att": att, "h": h, "act": act,
            "y": y.reshape(n, P, D), "flags": flags}


def round_bf16(x):
    """float64 -> bf16 bits, round to nearest even."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(x.shape, dtype=np.uint16)
    lib().oracle_round_bf16(_p(x), ctypes.c_int64(x.size), _p(out))
    return out


def widen_bf16(b):
    b = _u16(b)
    out = np.empty(b.shape, dtype=np.float64)
    lib().oracle_widen_bf16(_p(b), ctypes.c_int64(b.size), _p(out))
    return out


def decode_step(coarse, conv, chunks, scale_coarse, scale_chunk, chain=True, w_out_major=False,
                n_threads=1):
    """One meta-context step in the order of Section 2.3.3: append the new coarse
    unit (Eq. 13), attend over the grown cache, expand the result into prefix
    vectors (converter), and run the chunk-local attention of every in-flight
    chunk.  Each part's output is rounded to bf16 before the next part reads it.
    Mutates coarse['k'], coarse['v'], coarse['len'] in place.
    chain=True feeds the attention output, viewed as [B, Hq*dh], to the converter;
    otherwise conv['x'] is used.  Returns dict(out, lse, U, chunk_out, flags)."""
    flags = kv_append(coarse["k"], coarse["v"], coarse["len"], coarse["k_new"], coarse["v_new"])
    shared = None
    if "k_shared" in coarse:
        shared = {"k": coarse["k_shared"], "v": coarse["v_shared"],
                  "len": coarse["shared_len"], "id": coarse["shared_id"]}
    out, lse = attention(coarse["q"], coarse["k"], coarse["v"], coarse["len"], scale_coarse,
                         shared=shared, n_threads=n_threads)
    B = out.shape[0]
    x = round_bf16(out).reshape(B, -1) if chain else conv["x"]
    w = conv["w_out_major"] if w_out_major else conv["w_in_major"]
    U = converter(x, w, conv.get("bias"), w_out_major=w_out_major, n_threads=n_threads)
    co, _ = chunk_attention(chunks["q"], chunks["kc"], chunks["vc"], chunks["len"], scale_chunk,
                            slot=chunks.get("slot"), n_threads=n_threads)
    return {"out": out, "lse": lse, "U": U, "chunk_out": co, "flags": flags}
