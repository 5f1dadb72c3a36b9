"""Parity of the remaining kernels of an encoder layer (rotary encoding with the
split of the fused projection, gated activation, residual in the linear map) and
of the composed STEP of one layer with the CPU oracle, through the C boundary.
bf16 outputs: max abs error 2e-2, mean abs error 2e-3 against the fp64 oracle."""
import numpy as np
import pytest
import torch

import paper_2512_20687_b200 as ph
from paper_2512_20687_b200 import workloads as wl

from gpu_util import Ctx, assert_close, assert_close_scaled, dev_bf16, dev_i32, host_bits, host_f64

pytestmark = pytest.mark.gpu

NT = 16     # oracle threads


def cfg_small(i, **kw):
    return wl.scaled(wl.CONFIGS[i], **kw)


@pytest.mark.parametrize("idx,n", [(0, 37), (1, 37), (4, 37), (1, 2999), (4, 1185)])
def test_rope_split_matches_oracle(oracle, idx, n):
    # 2999 and 1185 items: more than the CTAs that are resident at once, so a CTA takes several, unevenly
    cfg = cfg_small(idx, B=n)
    Hq, Hkv, dh = cfg.Hq, cfg.Hkv, cfg.dh
    qkv = wl.normal_bf16(41, "qkv", (cfg.B, (Hq + 2 * Hkv) * dh))
    pos = (np.arange(cfg.B) * 229 % 8192).astype(np.int32)
    pos[:3] = [0, 1, 8191]
    wq, wk, wv = oracle.rope_split(qkv, pos, Hq, Hkv, dh, 10000.0)
    with Ctx(cfg) as c:
        q = torch.empty(cfg.B, Hq, dh, dtype=torch.bfloat16, device="cuda")
        k = torch.empty(cfg.B, Hkv, dh, dtype=torch.bfloat16, device="cuda")
        v = torch.empty_like(k)
        ph.photon_rope_split(c.h, dev_bf16(qkv), dev_i32(pos), q, k, v)
        assert c.status() == 0
    # a rotation of O(1) values rounded once: within half a bf16 step of the oracle (|x| < 8 here)
    assert np.abs(host_f64(q) - wq).max() <= 2.0 ** -6 and np.abs(host_f64(k) - wk).max() <= 2.0 ** -6
    assert_close(host_f64(q), wq, "rope q")
    assert_close(host_f64(k), wk, "rope k")
    assert np.array_equal(host_bits(v).reshape(cfg.B, -1), qkv[:, (Hq + Hkv) * dh:])       # v: a bit copy
    assert np.array_equal(host_bits(q)[0].reshape(-1), qkv[0, : Hq * dh])                   # position 0: identity


@pytest.mark.parametrize("n,F", [(64, 5632), (3, 8), (513, 1024)])
def test_swiglu_matches_oracle(oracle, n, F):
    gu = wl.normal_bf16(42, "gu", (n, 2 * F), std=1.5)
    want = oracle.swiglu(gu)
    with Ctx(cfg_small(0)) as c:
        out = torch.empty(n, F, dtype=torch.bfloat16, device="cuda")
        ph.photon_swiglu(c.h, dev_bf16(gu), out)
        assert c.status() == 0
    got = host_f64(out)
    # one rounding to bf16 (half a step is 2^-9 relative) on top of a fast exponential
    assert np.all(np.abs(got - want) <= 2.0 ** -8 * np.abs(want) + 1e-4)


@pytest.mark.parametrize("B,K,N", [(64, 2048, 2048), (200, 1024, 8192)])
def test_linear_adds_the_residual_before_rounding(oracle, B, K, N):
    x = wl.normal_bf16(43, "x", (B, K))
    w = wl.normal_bf16(43, "w", (K, N), std=K ** -0.5)
    res = wl.normal_bf16(43, "r", (B, N))
    want = oracle.linear(x, w, n_threads=NT) + wl.bf16_bits_to_f64(res)
    with Ctx(cfg_small(0)) as c:
        y = dev_bf16(res).clone()                                       # the residual aliases the output
        ph.photon_linear(c.h, dev_bf16(x), dev_bf16(w), ph.PHOTON_W_IN_MAJOR, None, y, residual=y)
        assert c.status() == 0
    assert_close(host_f64(y), want, "linear + residual")


@pytest.mark.parametrize("idx,B,S,F", [(0, 5, 40, 128), (1, 64, 512, 5632), (4, 130, 128, 2816)])
def test_encoder_step_matches_oracle(oracle, idx, B, S, F):
    """STEP of one layer: every intermediate that the next kernel reads, the grown
    cache (bit-exact given the same appended rows) and the layer's output."""
    cfg = cfg_small(idx, B=B, S=S)
    lw = wl.encoder_layer_inputs(cfg, F=F)
    co = wl.coarse_inputs(cfg, poison=True)
    lens = (co["len"] - (np.arange(B) % 7)).clip(0).astype(np.int32)     # ragged positions
    for u, n in enumerate(lens):
        co["k"][u, :, n:] = 0x7FC1
        co["v"][u, :, n:] = 0x7FC1
    scale = cfg.dh ** -0.5
    cache = {"k": co["k"].copy(), "v": co["v"].copy(), "len": lens.copy()}
    want = oracle.encoder_step(lw["x"], lw, cache, scale, n_threads=NT)
    with Ctx(cfg) as c:
        dk, dv, dl = dev_bf16(co["k"]), dev_bf16(co["v"]), dev_i32(lens)
        kv = ph.make_kv(dk, dv, dl)
        W = {n: dev_bf16(lw[n]) for n in ("g1", "wqkv", "wo", "g2", "wgu", "wdown")}
        layer = ph.make_layer(W["g1"], W["wqkv"], W["wo"], W["g2"], W["wgu"], W["wdown"], ph.PHOTON_W_IN_MAJOR, F)
        sc = ph.make_layer_scratch(B, cfg.Hq, cfg.Hkv, cfg.dh, F, "cuda", torch.bfloat16)
        x = dev_bf16(lw["x"])
        y = torch.empty_like(x)
        sc.tensors["gu"].fill_(-77.0)
        ph.photon_encoder_step(c.h, layer, sc, x, kv, y, scale=scale)
        assert c.status() == 0
        assert np.array_equal(dl.cpu().numpy(), lens + 1)
        t = sc.tensors
        # Where the 64-feature slabs of the gate/up projection occupy most of the GPU the activation is folded
        # into that kernel and the projection itself is never written; the activation's output is checked either way.
        sms = torch.cuda.get_device_properties(0).multi_processor_count
        fused = F % 64 == 0 and (F // 64) * ((B + 127) // 128) * 2 >= sms
        assert fused == (idx != 0)
        assert bool((t["gu"] == -77.0).all()) == fused
        # the chain as a whole: intermediates and output against the oracle's chain, with the slack a
        # chain of bf16 roundings needs (each kernel by itself is held to the plain bar below)
        for name in ("n", "qkv", "q", "att", "h") + (() if fused else ("gu",)) + ("act",):
            key = "n2" if name == "n" else name                          # `n` holds the second normalisation at the end
            got, ref = host_f64(t[name]).reshape(B, -1), wl.bf16_bits_to_f64(want[key]).reshape(B, -1)
            assert_close_scaled(got, ref, f"encoder step {name}", slack=2.0)
        # the split writes k and v straight into the cache: the new row holds the rotated key and a bit copy
        # of the value part of the fused projection, and no other row has changed
        hk, hv = host_bits(dk), host_bits(dv)
        v_part = host_bits(t["qkv"]).reshape(B, -1)[:, (cfg.Hq + cfg.Hkv) * cfg.dh:].reshape(B, cfg.Hkv, cfg.dh)
        new_k = np.stack([hk[u, :, lens[u]] for u in range(B)])
        assert_close_scaled(wl.bf16_bits_to_f64(new_k).reshape(B, -1), wl.bf16_bits_to_f64(want["k_new"]).reshape(B, -1),
                            "encoder step appended k", slack=2.0)
        for u in range(B):
            assert np.array_equal(hv[u, :, lens[u]], v_part[u])
            hk[u, :, lens[u]] = co["k"][u, :, lens[u]]
            hv[u, :, lens[u]] = co["v"][u, :, lens[u]]
        assert np.array_equal(hk, co["k"]) and np.array_equal(hv, co["v"])
    assert_close_scaled(host_f64(y), want["y"], f"encoder step cfg{idx}", slack=2.0)


def test_layer_step_gives_the_same_bits_for_both_weight_layouts():
    """The step of the default workload's layer with the weights stored [K, N] and stored [N, K] (the gate/up
    projection with the activation folded in reads its gate rows and its up rows apart in the second form):
    same bits in every intermediate and in the output."""
    cfg = cfg_small(1, B=64, S=512)
    F = 5632
    lw = wl.encoder_layer_inputs(cfg, F=F)
    co = wl.coarse_inputs(cfg)
    scale = cfg.dh ** -0.5
    res = []
    with Ctx(cfg) as c:
        for layout in (ph.PHOTON_W_IN_MAJOR, ph.PHOTON_W_OUT_MAJOR):
            dk, dv, dl = dev_bf16(co["k"]), dev_bf16(co["v"]), dev_i32(co["len"])
            kv = ph.make_kv(dk, dv, dl)
            W = {n: dev_bf16(lw[n] if layout == ph.PHOTON_W_IN_MAJOR or lw[n].ndim == 1 else np.ascontiguousarray(lw[n].T))
                 for n in ("g1", "wqkv", "wo", "g2", "wgu", "wdown")}
            layer = ph.make_layer(W["g1"], W["wqkv"], W["wo"], W["g2"], W["wgu"], W["wdown"], layout, F)
            sc = ph.make_layer_scratch(64, cfg.Hq, cfg.Hkv, cfg.dh, F, "cuda", torch.bfloat16)
            x = dev_bf16(lw["x"])
            y = torch.empty_like(x)
            ph.photon_encoder_step(c.h, layer, sc, x, kv, y, scale=scale)
            assert c.status() == 0
            res.append({n: host_bits(sc.tensors[n]) for n in ("qkv", "att", "h", "act")} | {"y": host_bits(y)})
    for n in res[0]:
        assert np.array_equal(res[0][n], res[1][n]), n


@pytest.mark.parametrize("idx,B,S,F", [(1, 64, 512, 5632)])
def test_each_kernel_of_the_layer_on_the_oracles_own_intermediates(oracle, idx, B, S, F):
    """Every kernel of the layer fed with the oracle's bf16 intermediate, so that no
    difference is carried from one kernel into the next: the plain bar per kernel."""
    cfg = cfg_small(idx, B=B, S=S)
    lw = wl.encoder_layer_inputs(cfg, F=F)
    co = wl.coarse_inputs(cfg)
    scale = cfg.dh ** -0.5
    lens = co["len"].copy()
    cache = {"k": co["k"].copy(), "v": co["v"].copy(), "len": lens.copy()}
    w = oracle.encoder_step(lw["x"], lw, cache, scale, n_threads=NT)
    f64 = wl.bf16_bits_to_f64
    D, Hq, Hkv, dh = cfg.D, cfg.Hq, cfg.Hkv, cfg.dh
    IN = ph.PHOTON_W_IN_MAJOR
    with Ctx(cfg) as c:
        def new(*shape):
            return torch.empty(shape, dtype=torch.bfloat16, device="cuda")
        n1, qkv, h, n2, gu, act, y = new(B, D), new(B, (Hq + 2 * Hkv) * dh), new(B, D), new(B, D), new(B, 2 * F), new(B, F), new(B, D)
        q, k, v, att = new(B, Hq, dh), new(B, Hkv, dh), new(B, Hkv, dh), new(B, Hq, dh)
        ph.photon_rmsnorm(c.h, dev_bf16(lw["x"]), dev_bf16(lw["g1"]), 1e-5, n1)
        ph.photon_linear(c.h, dev_bf16(w["n1"]), dev_bf16(lw["wqkv"]), IN, None, qkv)
        ph.photon_rope_split(c.h, dev_bf16(w["qkv"]), dev_i32(lens), q, k, v)
        kv = ph.make_kv(dev_bf16(cache["k"]), dev_bf16(cache["v"]), dev_i32(cache["len"]))       # the oracle's grown cache
        ph.photon_coarse_attn(c.h, kv, dev_bf16(w["q"]), att, None, scale)
        ph.photon_linear(c.h, dev_bf16(w["att"]), dev_bf16(lw["wo"]), IN, None, h, residual=dev_bf16(lw["x"]))
        ph.photon_rmsnorm(c.h, dev_bf16(w["h"]), dev_bf16(lw["g2"]), 1e-5, n2)
        ph.photon_linear(c.h, dev_bf16(w["n2"]), dev_bf16(lw["wgu"]), IN, None, gu)
        ph.photon_swiglu(c.h, dev_bf16(w["gu"]), act)
        ph.photon_linear(c.h, dev_bf16(w["act"]), dev_bf16(lw["wdown"]), IN, None, y, residual=dev_bf16(w["h"]))
        assert c.status() == 0
    for got, ref, what in ((n1, w["n1"], "norm 1"), (qkv, w["qkv"], "q/k/v projection"), (q, w["q"], "rotated q"),
                           (k, w["k_new"], "rotated k"), (att, w["att"], "attention"), (h, w["h"], "output projection"),
                           (n2, w["n2"], "norm 2"), (gu, w["gu"], "gate/up projection"), (act, w["act"], "activation")):
        assert_close_scaled(host_f64(got).reshape(B, -1), f64(ref).reshape(B, -1), what)
    assert np.array_equal(host_bits(v), w["v_new"])
    assert_close_scaled(host_f64(y), w["y"], "down projection")


@pytest.mark.parametrize("idx,B,chunks_per_seq", [(4, 16, 32), (1, 40, 2)])
def test_decoder_step_matches_oracle(oracle, idx, B, chunks_per_seq):
    """The same layer for the newest in-chunk position of every in-flight chunk: ragged
    chunk buffers (prefix rows + what has been written), positions = their lengths,
    the bounded chunk attention in the middle."""
    cfg = cfg_small(idx, B=B, chunks_per_seq=chunks_per_seq)
    Nc, F = cfg.Nc, 1024
    lcfg = wl.scaled(cfg, B=Nc)                                          # one token per chunk
    lw = wl.encoder_layer_inputs(lcfg, F=F)
    ch = wl.chunk_inputs(cfg, poison=True, strict_paper=True)            # len = P + n_in with room for one more row
    assert ch["len"].max() < ch["cap"]
    scale = cfg.dh ** -0.5
    cache = {"k": ch["kc"].copy(), "v": ch["vc"].copy(), "len": ch["len"].copy()}
    want = oracle.encoder_step(lw["x"], lw, cache, scale, n_threads=NT)
    with Ctx(cfg) as c:
        dk, dv, dl = dev_bf16(ch["kc"]), dev_bf16(ch["vc"]), dev_i32(ch["len"])
        kv = ph.make_kv(dk, dv, dl)
        W = {n: dev_bf16(lw[n]) for n in ("g1", "wqkv", "wo", "g2", "wgu", "wdown")}
        layer = ph.make_layer(W["g1"], W["wqkv"], W["wo"], W["g2"], W["wgu"], W["wdown"], ph.PHOTON_W_IN_MAJOR, F)
        sc = ph.make_layer_scratch(Nc, cfg.Hq, cfg.Hkv, cfg.dh, F, "cuda", torch.bfloat16)
        x = dev_bf16(lw["x"])
        y = torch.empty_like(x)
        ph.photon_decoder_step(c.h, layer, sc, x, kv, y, scale=scale)
        assert c.status() == 0
        assert np.array_equal(dl.cpu().numpy(), ch["len"] + 1)
        for name in ("qkv", "q", "att", "h", "act"):
            got, ref = host_f64(sc.tensors[name]).reshape(Nc, -1), wl.bf16_bits_to_f64(want[name]).reshape(Nc, -1)
            assert_close_scaled(got, ref, f"decoder step {name}", slack=2.0)
        hk = host_bits(dk)
        new_k = np.stack([hk[u, :, ch["len"][u]] for u in range(Nc)])          # written by the split itself
        assert_close_scaled(wl.bf16_bits_to_f64(new_k).reshape(Nc, -1), wl.bf16_bits_to_f64(want["k_new"]).reshape(Nc, -1),
                            "decoder step appended k", slack=2.0)
    assert_close_scaled(host_f64(y), want["y"], f"decoder step cfg{idx}", slack=2.0)


@pytest.mark.parametrize("idx,B,chunks_per_seq", [(1, 24, 2), (4, 6, 32), (0, 2, 8)])
def test_converter_output_reaches_the_chunk_buffers(oracle, idx, B, chunks_per_seq):
    """The chain the decode step leaves open: the converter's prefix vectors go through a
    decoder layer (positions 0..P-1), their keys and values become the first P rows of
    empty chunk buffers picked by unit_ids, they attend causally among themselves, and one
    decoder step for the first in-chunk position then reads exactly those rows."""
    cfg = cfg_small(idx, B=B, chunks_per_seq=chunks_per_seq)
    n, P, D, F = cfg.Nc, cfg.P, cfg.D, 1024
    cv = wl.converter_inputs(wl.scaled(cfg, B=n))
    lw = wl.encoder_layer_inputs(wl.scaled(cfg, B=n * P), F=F)
    cap = cfg.P + cfg.C
    n_units = n + 3
    ids = np.random.default_rng(idx).permutation(n_units)[:n].astype(np.int32)
    scale = cfg.dh ** -0.5
    U_or = oracle.round_bf16(oracle.converter(cv["x"], cv["w_in_major"], n_threads=NT))
    ochunks = {"k": np.full((n_units, cfg.Hkv, cap, cfg.dh), 0x7FC1, np.uint16),
               "v": np.full((n_units, cfg.Hkv, cap, cfg.dh), 0xFFC1, np.uint16), "len": np.zeros(n_units, np.int32)}
    want = oracle.decoder_prefill(U_or, lw, ochunks, scale, unit_ids=ids, n_threads=NT)
    with Ctx(cfg, max_queries=max(n * P, n_units)) as c:
        W = {k: dev_bf16(lw[k]) for k in ("g1", "wqkv", "wo", "g2", "wgu", "wdown")}
        layer = ph.make_layer(W["g1"], W["wqkv"], W["wo"], W["g2"], W["wgu"], W["wdown"], ph.PHOTON_W_IN_MAJOR, F)
        sc = ph.make_layer_scratch(n * P, cfg.Hq, cfg.Hkv, cfg.dh, F, "cuda", torch.bfloat16)
        dk, dv = dev_bf16(ochunks["k"] * 0 + 0x7FC1), dev_bf16(ochunks["v"] * 0 + 0xFFC1)
        dl = dev_i32(np.zeros(n_units, np.int32))
        kv = ph.make_kv(dk, dv, dl)
        U = torch.empty(n, P, D, dtype=torch.bfloat16, device="cuda")
        ph.photon_converter(c.h, dev_bf16(cv["x"]), dev_bf16(cv["w_in_major"]), ph.PHOTON_W_IN_MAJOR, None, U)
        assert_close(host_f64(U), wl.bf16_bits_to_f64(U_or), "converter")
        y = torch.empty_like(U)
        ph.photon_decoder_prefill(c.h, layer, sc, U, kv, dev_i32(ids), y, scale=scale)
        assert c.status() == 0
        assert np.array_equal(dl.cpu().numpy(), ochunks["len"])
        hk = host_bits(dk)
        got_k = host_bits(sc.tensors["k_new"]).reshape(n, P, cfg.Hkv, cfg.dh)
        for i, u in enumerate(ids):
            assert np.array_equal(hk[u, :, :P], got_k[i].transpose(1, 0, 2))      # the device's own rows, installed bit-exactly
            assert np.all(hk[u, :, P:] == 0x7FC1)
        for name in ("qkv", "q", "k_new", "att", "h", "act"):
            got, ref = host_f64(sc.tensors[name]).reshape(n * P, -1), wl.bf16_bits_to_f64(want[name]).reshape(n * P, -1)
            # one kernel more ahead of it than the encoder step (the converter), and the activation multiplies
            # two intermediates: three times the single-kernel bar
            assert_close_scaled(got, ref, f"prefill {name}", slack=3.0)
        assert_close_scaled(host_f64(y), want["y"], "prefill output", slack=3.0)
        # one decoder step for the first in-chunk position of the first chunks: it sees the P installed rows and itself
        m = min(n, cfg.Nc)
        lw2 = wl.encoder_layer_inputs(wl.scaled(cfg, B=n_units), F=F, replica=1)
        x2 = dev_bf16(lw2["x"])
        y2 = torch.empty_like(x2)
        sc2 = ph.make_layer_scratch(n_units, cfg.Hq, cfg.Hkv, cfg.dh, F, "cuda", torch.bfloat16)
        ph.photon_decoder_step(c.h, layer, sc2, x2, kv, y2, scale=scale)
        assert c.status() == 0
        want2 = oracle.encoder_step(lw2["x"], lw, ochunks, scale, n_threads=NT)
        assert np.array_equal(dl.cpu().numpy(), ochunks["len"])
        assert_close_scaled(host_f64(y2), want2["y"], "decoder step after prefill", slack=3.0)


@pytest.mark.parametrize("layout", ["in", "out"])
def test_decoder_step_with_thousands_of_chunks_fuses_the_activation(oracle, layout):
    """5120 in-flight chunks: the gate/up projection takes the persistent large-tile kernel with
    the activation in its epilogue (the [rows, 2F] intermediate is never written); both weight orders."""
    cfg = cfg_small(0, B=640, chunks_per_seq=8)                          # D 256, 4q/2kv x 64, P = C = 4
    Nc, F = cfg.Nc, 1024
    lw = wl.encoder_layer_inputs(wl.scaled(cfg, B=Nc), F=F)
    ch = wl.chunk_inputs(cfg, poison=True, strict_paper=True)
    scale = cfg.dh ** -0.5
    cache = {"k": ch["kc"].copy(), "v": ch["vc"].copy(), "len": ch["len"].copy()}
    want = oracle.encoder_step(lw["x"], lw, cache, scale, n_threads=NT)
    out_major = layout == "out"
    with Ctx(cfg) as c:
        kv = ph.make_kv(dev_bf16(ch["kc"]), dev_bf16(ch["vc"]), dev_i32(ch["len"]))
        names = ("g1", "wqkv", "wo", "g2", "wgu", "wdown")
        W = {n: dev_bf16(np.ascontiguousarray(lw[n].T) if out_major and lw[n].ndim == 2 else lw[n]) for n in names}
        layer = ph.make_layer(*(W[n] for n in names), ph.PHOTON_W_OUT_MAJOR if out_major else ph.PHOTON_W_IN_MAJOR, F)
        sc = ph.make_layer_scratch(Nc, cfg.Hq, cfg.Hkv, cfg.dh, F, "cuda", torch.bfloat16)
        sc.tensors["gu"].fill_(7.0)
        x = dev_bf16(lw["x"])
        y = torch.empty_like(x)
        n0 = ph.photon_launch_count(c.h)
        ph.photon_decoder_step(c.h, layer, sc, x, kv, y, scale=scale)
        assert c.status() == 0
        assert ph.photon_launch_count(c.h) - n0 == 8                     # one launch fewer than the nine of a small batch
        assert bool((sc.tensors["gu"] == 7.0).all())                     # the intermediate was not written
        assert_close_scaled(host_f64(sc.tensors["act"]), wl.bf16_bits_to_f64(want["act"]), "fused activation", slack=2.0)
    assert_close_scaled(host_f64(y), want["y"], "decoder step, 5120 chunks", slack=2.0)


def test_encoder_step_on_a_full_cache_and_on_pages(oracle):
    """The split appends by itself.  A unit whose cache is full sets the capacity bit and keeps its
    rows and its length while the other units step; a paged cache gives the bits of the contiguous one."""
    cfg = cfg_small(0, B=6, S=128)
    F = 128
    lw = wl.encoder_layer_inputs(cfg, F=F)
    co = wl.coarse_inputs(cfg)
    cap = co["k"].shape[2]
    lens = np.array([5, cap, 17, cap - 1, 0, 64], dtype=np.int32)
    scale = cfg.dh ** -0.5
    with Ctx(cfg) as c:
        W = {n: dev_bf16(lw[n]) for n in ("g1", "wqkv", "wo", "g2", "wgu", "wdown")}
        layer = ph.make_layer(W["g1"], W["wqkv"], W["wo"], W["g2"], W["wgu"], W["wdown"], ph.PHOTON_W_IN_MAJOR, F)
        sc = ph.make_layer_scratch(cfg.B, cfg.Hq, cfg.Hkv, cfg.dh, F, "cuda", torch.bfloat16)
        x = dev_bf16(lw["x"])
        dk, dv, dl = dev_bf16(co["k"]), dev_bf16(co["v"]), dev_i32(lens)
        y = torch.empty_like(x)
        ph.photon_encoder_step(c.h, layer, sc, x, ph.make_kv(dk, dv, dl), y, scale=scale)
        assert c.status() == ph.PHOTON_DEV_CAPACITY
        grown = lens + 1
        grown[1] = cap
        assert np.array_equal(dl.cpu().numpy(), grown)
        assert np.array_equal(host_bits(dk)[1], co["k"][1]) and np.array_equal(host_bits(dv)[1], co["v"][1])
        # the same step on pages scattered over a pool (cap = 2 pages of 64 rows per unit), lengths that fit
        assert cap == 128
        fit = np.minimum(lens, cap - 1).astype(np.int32)
        ck, cv, cl = dev_bf16(co["k"]), dev_bf16(co["v"]), dev_i32(fit)
        y1 = torch.empty_like(x)
        ph.photon_encoder_step(c.h, layer, sc, x, ph.make_kv(ck, cv, cl), y1, scale=scale)
        n_pages = 2 * cfg.B + 3
        ids = np.random.default_rng(5).permutation(n_pages)[: 2 * cfg.B].astype(np.int32).reshape(cfg.B, 2)
        pk = np.full((n_pages, cfg.Hkv, 64, cfg.dh), 0x7FC1, dtype=np.uint16)
        pv = pk.copy()
        for u in range(cfg.B):
            for r in range(2):
                pk[ids[u, r]] = co["k"][u, :, 64 * r: 64 * r + 64]
                pv[ids[u, r]] = co["v"][u, :, 64 * r: 64 * r + 64]
        gk, gv, gl = dev_bf16(pk), dev_bf16(pv), dev_i32(fit)
        y2 = torch.empty_like(x)
        ph.photon_encoder_step(c.h, layer, sc, x, ph.make_kv(gk, gv, gl, page_table=dev_i32(ids)), y2, scale=scale)
        assert c.status() == 0
        assert np.array_equal(gl.cpu().numpy(), fit + 1) and np.array_equal(host_bits(y2), host_bits(y1))
        hk, hv, fk, fv = host_bits(gk), host_bits(gv), host_bits(ck), host_bits(cv)
        for u in range(cfg.B):
            for r in range(2):
                assert np.array_equal(hk[ids[u, r]], fk[u, :, 64 * r: 64 * r + 64])
                assert np.array_equal(hv[ids[u, r]], fv[u, :, 64 * r: 64 * r + 64])


def test_encoder_step_refuses_bad_arguments():
    cfg = cfg_small(0, B=2, S=8)
    with Ctx(cfg) as c:
        co = wl.coarse_inputs(cfg)
        kv = ph.make_kv(dev_bf16(co["k"]), dev_bf16(co["v"]), dev_i32(co["len"]))
        lw = wl.encoder_layer_inputs(cfg, F=64)
        W = {n: dev_bf16(lw[n]) for n in ("g1", "wqkv", "wo", "g2", "wgu", "wdown")}
        sc = ph.make_layer_scratch(2, cfg.Hq, cfg.Hkv, cfg.dh, 64, "cuda", torch.bfloat16)
        x = dev_bf16(lw["x"])
        n0 = ph.photon_launch_count(c.h)
        for bad in (dict(F=60), dict(theta=1.0), dict(eps=-1.0)):
            kw = dict(F=64, eps=1e-5, theta=10000.0)
            kw.update(bad)
            layer = ph.make_layer(W["g1"], W["wqkv"], W["wo"], W["g2"], W["wgu"], W["wdown"], ph.PHOTON_W_IN_MAJOR, **kw)
            with pytest.raises(ph.PhotonError) as e:
                ph.photon_encoder_step(c.h, layer, sc, x, kv, x)
            assert e.value.code == ph.PHOTON_ERR_INVALID_ARG
        layer = ph.make_layer(W["g1"], None, W["wo"], W["g2"], W["wgu"], W["wdown"], ph.PHOTON_W_IN_MAJOR, 64)
        with pytest.raises(ph.PhotonError):
            ph.photon_encoder_step(c.h, layer, sc, x, kv, x)
        assert ph.photon_launch_count(c.h) == n0 and c.status() == 0
