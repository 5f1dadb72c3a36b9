"""Pins for the oracle's element-wise layer steps (rotary encoding with the split
of the fused projection, gated activation) and for the composed encoder step:
torch in fp64, closed forms, invariants.  No GPU."""
import math

import numpy as np
import torch

from paper_2512_20687_b200 import workloads as wl


def bf(x):
    return wl.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def rnd(seed, name, shape, std=1.0):
    return wl.normal_bf16(seed, name, shape, std)


def f64(b):
    return wl.bf16_bits_to_f64(b)


def _torch_rope(x, pos, theta):
    """The rotate-half formulation of the LLaMA reference code, in fp64: x [n, H, dh]."""
    dh = x.shape[-1]
    inv = theta ** (-torch.arange(0, dh, 2, dtype=torch.float64) / dh)
    ang = pos[:, None].double() * inv[None, :]
    cos, sin = torch.cat([ang.cos(), ang.cos()], -1)[:, None, :], torch.cat([ang.sin(), ang.sin()], -1)[:, None, :]
    rot = torch.cat([-x[..., dh // 2:], x[..., : dh // 2]], -1)
    return x * cos + rot * sin


def test_rope_split_against_rotate_half_in_torch(oracle):
    n, Hq, Hkv, dh = 5, 4, 2, 16
    qkv = rnd(31, "qkv", (n, (Hq + 2 * Hkv) * dh))
    pos = np.array([0, 1, 7, 500, 8191], np.int32)
    q, k, v = oracle.rope_split(qkv, pos, Hq, Hkv, dh, 10000.0)
    X = torch.from_numpy(f64(qkv))
    tq = X[:, : Hq * dh].reshape(n, Hq, dh)
    tk = X[:, Hq * dh: (Hq + Hkv) * dh].reshape(n, Hkv, dh)
    tp = torch.from_numpy(pos)
    np.testing.assert_allclose(q, _torch_rope(tq, tp, 10000.0).numpy(), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(k, _torch_rope(tk, tp, 10000.0).numpy(), rtol=1e-12, atol=1e-12)
    assert np.array_equal(v.reshape(n, -1), f64(qkv)[:, (Hq + Hkv) * dh:])       # v: a copy
    assert np.array_equal(q[0], tq[0].numpy()) and np.array_equal(k[0], tk[0].numpy())   # position 0: identity


def test_rope_closed_forms_and_relative_positions(oracle):
    dh = 8
    # feature pair (0, 4) has frequency 1: position 1 rotates (1, 0) to (cos 1, sin 1)
    x = np.zeros((1, 3 * dh), np.float32)
    x[0, 0] = 1.0
    q, _, _ = oracle.rope_split(bf(x), np.array([1], np.int32), 1, 1, dh, 10000.0)
    assert abs(q[0, 0, 0] - math.cos(1.0)) < 1e-15 and abs(q[0, 0, 4] - math.sin(1.0)) < 1e-15
    # lengths are preserved, and <rope(q, m), rope(k, n)> depends on m - n only
    qkv = rnd(32, "qkv", (4, 3 * dh))
    qkv[1:] = qkv[0]
    pos = np.array([3, 10, 100, 107], np.int32)
    q, k, _ = oracle.rope_split(qkv, pos, 1, 1, dh, 10000.0)
    X = f64(qkv)
    np.testing.assert_allclose((q ** 2).sum(-1)[:, 0], (X[:, :dh] ** 2).sum(-1), rtol=1e-13)
    d1 = q[1, 0] @ k[0, 0]          # 10 - 3
    d2 = q[3, 0] @ k[2, 0]          # 107 - 100
    assert abs(d1 - d2) < 1e-12


def test_swiglu_against_torch(oracle):
    gu = rnd(33, "gu", (6, 40), std=2.0)
    got = oracle.swiglu(gu)
    G = torch.from_numpy(f64(gu))
    want = torch.nn.functional.silu(G[:, :20]) * G[:, 20:]
    np.testing.assert_allclose(got, want.numpy(), rtol=1e-13, atol=1e-14)
    z = np.zeros((1, 4), np.float32)
    z[0, 2:] = 5.0
    assert not oracle.swiglu(bf(z)).any()                                        # silu(0) = 0
    big = np.array([[40.0, -40.0, 3.0, 3.0]], np.float32)
    np.testing.assert_allclose(oracle.swiglu(bf(big))[0], [120.0, -120.0 * math.exp(-40.0)], rtol=1e-12)


def test_decoder_prefill_against_torch_causal_attention(oracle):
    """The prefix pass: the P rows of every chunk attend causally among themselves at
    positions 0..P-1; torch's is_causal attention on the oracle's rotated q, k and v,
    and the chunk buffers afterwards."""
    cfg = wl.scaled(wl.CONFIGS[0], B=3, D=256, chunks_per_seq=2)              # P = 4, cap = 8
    lw = wl.encoder_layer_inputs(wl.scaled(cfg, B=cfg.Nc * cfg.P), F=128)
    n, P, D, Hq, Hkv, dh = cfg.Nc, cfg.P, cfg.D, cfg.Hq, cfg.Hkv, cfg.dh
    U = lw["x"].reshape(n, P, D)
    cap = cfg.P + cfg.C
    chunks = {"k": np.full((n + 2, Hkv, cap, dh), 0x7FC1, np.uint16), "v": np.full((n + 2, Hkv, cap, dh), 0x7FC1, np.uint16),
              "len": np.zeros(n + 2, np.int32)}
    ids = np.array([5, 0, 7, 2, 3, 1], np.int32)
    scale = dh ** -0.5
    r = oracle.decoder_prefill(U, lw, chunks, scale, unit_ids=ids)
    assert r["flags"] == 0
    assert list(chunks["len"]) == [P, P, P, P, 0, P, 0, P]
    T = lambda b: torch.from_numpy(f64(b))
    for i, u in enumerate(ids):
        assert np.array_equal(chunks["k"][u, :, :P], r["k_new"].reshape(n, P, Hkv, dh)[i].transpose(1, 0, 2))
        assert np.all(chunks["k"][u, :, P:] == 0x7FC1)
    q = T(r["q"]).reshape(n, P, Hq, dh).permute(0, 2, 1, 3)
    k = T(r["k_new"]).reshape(n, P, Hkv, dh).permute(0, 2, 1, 3).repeat_interleave(Hq // Hkv, dim=1)
    v = T(r["v_new"]).reshape(n, P, Hkv, dh).permute(0, 2, 1, 3).repeat_interleave(Hq // Hkv, dim=1)
    att = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True, scale=scale)
    np.testing.assert_allclose(f64(r["att"]).reshape(n, P, Hq, dh), att.permute(0, 2, 1, 3).numpy(), rtol=2 ** -8, atol=1e-6)
    # positions: row r of every chunk is rotated by r; row 0 is not rotated at all
    X = T(r["qkv"]).reshape(n, P, -1)
    assert np.array_equal(f64(r["q"]).reshape(n, P, Hq * dh)[:, 0], X[:, 0, : Hq * dh].numpy())
    y = T(r["act"]) @ T(lw["wdown"]) + T(r["h"])
    np.testing.assert_allclose(r["y"].reshape(n * P, D), y.numpy(), rtol=1e-11, atol=1e-12)


def test_encoder_step_against_a_torch_llama_layer(oracle):
    """One layer, written with torch's own rms_norm / linear / silu / softmax in fp64
    on the oracle's bf16 intermediates where the chain is rounded, otherwise
    independent of the oracle's code."""
    cfg = wl.scaled(wl.CONFIGS[0], B=3, S=9, D=256)       # Hq 4, Hkv 2, dh 64
    lw = wl.encoder_layer_inputs(cfg, F=128)
    co = wl.coarse_inputs(cfg)
    co["len"] = np.array([8, 3, 0], np.int32)
    cache = {"k": co["k"].copy(), "v": co["v"].copy(), "len": co["len"].copy()}
    scale = cfg.dh ** -0.5
    r = oracle.encoder_step(lw["x"], lw, cache, scale)
    assert r["flags"] == 0 and np.array_equal(cache["len"], co["len"] + 1)
    T = lambda b: torch.from_numpy(f64(b))
    B, D, Hq, Hkv, dh = cfg.B, cfg.D, cfg.Hq, cfg.Hkv, cfg.dh
    x = T(lw["x"])
    n1 = torch.nn.functional.rms_norm(x, (D,), T(lw["g1"]), eps=1e-5)
    np.testing.assert_allclose(f64(r["n1"]), n1.numpy(), rtol=2 ** -8)
    qkv = T(r["n1"]) @ T(lw["wqkv"])
    np.testing.assert_allclose(f64(r["qkv"]), qkv.numpy(), rtol=2 ** -8, atol=1e-6)
    # the appended rows are the rotated key and the value of this step
    for b in range(B):
        at = co["len"][b]
        assert np.array_equal(cache["k"][b, :, at], r["k_new"][b]) and np.array_equal(cache["v"][b, :, at], r["v_new"][b])
    q = T(r["q"]).unsqueeze(2)                                                   # [B, Hq, 1, dh]
    kk = T(cache["k"]).repeat_interleave(Hq // Hkv, dim=1)
    vv = T(cache["v"]).repeat_interleave(Hq // Hkv, dim=1)
    mask = (torch.arange(cache["k"].shape[2])[None, :] < torch.from_numpy(cache["len"])[:, None])[:, None, None, :]
    att = torch.nn.functional.scaled_dot_product_attention(q, kk, vv, attn_mask=mask, scale=scale).squeeze(2)
    np.testing.assert_allclose(f64(r["att"]), att.reshape(B, -1).numpy(), rtol=2 ** -8, atol=1e-6)
    h = T(r["att"]) @ T(lw["wo"]) + x
    np.testing.assert_allclose(f64(r["h"]), h.numpy(), rtol=2 ** -8, atol=1e-6)
    n2 = torch.nn.functional.rms_norm(T(r["h"]), (D,), T(lw["g2"]), eps=1e-5)
    gu = T(wl.f32_to_bf16_bits(n2.numpy().astype(np.float32))) @ T(lw["wgu"])
    np.testing.assert_allclose(f64(r["gu"]), gu.numpy(), rtol=2 ** -7, atol=1e-2)
    G = T(r["gu"])
    act = torch.nn.functional.silu(G[:, : lw["F"]]) * G[:, lw["F"]:]
    np.testing.assert_allclose(f64(r["act"]), act.numpy(), rtol=2 ** -8, atol=1e-6)
    y = T(r["act"]) @ T(lw["wdown"]) + T(r["h"])
    np.testing.assert_allclose(r["y"], y.numpy(), rtol=1e-11, atol=1e-12)
