"""Pins for the oracle's whole-chunk causal attention (the local decoder at
many positions of a chunk at once): a hand-worked example, an explicit
{0, -inf} mask matrix in numpy, torch's causal attention in fp64, closed forms,
brute force in pure Python, and the causality invariants.  No GPU."""
import math
import os

import numpy as np
import pytest
import torch

from paper_2512_20687_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "causal_chunk_worked_example.txt")


def bf(x):
    return wl.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def rnd(seed, name, shape, std=1.0):
    return wl.normal_bf16(seed, name, shape, std)


def f64(b):
    return wl.bf16_bits_to_f64(b)


def _golden():
    g = {}
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, _, rest = line.partition(" ")
        if key == "scale_ln":
            g["scale"] = math.log(float(rest))
        else:
            g[key] = np.array([[float(t) for t in row.split()] for row in rest.split(";")])
    return g


@pytest.mark.parametrize("row0,valid", [(0, 3), (1, 3), (2, 3), (0, 2), (0, 0)])
def test_hand_worked_chunk(oracle, row0, valid):
    """The three-position example of tests/golden, asked for as a whole, from a
    later first row, and with the last position(s) not yet present."""
    g = _golden()
    n, dh = g["K"].shape
    R = n - row0
    q = bf(g["Q"][row0:]).reshape(1, R, 1, dh)
    k, v = bf(g["K"]).reshape(1, 1, n, dh), bf(g["V"]).reshape(1, 1, n, dh)
    out = oracle.chunk_causal_attention(q, k, v, np.array([valid], np.int32), g["scale"], row0=row0)
    want = g["OUT"][row0:].copy()
    want[max(0, valid - row0):] = 0.0                 # positions that do not exist yet
    np.testing.assert_allclose(out[0, :, 0], want, rtol=0, atol=1e-13)


def _case(seed, n=5, Hq=4, Hkv=2, dh=16, cap=11, R=None, lens=None):
    R = cap if R is None else R
    q = rnd(seed, "q", (n, R, Hq, dh))
    k = rnd(seed, "k", (n, Hkv, cap, dh))
    v = rnd(seed, "v", (n, Hkv, cap, dh))
    lens = np.array([cap, 1, cap - 1, 4, 7][:n] if lens is None else lens, np.int32)
    return q, k, v, lens


@pytest.mark.parametrize("row0,R", [(0, 11), (3, 8), (3, 4), (10, 1)])
def test_explicit_mask_matrix(oracle, row0, R):
    """Dense softmax under the {0, -inf} mask written out as a matrix: entry
    (t, i) is 0 iff i <= row0 + t, exactly the mask below Eq. 7 restricted to the
    rows asked for.  Positions beyond the chunk's length give zero rows."""
    q, k, v, lens = _case(11, R=R)
    n, _, Hq, dh = q.shape
    Hkv, cap = k.shape[1], k.shape[2]
    scale = dh ** -0.5
    out = oracle.chunk_causal_attention(q, k, v, lens, scale, row0=row0)
    G = Hq // Hkv
    mask = np.where(np.arange(cap)[None, :] <= (row0 + np.arange(R))[:, None], 0.0, -np.inf)
    for c in range(n):
        for hq in range(Hq):
            logits = scale * f64(q[c, :, hq]) @ f64(k[c, hq // G]).T + mask
            w = np.exp(logits - logits.max(axis=1, keepdims=True))
            w /= w.sum(axis=1, keepdims=True)
            want = w @ f64(v[c, hq // G])
            want[(row0 + np.arange(R)) >= lens[c]] = 0.0
            np.testing.assert_allclose(out[c, :, hq], want, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("Hq,Hkv,dh,cap", [(4, 2, 64, 24), (8, 8, 128, 24), (16, 4, 128, 8), (3, 1, 16, 64)])
def test_against_torch_causal_sdpa_fp64(oracle, Hq, Hkv, dh, cap):
    """Full chunks (every position present, all rows asked for) against torch's
    scaled_dot_product_attention with is_causal=True in fp64."""
    n = 3
    q, k, v, _ = _case(12, n=n, Hq=Hq, Hkv=Hkv, dh=dh, cap=cap, lens=[cap] * n)
    scale = dh ** -0.5
    out = oracle.chunk_causal_attention(q, k, v, np.full(n, cap, np.int32), scale)
    G = Hq // Hkv
    tq = torch.from_numpy(f64(q)).permute(0, 2, 1, 3)                           # [n, Hq, cap, dh]
    tk = torch.from_numpy(f64(k)).repeat_interleave(G, dim=1)
    tv = torch.from_numpy(f64(v)).repeat_interleave(G, dim=1)
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=scale)
    np.testing.assert_allclose(out, want.permute(0, 2, 1, 3).numpy(), rtol=1e-11, atol=1e-12)


def test_brute_force_in_pure_python(oracle):
    q, k, v, lens = _case(13, n=2, Hq=2, Hkv=1, dh=4, cap=5, lens=[5, 3])
    scale = 0.37
    out = oracle.chunk_causal_attention(q, k, v, lens, scale)
    Q, K, V = f64(q), f64(k), f64(v)
    for c in range(2):
        for t in range(5):
            for h in range(2):
                if t >= lens[c]:
                    assert not out[c, t, h].any()
                    continue
                s = [scale * sum(Q[c, t, h, d] * K[c, 0, i, d] for d in range(4)) for i in range(t + 1)]
                z = sum(math.exp(x) for x in s)
                for d in range(4):
                    want = sum(math.exp(s[i]) / z * V[c, 0, i, d] for i in range(t + 1))
                    assert abs(out[c, t, h, d] - want) < 1e-13


def test_zero_queries_give_running_means_and_first_row_its_value(oracle):
    """q = 0: all weights equal, so position t returns the mean of V_0..V_t; and
    whatever q is, position 0 sees one key and returns V_0 exactly."""
    q, k, v, _ = _case(14, n=2, Hq=2, Hkv=2, dh=8, cap=9, lens=[9, 9])
    out = oracle.chunk_causal_attention(q, k, v, np.array([9, 9], np.int32), 0.5)
    for h in range(2):
        assert np.array_equal(out[:, 0, h], f64(v[:, h, 0]))
    out0 = oracle.chunk_causal_attention(np.zeros_like(q), k, v, np.array([9, 9], np.int32), 0.5)
    means = np.cumsum(f64(v), axis=2) / np.arange(1, 10)[None, None, :, None]    # [n, Hkv, cap, dh]
    np.testing.assert_allclose(out0, means.transpose(0, 2, 1, 3), rtol=1e-13, atol=1e-14)


def test_later_rows_never_reach_earlier_positions(oracle):
    """Causality: overwrite rows > t (NaN bit patterns included) and positions <= t
    keep bit-identical outputs; each position changes when its own key row does."""
    q, k, v, lens = _case(15, n=1, Hq=2, Hkv=1, dh=16, cap=10, lens=[10])
    base = oracle.chunk_causal_attention(q, k, v, lens, 0.25)
    for t in (0, 4, 8):
        k2, v2 = k.copy(), v.copy()
        k2[0, 0, t + 1:] = 0x7FC1
        v2[0, 0, t + 1:] = 0xFFFF
        got = oracle.chunk_causal_attention(q, k2, v2, lens, 0.25)
        assert np.array_equal(got[0, : t + 1], base[0, : t + 1])
        assert not np.isfinite(got[0, t + 1:]).any()
    v3 = v.copy()
    v3[0, 0, 5] = rnd(16, "v5", (16,))
    got = oracle.chunk_causal_attention(q, k, v3, lens, 0.25)
    assert np.array_equal(got[0, :5], base[0, :5])
    assert all(not np.array_equal(got[0, t], base[0, t]) for t in range(5, 10))


def test_last_position_equals_the_single_query_form(oracle):
    """The row at position len-1 is the decode step's bounded attention of the
    newest position (two entry points of the oracle that share only the inner
    softmax; both are pinned separately above and in the other pin file)."""
    q, k, v, lens = _case(17)
    n, R, Hq, dh = q.shape
    out = oracle.chunk_causal_attention(q, k, v, lens, 0.3)
    last = np.stack([q[c, lens[c] - 1] for c in range(n)])
    single, _ = oracle.chunk_attention(last, k, v, lens, 0.3)
    for c in range(n):
        np.testing.assert_allclose(out[c, lens[c] - 1], single[c], rtol=0, atol=0)


def test_slot_gather_and_bad_slots(oracle):
    q, k, v, lens = _case(18)
    slot = np.array([4, 0, 0, 7, -1], np.int32)
    out, flags = oracle.chunk_causal_attention(q, k, v, lens, 0.3, slot=slot, want_flags=True)
    assert flags == oracle.DEV_BAD_INDEX
    assert not out[3].any() and not out[4].any()
    direct = oracle.chunk_causal_attention(q[[0, 1, 2]], k[[4, 0, 0]], v[[4, 0, 0]], lens[[4, 0, 0]], 0.3)
    assert np.array_equal(out[:3], direct)
