"""Pins for the CPU oracle: each test checks it against something other than
itself - hand-worked values, library routines, closed forms, brute force on
tiny inputs, invariants.  No GPU."""
import math
import os

import numpy as np
import pytest
import scipy.special
import torch

from paper_2512_20687_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf(x):
    """float array -> bf16 bits (values must be representable or are rounded)."""
    return wl.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def rnd(seed, name, shape, std=1.0):
    return wl.normal_bf16(seed, name, shape, std)


def f64(b):
    return wl.bf16_bits_to_f64(b)


# ---------------------------------------------------------------- golden cases

def _parse_golden(path):
    cases, cur = [], None
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        key, _, rest = line.partition(" ")
        if key == "case":
            cur = {"name": rest}
            cases.append(cur)
        elif key in ("K", "V"):
            cur[key] = np.array([[float(t) for t in row.split()] for row in rest.split(";")])
        elif key in ("q", "out"):
            cur[key] = np.array([float(t) for t in rest.split()])
        elif key in ("scale_ln", "lse_ln"):
            cur[key] = math.log(float(rest))
    return cases


@pytest.mark.parametrize("case", _parse_golden(os.path.join(GOLDEN, "attention_worked_examples.txt")),
                         ids=lambda c: c["name"])
def test_hand_worked_examples(oracle, case):
    K, V, q = case["K"], case["V"], case["q"]
    n, dh = K.shape
    k = bf(K).reshape(1, 1, n, dh)
    v = bf(V).reshape(1, 1, n, dh)
    out, lse = oracle.attention(bf(q).reshape(1, 1, dh), k, v, np.array([n], np.int32),
                                case["scale_ln"])
    np.testing.assert_allclose(out[0, 0], case["out"], rtol=0, atol=1e-13)
    assert abs(lse[0, 0] - case["lse_ln"]) < 1e-13


# ---------------------------------------------------------------- library routines

def test_one_hot_values_return_library_softmax(oracle):
    """V = identity rows makes the output equal to the attention weights;
    they must match scipy's softmax of the logits, sum to 1, and the lse must
    match scipy's logsumexp."""
    n, dh = 24, 32
    q = rnd(11, "q", (1, 1, dh))
    k = rnd(11, "k", (1, 1, n, dh))
    v = bf(np.eye(n, dh)).reshape(1, 1, n, dh)
    scale = dh ** -0.5
    out, lse = oracle.attention(q, k, v, np.array([n], np.int32), scale)
    logits = scale * (f64(k[0, 0]) @ f64(q[0, 0]))
    want = scipy.special.softmax(logits)
    np.testing.assert_allclose(out[0, 0, :n], want, rtol=1e-13, atol=1e-15)
    assert abs(out[0, 0].sum() - 1.0) < 1e-12
    assert abs(lse[0, 0] - scipy.special.logsumexp(logits)) < 1e-12


@pytest.mark.parametrize("Hq,Hkv,dh", [(4, 2, 64), (16, 4, 128), (8, 8, 128), (6, 2, 16)])
def test_against_torch_sdpa_fp64(oracle, Hq, Hkv, dh):
    """Grouped-query attention with ragged lengths against torch's
    scaled_dot_product_attention in fp64 (KV heads repeated contiguously, which
    is how the library defines grouped heads)."""
    n_units, cap = 5, 37
    lens = np.array([37, 1, 20, 36, 7], np.int32)
    q = rnd(5, "q", (n_units, Hq, dh))
    k = rnd(5, "k", (n_units, Hkv, cap, dh))
    v = rnd(5, "v", (n_units, Hkv, cap, dh))
    scale = dh ** -0.5
    out, lse = oracle.attention(q, k, v, lens, scale)
    G = Hq // Hkv
    tq = torch.from_numpy(f64(q)).unsqueeze(2)                                   # [n, Hq, 1, dh]
    tk = torch.from_numpy(f64(k)).repeat_interleave(G, dim=1)
    tv = torch.from_numpy(f64(v)).repeat_interleave(G, dim=1)
    mask = (torch.arange(cap)[None, :] < torch.from_numpy(lens)[:, None])[:, None, None, :]
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=mask, scale=scale)
    np.testing.assert_allclose(out, want.squeeze(2).numpy(), rtol=1e-11, atol=1e-12)
    logits = scale * torch.einsum("nhd,nhkd->nhk", tq.squeeze(2), tk)
    logits = logits.masked_fill(~mask.squeeze(2), -math.inf)
    np.testing.assert_allclose(lse, torch.logsumexp(logits, -1).numpy(), rtol=1e-12, atol=1e-12)


def test_group_mapping_is_contiguous(oracle):
    """Hq=4, Hkv=2: heads 0,1 read KV head 0 and heads 2,3 read KV head 1."""
    dh, n = 8, 3
    k = rnd(1, "k", (1, 2, n, dh))
    v = np.empty((1, 2, n, dh), np.uint16)
    v[0, 0], v[0, 1] = bf(np.full((n, dh), 1.0)), bf(np.full((n, dh), 2.0))
    out, _ = oracle.attention(rnd(1, "q", (1, 4, dh)), k, v, np.array([n], np.int32), 0.3)
    np.testing.assert_allclose(out[0, :, 0], [1, 1, 2, 2], atol=1e-14)


# ---------------------------------------------------------------- bounded == full masked

def test_bounded_attention_equals_full_masked_attention(oracle):
    """Concatenate every chunk's rows into one long sequence and compute dense
    softmax attention under the explicit {0, -inf} mask that lets each query see
    only the first len_c rows of its own chunk (the mask below Eq. 7).  The
    result must equal the chunk-local form."""
    Nc, Hq, Hkv, dh, P, C = 6, 4, 2, 16, 3, 5
    cap = P + C
    lens = np.array([P, P + 1, P + C, P + 2, P + C - 1, P + 3], np.int32)
    q = rnd(2, "q", (Nc, Hq, dh))
    kc = rnd(2, "kc", (Nc, Hkv, cap, dh))
    vc = rnd(2, "vc", (Nc, Hkv, cap, dh))
    scale = dh ** -0.5
    out, _ = oracle.chunk_attention(q, kc, vc, lens, scale)
    G = Hq // Hkv
    for hq in range(Hq):
        kvh = hq // G
        Kall = f64(kc[:, kvh]).reshape(Nc * cap, dh)        # the one long sequence
        Vall = f64(vc[:, kvh]).reshape(Nc * cap, dh)
        mask = np.full((Nc, Nc * cap), -np.inf)
        for c in range(Nc):
            mask[c, c * cap: c * cap + lens[c]] = 0.0
        logits = scale * (f64(q[:, hq]) @ Kall.T) + mask
        w = np.exp(logits - logits.max(axis=1, keepdims=True))
        w /= w.sum(axis=1, keepdims=True)
        np.testing.assert_allclose(out[:, hq], w @ Vall, rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------- closed forms

def test_single_key_returns_its_value_exactly(oracle):
    dh = 64
    k = rnd(3, "k", (1, 1, 4, dh))
    v = rnd(3, "v", (1, 1, 4, dh))
    out, lse = oracle.attention(rnd(3, "q", (1, 2, dh)), k, v, np.array([1], np.int32), 0.125)
    assert np.array_equal(out[0, 0], f64(v[0, 0, 0])) and np.array_equal(out[0, 1], f64(v[0, 0, 0]))


def test_zero_query_and_equal_keys_give_the_mean_of_values(oracle):
    dh, n = 32, 9
    v = rnd(4, "v", (1, 1, n, dh))
    k = rnd(4, "k", (1, 1, n, dh))
    lens = np.array([n - 2], np.int32)
    mean = f64(v[0, 0, : n - 2]).mean(axis=0)
    out, lse = oracle.attention(np.zeros((1, 1, dh), np.uint16), k, v, lens, 0.7)
    np.testing.assert_allclose(out[0, 0], mean, rtol=1e-13, atol=1e-14)
    assert abs(lse[0, 0] - math.log(n - 2)) < 1e-13
    k_same = np.broadcast_to(k[:, :, :1], k.shape).copy()
    out2, _ = oracle.attention(rnd(4, "q", (1, 1, dh)), k_same, v, lens, 0.7)
    np.testing.assert_allclose(out2[0, 0], mean, rtol=1e-13, atol=1e-14)


def test_equal_values_are_returned(oracle):
    dh, n = 16, 7
    v = np.broadcast_to(rnd(6, "v", (1, 1, 1, dh)), (1, 1, n, dh)).copy()
    out, _ = oracle.attention(rnd(6, "q", (1, 1, dh)), rnd(6, "k", (1, 1, n, dh)), v,
                              np.array([n], np.int32), 1.0)
    np.testing.assert_allclose(out[0, 0], f64(v[0, 0, 0]), rtol=1e-14)


def test_huge_logits_do_not_overflow(oracle):
    """scale 1e4 puts logits near +-1e5: the result must be the value row of
    the largest logit, finite."""
    dh, n = 8, 5
    q, k, v = rnd(7, "q", (1, 1, dh)), rnd(7, "k", (1, 1, n, dh)), rnd(7, "v", (1, 1, n, dh))
    out, lse = oracle.attention(q, k, v, np.array([n], np.int32), 1e4)
    best = int(np.argmax(f64(k[0, 0]) @ f64(q[0, 0])))
    np.testing.assert_allclose(out[0, 0], f64(v[0, 0, best]), rtol=1e-12)
    assert np.isfinite(lse).all()


def test_empty_cache_gives_zero_row_and_minus_inf(oracle):
    dh = 8
    out, lse = oracle.attention(rnd(8, "q", (2, 1, dh)), rnd(8, "k", (2, 1, 3, dh)),
                                rnd(8, "v", (2, 1, 3, dh)), np.array([0, 2], np.int32), 1.0)
    assert np.all(out[0] == 0) and lse[0, 0] == -np.inf and np.isfinite(lse[1, 0])


# ---------------------------------------------------------------- invariants

def _chunk_case(seed=9, poison=False):
    cfg = wl.scaled(wl.CONFIGS[0], B=3, chunks_per_seq=4, seed=seed)
    return cfg, wl.chunk_inputs(cfg, poison=poison)


def test_rows_past_len_and_other_chunks_never_matter(oracle):
    cfg, a = _chunk_case(poison=False)
    _, b = _chunk_case(poison=True)                  # NaN patterns in every masked row
    scale = cfg.dh ** -0.5
    oa, _ = oracle.chunk_attention(a["q"], a["kc"], a["vc"], a["len"], scale)
    ob, _ = oracle.chunk_attention(b["q"], b["kc"], b["vc"], b["len"], scale)
    assert np.array_equal(oa, ob) and np.isfinite(ob).all()
    # overwrite every chunk but #5 with other data: chunk 5's rows stay bit-identical
    c = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in a.items()}
    other = np.arange(cfg.Nc) != 5
    c["kc"][other] = rnd(99, "x", c["kc"][other].shape)
    c["vc"][other] = rnd(98, "x", c["vc"][other].shape)
    c["q"][other] = rnd(97, "x", c["q"][other].shape)
    oc, _ = oracle.chunk_attention(c["q"], c["kc"], c["vc"], c["len"], scale)
    assert np.array_equal(oc[5], oa[5]) and not np.array_equal(oc[4], oa[4])


def test_batch_permutation_equivariance(oracle):
    cfg, a = _chunk_case()
    scale = cfg.dh ** -0.5
    oa, _ = oracle.chunk_attention(a["q"], a["kc"], a["vc"], a["len"], scale)
    perm = np.random.default_rng(0).permutation(cfg.Nc)
    ob, _ = oracle.chunk_attention(a["q"][perm], a["kc"][perm], a["vc"][perm], a["len"][perm], scale)
    assert np.array_equal(ob, oa[perm])
    # the same through the gather index instead of moving data
    oc, _ = oracle.chunk_attention(a["q"][perm], a["kc"], a["vc"], a["len"], scale,
                                   slot=perm.astype(np.int32))
    assert np.array_equal(oc, oa[perm])


def test_key_permutation_invariance(oracle):
    dh, n = 64, 33
    q, k, v = rnd(12, "q", (1, 1, dh)), rnd(12, "k", (1, 1, n, dh)), rnd(12, "v", (1, 1, n, dh))
    lens = np.array([n], np.int32)
    o1, l1 = oracle.attention(q, k, v, lens, 0.125)
    perm = np.random.default_rng(1).permutation(n)
    o2, l2 = oracle.attention(q, k[:, :, perm].copy(), v[:, :, perm].copy(), lens, 0.125)
    np.testing.assert_allclose(o1, o2, rtol=1e-12, atol=1e-14)
    assert abs(l1[0, 0] - l2[0, 0]) < 1e-12


@pytest.mark.parametrize("cuts", [[0, 50], [0, 17, 50], [0, 0, 1, 1, 30, 50, 50], [0, 49, 50],
                                   list(range(0, 51, 5))])
def test_split_then_lse_merge_equals_single_pass(oracle, cuts):
    dh, n = 64, 50
    q, k, v = rnd(13, "q", (dh,)), rnd(13, "k", (n, dh)), rnd(13, "v", (n, dh))
    full_o, full_lse = oracle.attn_range(q, k, v, 0, n, 0.125)
    parts = [oracle.attn_range(q, k, v, a, b, 0.125) for a, b in zip(cuts[:-1], cuts[1:])]
    o, lse = oracle.lse_merge(np.stack([p[0] for p in parts]), np.array([p[1] for p in parts]))
    np.testing.assert_allclose(o, full_o, rtol=1e-12, atol=1e-14)
    assert abs(lse - full_lse) < 1e-12
    # and the range form agrees with the batched entry point
    bo, bl = oracle.attention(q.reshape(1, 1, dh), k.reshape(1, 1, n, dh), v.reshape(1, 1, n, dh),
                              np.array([n], np.int32), 0.125)
    assert np.array_equal(bo[0, 0], full_o) and bl[0, 0] == full_lse


def test_lse_merge_matches_direct_formula_on_given_parts():
    """Two parts with known weights: lse = ln 1 and ln 3 -> weights 1/4, 3/4."""
    from oracle import photon_oracle as orc
    o, lse = orc.lse_merge(np.array([[4.0, 0.0], [0.0, 4.0]]), np.array([0.0, math.log(3.0)]))
    np.testing.assert_allclose(o, [1.0, 3.0], rtol=1e-14)
    assert abs(lse - math.log(4.0)) < 1e-14
    o, lse = orc.lse_merge(np.array([[1.0, 2.0], [5.0, 5.0]]), np.array([-np.inf, 0.5]))
    np.testing.assert_allclose(o, [5.0, 5.0]) and lse == 0.5


def test_shared_prefix_equals_physically_copied_prefix(oracle):
    Hq, Hkv, dh = 4, 2, 32
    n_units, cap, cap_sh = 5, 6, 11
    lens = np.array([6, 0, 3, 1, 5], np.int32)
    sh_len = np.array([11, 4], np.int32)
    sh_id = np.array([0, 1, -1, 0, 1], np.int32)
    q = rnd(14, "q", (n_units, Hq, dh))
    k, v = rnd(14, "k", (n_units, Hkv, cap, dh)), rnd(14, "v", (n_units, Hkv, cap, dh))
    ks, vs = rnd(14, "ks", (2, Hkv, cap_sh, dh)), rnd(14, "vs", (2, Hkv, cap_sh, dh))
    out, lse = oracle.attention(q, k, v, lens, 0.2,
                                shared={"k": ks, "v": vs, "len": sh_len, "id": sh_id})
    big = cap + cap_sh
    kk = np.zeros((n_units, Hkv, big, dh), np.uint16)
    vv = np.zeros_like(kk)
    ll = np.zeros(n_units, np.int32)
    for u in range(n_units):
        s = sh_id[u]
        pre = sh_len[s] if s >= 0 else 0
        if s >= 0:
            kk[u, :, :pre], vv[u, :, :pre] = ks[s, :, :pre], vs[s, :, :pre]
        kk[u, :, pre:pre + lens[u]], vv[u, :, pre:pre + lens[u]] = k[u, :, :lens[u]], v[u, :, :lens[u]]
        ll[u] = pre + lens[u]
    out2, lse2 = oracle.attention(q, kk, vv, ll, 0.2)
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)


def test_bad_indices_are_flagged_and_zeroed(oracle):
    dh = 8
    q, k, v = rnd(15, "q", (3, 1, dh)), rnd(15, "k", (2, 1, 4, dh)), rnd(15, "v", (2, 1, 4, dh))
    out, lse, flags = oracle.attention(q, k, v, np.array([4, 4], np.int32), 1.0,
                                       slot=np.array([1, 7, 0], np.int32), want_flags=True)
    assert flags == oracle.DEV_BAD_INDEX and np.all(out[1] == 0) and lse[1, 0] == -np.inf
    assert np.isfinite(lse[0, 0]) and np.any(out[2] != 0)


# ---------------------------------------------------------------- converter

def test_converter_one_hot_returns_weight_row_bit_exactly(oracle):
    D, P = 16, 3
    c = wl.converter_inputs(wl.scaled(wl.CONFIGS[0], D=D, P=P, B=D))
    x = bf(np.eye(D))
    U = oracle.converter(x, c["w_in_major"])
    assert np.array_equal(U.reshape(D, P * D), f64(c["w_in_major"]))
    U2 = oracle.converter(x, c["w_out_major"], w_out_major=True)
    assert np.array_equal(U, U2)


def test_converter_identity_blocks_copy_the_input(oracle):
    D, P, B = 8, 4, 5
    w = bf(np.concatenate([np.eye(D) * (r + 1) for r in range(P)], axis=1))      # [D, P*D]
    x = rnd(16, "x", (B, D))
    U = oracle.converter(x, w)
    for r in range(P):
        assert np.array_equal(U[:, r], (r + 1) * f64(x))


@pytest.mark.parametrize("with_bias", [False, True])
def test_converter_matches_numpy_matmul(oracle, with_bias):
    cfg = wl.scaled(wl.CONFIGS[0], B=7, D=48, P=3)
    c = wl.converter_inputs(cfg, with_bias=with_bias)
    U = oracle.converter(c["x"], c["w_in_major"], c["bias"])
    want = f64(c["x"]) @ f64(c["w_in_major"])
    if with_bias:
        want = want + f64(c["bias"])[None, :]
    np.testing.assert_allclose(U.reshape(7, -1), want, rtol=1e-12, atol=1e-13)
    Ut = oracle.converter(c["x"], c["w_out_major"], c["bias"], w_out_major=True, n_threads=3)
    assert np.array_equal(U, Ut)
    # prefix r, feature j sits at column r*D + j
    assert U.shape == (7, 3, 48)
    np.testing.assert_allclose(U[2, 1, 5], want[2, 1 * 48 + 5], rtol=1e-12)


def test_converter_is_linear(oracle):
    D, P = 32, 2
    c = wl.converter_inputs(wl.scaled(wl.CONFIGS[0], B=2, D=D, P=P))
    x = c["x"]
    U = oracle.converter(x, c["w_in_major"])
    combo = bf(2.0 * f64(x[:1]) - 0.5 * f64(x[1:]))          # exact? only if representable:
    if np.array_equal(f64(combo), 2.0 * f64(x[:1]) - 0.5 * f64(x[1:])):
        Uc = oracle.converter(combo, c["w_in_major"])
        np.testing.assert_allclose(Uc[0], 2.0 * U[0] - 0.5 * U[1], rtol=1e-11, atol=1e-12)
    U2 = oracle.converter(bf(2.0 * f64(x)), c["w_in_major"])        # scaling by 2 is exact in bf16
    np.testing.assert_allclose(U2, 2.0 * U, rtol=1e-14)


# ---------------------------------------------------------------- append

def test_append_is_a_bit_copy_in_order_and_leaves_the_rest_untouched(oracle):
    n_units, Hkv, cap, dh = 3, 2, 5, 8
    sentinel = np.uint16(0xABCD)
    k = np.full((n_units, Hkv, cap, dh), sentinel)
    v = np.full((n_units, Hkv, cap, dh), sentinel)
    ln = np.zeros(n_units, np.int32)
    news = []
    for step in range(4):
        kn, vn = rnd(20 + step, "kn", (n_units, Hkv, dh)), rnd(20 + step, "vn", (n_units, Hkv, dh))
        kn[0, 0, 0] = 0x7FC1            # NaN payload bits must survive
        news.append((kn, vn))
        assert oracle.kv_append(k, v, ln, kn, vn) == 0
    assert np.array_equal(ln, [4, 4, 4])
    for step, (kn, vn) in enumerate(news):
        assert np.array_equal(k[:, :, step], kn) and np.array_equal(v[:, :, step], vn)
    assert np.all(k[:, :, 4] == sentinel) and np.all(v[:, :, 4] == sentinel)


def test_append_overflow_and_bad_index(oracle):
    n_units, Hkv, cap, dh = 3, 1, 2, 4
    k = np.zeros((n_units, Hkv, cap, dh), np.uint16)
    v = np.zeros_like(k)
    ln = np.array([2, 1, 0], np.int32)
    kn, vn = rnd(30, "kn", (3, Hkv, dh)), rnd(30, "vn", (3, Hkv, dh))
    flags = oracle.kv_append(k, v, ln, kn, vn)
    assert flags == oracle.DEV_CAPACITY
    assert np.array_equal(ln, [2, 2, 1]) and np.all(k[0] == 0)
    assert np.array_equal(k[1, 0, 1], kn[1, 0]) and np.array_equal(v[2, 0, 0], vn[2, 0])
    flags = oracle.kv_append(k, v, ln, kn[:2], vn[:2], unit_ids=np.array([2, 9], np.int32))
    assert flags == oracle.DEV_BAD_INDEX and np.array_equal(ln, [2, 2, 2])
    assert np.array_equal(k[2, 0, 1], kn[0, 0])


def test_append_installs_a_block_of_prefix_rows_by_unit_index(oracle):
    """n_rows = P rows at once into chosen chunk buffers (source [n, P, Hkv, dh])."""
    n_units, Hkv, cap, dh, P = 4, 2, 6, 8, 3
    k = np.zeros((n_units, Hkv, cap, dh), np.uint16)
    v = np.zeros_like(k)
    ln = np.zeros(n_units, np.int32)
    kn, vn = rnd(31, "kn", (2, P, Hkv, dh)), rnd(31, "vn", (2, P, Hkv, dh))
    ids = np.array([3, 1], np.int32)
    assert oracle.kv_append(k, v, ln, kn, vn, unit_ids=ids, n_rows=P) == 0
    assert np.array_equal(ln, [0, 3, 0, 3])
    for i, u in enumerate(ids):
        for r in range(P):
            for h in range(Hkv):
                assert np.array_equal(k[u, h, r], kn[i, r, h]) and np.array_equal(v[u, h, r], vn[i, r, h])
    assert np.all(k[0] == 0) and np.all(k[2] == 0) and np.all(k[:, :, P:] == 0)


# ---------------------------------------------------------------- rounding

def test_round_bf16_ties_and_library_agreement(oracle):
    # hand cases: 1 + 2^-8 is a tie -> even (1.0); 1 + 3*2^-8 is a tie -> 1 + 2^-6
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -30,
                  -(1.0 + 2.0 ** -8), 0.0, 3.3895313892515355e38, 3.4e38, 2.0 ** -133, 2.0 ** -134,
                  1.5 * 2.0 ** -133])
    got = oracle.round_bf16(x)
    want = np.array([0x3F80, 0x3F80, 0x3F82, 0x3F81, 0xBF80, 0x0000, 0x7F7F, 0x7F80, 0x0001, 0x0000,
                     0x0002], np.uint16)
    assert np.array_equal(got, want)
    # float32-exact random values: torch's float32 -> bf16 conversion is the library routine
    r = np.random.default_rng(3).standard_normal(20000).astype(np.float32)
    t = torch.from_numpy(r).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.round_bf16(r.astype(np.float64)), t)
    assert np.array_equal(oracle.widen_bf16(t), f64(t))


# ---------------------------------------------------------------- the step

def test_decode_step_order_append_then_attend_then_convert(oracle):
    """The step appends first, so the newest latent attends to itself (the cache
    grows from KV_{<=g-1} to KV_{<=g} before X_g is formed, Eq. 12), and the
    converter consumes the bf16-rounded attention output."""
    cfg = wl.CONFIGS[0]
    s = wl.step_inputs(cfg, poison=True)
    co, cv, ch = s["coarse"], s["converter"], s["chunks"]
    k0, len0 = co["k"].copy(), co["len"].copy()
    r = oracle.decode_step(co, cv, ch, cfg.dh ** -0.5, cfg.dh ** -0.5, chain=True)
    assert r["flags"] == 0 and np.array_equal(co["len"], len0 + 1)
    assert np.array_equal(co["k"][:, :, cfg.S - 1], co["k_new"])
    assert np.array_equal(co["k"][:, :, : cfg.S - 1], k0[:, :, : cfg.S - 1])
    # attention over exactly S rows, computed independently with torch in fp64
    G = cfg.Hq // cfg.Hkv
    tk = torch.from_numpy(f64(co["k"])).repeat_interleave(G, 1)
    tv = torch.from_numpy(f64(co["v"])).repeat_interleave(G, 1)
    want = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(f64(co["q"])).unsqueeze(2), tk, tv, scale=cfg.dh ** -0.5).squeeze(2).numpy()
    np.testing.assert_allclose(r["out"], want, rtol=1e-11, atol=1e-12)
    xb = torch.from_numpy(want.reshape(cfg.B, -1)).float().to(torch.bfloat16).double().numpy()
    np.testing.assert_allclose(r["U"].reshape(cfg.B, -1), xb @ f64(cv["w_in_major"]),
                               rtol=1e-9, atol=1e-9)
    assert r["U"].shape == (cfg.B, cfg.P, cfg.D) and r["chunk_out"].shape == (cfg.Nc, cfg.Hq, cfg.dh)
