"""Parity of the CUDA path (through the C boundary) with the CPU oracle on the
same seeded inputs.  Append and index work is bit-exact; bf16 outputs are held
to max abs error 2e-2 and mean abs error 2e-3 against the fp64 oracle."""
import numpy as np
import pytest
import torch

import paper_2512_20687_b200 as ph
from paper_2512_20687_b200 import workloads as wl

from gpu_util import (Ctx, assert_close, chunks_to_dev, coarse_to_dev, dev_bf16, dev_i32, host_bits,
                      host_f64, shared_of)

pytestmark = pytest.mark.gpu

NT = 16     # oracle threads


def cfg_small(i, **kw):
    return wl.scaled(wl.CONFIGS[i], **kw)


# ------------------------------------------------------------------ append

@pytest.mark.parametrize("idx", [0, 1, 4])
def test_append_is_bit_exact(oracle, idx):
    cfg = wl.CONFIGS[idx] if idx < 4 else cfg_small(4, B=64)
    co = wl.coarse_inputs(cfg, poison=True)
    with Ctx(cfg) as c:
        d = coarse_to_dev(co)
        ph.photon_kv_append(c.h, d["kv"], d["k_new"], d["v_new"])
        assert c.status() == 0
        flags = oracle.kv_append(co["k"], co["v"], co["len"], co["k_new"], co["v_new"])
        assert flags == 0
        assert np.array_equal(host_bits(d["k"]), co["k"])
        assert np.array_equal(host_bits(d["v"]), co["v"])
        assert np.array_equal(d["len"].cpu().numpy(), co["len"])


def test_append_by_unit_index_blocks_overflow_and_bad_ids(oracle):
    cfg = wl.CONFIGS[0]
    n_units, cap, P = 9, cfg.P + cfg.C, cfg.P
    k = wl.normal_bf16(7, "k", (n_units, cfg.Hkv, cap, cfg.dh))
    v = wl.normal_bf16(7, "v", (n_units, cfg.Hkv, cap, cfg.dh))
    ln = np.array([0, 0, 5, 0, 8, 2, 0, 0, 1], np.int32)
    ids = np.array([6, 2, 0, 4, 11, -1, 8], np.int32)        # 2 and 4 lack room; 11 and -1 are bad
    kn = wl.normal_bf16(7, "kn", (len(ids), P, cfg.Hkv, cfg.dh))
    vn = wl.normal_bf16(7, "vn", (len(ids), P, cfg.Hkv, cfg.dh))
    with Ctx(cfg) as c:
        dk, dv, dl = dev_bf16(k), dev_bf16(v), dev_i32(ln)
        kv = ph.make_kv(dk, dv, dl)
        ph.photon_kv_append(c.h, kv, dev_bf16(kn), dev_bf16(vn), unit_ids=dev_i32(ids), n_rows=P)
        bits = c.status()
        flags = oracle.kv_append(k, v, ln, kn, vn, unit_ids=ids, n_rows=P)
        assert bits == flags == (ph.PHOTON_DEV_CAPACITY | ph.PHOTON_DEV_BAD_INDEX)
        assert np.array_equal(host_bits(dk), k) and np.array_equal(host_bits(dv), v)
        assert np.array_equal(dl.cpu().numpy(), ln)
        assert c.status() == 0          # cleared by the previous read


# ------------------------------------------------------------------ coarse attention

def run_coarse(c, co, scale, appended=True, flat=False):
    d = coarse_to_dev(co)
    out = torch.empty_like(d["q"])
    lse = torch.empty(d["q"].shape[:2], dtype=torch.float32, device="cuda")
    (ph.photon_flat_attn if flat else ph.photon_coarse_attn)(c.h, d["kv"], d["q"], out, lse, scale)
    torch.cuda.synchronize()
    return host_f64(out), lse.cpu().numpy().astype(np.float64), host_bits(out)


@pytest.mark.parametrize("idx", [0, 1, 2, 3, 4])
def test_coarse_attention_matches_oracle_at_full_size(oracle, idx):
    cfg = wl.CONFIGS[idx]
    co = wl.coarse_inputs(cfg, poison=True)
    oracle.kv_append(co["k"], co["v"], co["len"], co["k_new"], co["v_new"])    # attend over S rows
    scale = cfg.dh ** -0.5
    want, want_lse = oracle.attention(co["q"], co["k"], co["v"], co["len"], scale,
                                      shared=shared_of(co), n_threads=NT)
    with Ctx(cfg) as c:
        got, lse, _ = run_coarse(c, co, scale)
        assert c.status() == 0
    assert_close(got, want, f"coarse cfg{idx}")
    assert np.abs(lse - want_lse).max() < 2e-3


def test_level1_cache_of_hierarchical_generation(oracle):
    """The cache hierarchical generation keeps one level below the top (context / C1
    rows per sequence: 2048 for the 1B-class workload) through the same attention call:
    the second global workload of the schedule comparison, at its full size."""
    rows = wl.global_caches(wl.CONFIGS[1], "hierarchical")[0]["rows"]
    assert rows == 2048
    cfg = cfg_small(1, S=rows)
    co = wl.coarse_inputs(cfg, poison=True)
    oracle.kv_append(co["k"], co["v"], co["len"], co["k_new"], co["v_new"])
    scale = cfg.dh ** -0.5
    want, want_lse = oracle.attention(co["q"], co["k"], co["v"], co["len"], scale, n_threads=NT)
    with Ctx(cfg) as c:
        got, lse, _ = run_coarse(c, co, scale)
        assert c.status() == 0
    assert_close(got, want, "level-1 cache")
    assert np.abs(lse - want_lse).max() < 2e-3


@pytest.mark.parametrize("n_ctas", [1, 2, 3, 7, 37, 101, 259, 296, 0])
def test_grid_size_and_cut_points_do_not_change_the_result(oracle, n_ctas):
    """Ragged lengths incl. 0 and 1; the grid size moves the points where caches
    are cut and merged (one CTA: no cut at all; many: most units cut, some CTAs idle)."""
    cfg = cfg_small(1, B=9, S=701)
    co = wl.coarse_inputs(cfg, poison=True)
    lens = np.array([700, 0, 1, 2, 127, 128, 129, 513, 699], np.int32)
    for u, n in enumerate(lens):
        co["k"][u, :, n:] = 0x7FC1
        co["v"][u, :, n:] = 0xFFC1
    co["len"] = lens
    scale = cfg.dh ** -0.5
    want, want_lse = oracle.attention(co["q"], co["k"], co["v"], lens, scale, n_threads=NT)
    with Ctx(cfg) as c:
        ph.photon_set_attention_ctas(c.h, n_ctas)
        got, lse, bits1 = run_coarse(c, co, scale)
        _, _, bits2 = run_coarse(c, co, scale)
        assert c.status() == 0
    assert np.array_equal(bits1, bits2)           # tickets are back at zero, merge order is fixed
    assert_close(got, want, f"ctas={n_ctas}")
    assert np.all(got[1] == 0) and np.all(np.isneginf(lse[1]))
    fin = np.isfinite(want_lse)
    assert np.abs(lse[fin] - want_lse[fin]).max() < 2e-3


@pytest.mark.parametrize("G,dh", [(1, 64), (2, 64), (8, 128), (16, 64), (16, 128)])
def test_coarse_attention_other_group_sizes(oracle, G, dh):
    Hkv = 2
    cfg = cfg_small(1, B=5, S=300, Hq=G * Hkv, Hkv=Hkv, dh=dh, D=G * Hkv * dh)
    co = wl.coarse_inputs(cfg, poison=True)
    co["len"] = np.array([299, 64, 65, 7, 200], np.int32)
    for u, n in enumerate(co["len"]):
        co["k"][u, :, n:] = 0x7FC1
        co["v"][u, :, n:] = 0x7FC1
    scale = cfg.dh ** -0.5
    want, want_lse = oracle.attention(co["q"], co["k"], co["v"], co["len"], scale, n_threads=NT)
    with Ctx(cfg) as c:
        got, lse, _ = run_coarse(c, co, scale)
        assert c.status() == 0
    assert_close(got, want, f"G={G} dh={dh}")
    assert np.abs(lse - want_lse).max() < 2e-3


# group sizes and head sizes the shared-prefix kernel accepts: a row tile of 128 query rows holds 128 / G units
# (126 of its rows are used for G = 3); the batch is never a whole number of tiles
# ... and own caches of at most 40 rows (a second kernel reads them) or at most 24 (they ride along in the first)
@pytest.mark.parametrize("S", [40, 24])
@pytest.mark.parametrize("max_splits", [1, 0])
@pytest.mark.parametrize("G,dh,B", [(4, 128, 37), (1, 64, 150), (2, 128, 75), (3, 64, 50), (8, 128, 21), (16, 64, 13)])
def test_shared_prefix_variants(oracle, G, dh, B, max_splits, S):
    """Two shared segments of different length, units without a prefix, empty own caches."""
    Hkv = 4 if G == 4 else 2
    cfg = cfg_small(3, B=B, S=S, shared_S=300, Hq=G * Hkv, Hkv=Hkv, dh=dh, D=G * Hkv * dh)
    co = wl.coarse_inputs(cfg, poison=True)
    ks = wl.normal_bf16(3, "ks2", (2, cfg.Hkv, 300, cfg.dh))
    vs = wl.normal_bf16(3, "vs2", (2, cfg.Hkv, 300, cfg.dh))
    sh_len = np.array([300, 77], np.int32)
    ks[1, :, 77:] = 0x7FC1
    vs[1, :, 77:] = 0x7FC1
    sh_id = (np.arange(cfg.B) % 3 - 1).astype(np.int32)       # -1, 0, 1, -1, ...
    lens = (np.arange(cfg.B) % 5 * (S // 4 - 1)).astype(np.int32)        # 0, 9, 18, 27, 36 of 40 rows; 0 .. 20 of 24
    for u, n in enumerate(lens):
        co["k"][u, :, n:] = 0x7FC1
        co["v"][u, :, n:] = 0x7FC1
    co.update(k_shared=ks, v_shared=vs, shared_len=sh_len, shared_id=sh_id, len=lens)
    scale = cfg.dh ** -0.5
    want, want_lse = oracle.attention(co["q"], co["k"], co["v"], lens, scale, shared=shared_of(co),
                                      n_threads=NT)
    with Ctx(cfg, max_splits=max_splits) as c:
        got, lse, _ = run_coarse(c, co, scale)
        assert c.status() == 0
    assert_close(got, want, f"shared prefix G={G} dh={dh} splits={max_splits} S={S}")
    empty = (lens == 0) & (sh_id < 0)
    assert empty.any() and np.all(got[empty] == 0) and np.all(np.isneginf(lse[empty]))
    fin = np.isfinite(want_lse)
    assert np.abs(lse[fin] - want_lse[fin]).max() < 2e-3


@pytest.mark.parametrize("folded", [False, True])
def test_attention_that_lined_up_behind_an_append_which_opens_new_tiles(oracle, folded):
    """The attention's CTAs start, and deal the tiles, while the kernels before it in the stream still run: a long
    read (the probe) holds the stream, the append behind it has not run yet, so the lengths the deal is made from are
    the old ones.  Units at 64 and 128 rows open a new tile with the append: after the dependency wait the deal is
    found stale, the loads that went out early are left to land and everything is dealt again.  The result must be
    what the oracle gives for the grown caches, and the same bits as a run with nothing in front of it.  folded: the
    same start behind a long read for the step's attention with the append folded in (its lengths do not change
    under it)."""
    cfg = cfg_small(1, B=21, S=400)
    s_in = wl.step_inputs(cfg, poison=True)
    co, cv, chk = s_in["coarse"], s_in["converter"], s_in["chunks"]
    lens = np.array([64, 128, 63, 0, 399, 192, 1, 127, 256, 320, 64, 64, 128, 5, 300, 191, 255, 64, 383, 128, 2], np.int32)
    co["k"] = wl.normal_bf16(11, "k", co["k"].shape)
    co["v"] = wl.normal_bf16(11, "v", co["v"].shape)
    for u, n in enumerate(lens):
        co["k"][u, :, n:] = 0x7FC1
        co["v"][u, :, n:] = 0xFFC1
    co["len"] = lens
    scale = cfg.dh ** -0.5
    held = torch.empty(192 << 20, dtype=torch.uint8, device="cuda").random_()       # about 30 us of reading
    outs = []
    with Ctx(cfg) as c:
        for hold in (True, False):
            d, dc = coarse_to_dev(co), chunks_to_dev(chk)
            out = torch.empty_like(d["q"])
            lse = torch.empty(cfg.B, cfg.Hq, dtype=torch.float32, device="cuda")
            torch.cuda.synchronize()
            if hold:
                ph.photon_read_probe(c.h, held)
            if folded:
                U = torch.empty(cfg.B, cfg.P, cfg.D, dtype=torch.bfloat16, device="cuda")
                oc = torch.empty_like(dc["q"])
                args = ph.make_step_args(d["kv"], d["k_new"], d["v_new"], d["q"], out, scale, dev_bf16(cv["w_out_major"]),
                                         ph.PHOTON_W_OUT_MAJOR, U, cfg.B, chunks=dc["kv"], q_chunk=dc["q"], out_chunk=oc,
                                         Nc=cfg.Nc, scale_chunk=scale, lse_coarse=lse)
                ph.photon_decode_step(c.h, args)
            else:
                ph.photon_kv_append(c.h, d["kv"], d["k_new"], d["v_new"])
                ph.photon_coarse_attn(c.h, d["kv"], d["q"], out, lse, scale)
            assert c.status() == 0
            outs.append((host_bits(out), lse.cpu().numpy(), host_bits(d["k"]), d["len"].cpu().numpy()))
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
    assert oracle.kv_append(co["k"], co["v"], co["len"], co["k_new"], co["v_new"]) == 0
    assert np.array_equal(outs[0][2], co["k"]) and np.array_equal(outs[0][3], co["len"])
    want, want_lse = oracle.attention(co["q"], co["k"], co["v"], co["len"], scale, n_threads=NT)
    assert_close(wl.bf16_bits_to_f64(outs[0][0]), want, "attention behind an append")
    fin = np.isfinite(want_lse)
    assert np.abs(outs[0][1][fin] - want_lse[fin]).max() < 2e-3


@pytest.mark.parametrize("max_splits", [1, 0])
def test_shared_prefix_with_logits_that_grow_along_the_prefix(oracle, max_splits):
    """Keys of later tiles score far higher than earlier ones for some query heads, so the reference
    maximum of those rows has to be raised, and their accumulator rescaled, in the middle of a key range."""
    cfg = cfg_small(3, B=40, S=8, shared_S=640)
    co = wl.coarse_inputs(cfg)
    co["len"][:] = 8
    qf = wl.bf16_bits_to_f64(co["q"])                               # [B, Hq, dh]
    ks = wl.bf16_bits_to_f64(co["k_shared"])                        # [1, Hkv, 640, dh]
    for kvh in range(cfg.Hkv):
        hq = kvh * cfg.G                                            # first query head of the group, unit 3
        for t in range(1, 5):                                       # one boosted key per 128-key tile, growing
            ks[0, kvh, 128 * t + 5] = qf[3, hq] * (0.6 * t)
    co["k_shared"] = wl.f32_to_bf16_bits(ks.astype(np.float32))
    scale = cfg.dh ** -0.5
    want, want_lse = oracle.attention(co["q"], co["k"], co["v"], co["len"], scale, shared=shared_of(co),
                                      n_threads=NT)
    with Ctx(cfg, max_splits=max_splits) as c:
        got, lse, _ = run_coarse(c, co, scale)
        assert c.status() == 0
    assert_close(got, want, "growing logits")
    assert np.abs(lse - want_lse).max() < 2e-3 * max(1.0, np.abs(want_lse).max() / 10)


def test_bad_shared_id_is_flagged_and_zeroed(oracle):
    cfg = cfg_small(3, B=6, S=20, shared_S=50)
    co = wl.coarse_inputs(cfg)
    co["len"][:] = 20
    co["shared_id"] = np.array([0, 0, 5, 0, -1, 0], np.int32)
    scale = cfg.dh ** -0.5
    want, _, flags = oracle.attention(co["q"], co["k"], co["v"], co["len"], scale,
                                      shared=shared_of(co), want_flags=True)
    with Ctx(cfg) as c:
        got, lse, _ = run_coarse(c, co, scale)
        assert c.status() == flags == ph.PHOTON_DEV_BAD_INDEX
    assert np.all(got[2] == 0) and np.all(np.isneginf(lse[2]))
    assert_close(got, want, "bad shared id")


def test_attention_is_deterministic_and_batch_permutation_equivariant():
    """Repeated calls are bit-identical.  Permuting the batch permutes the result; because the
    points where a cache is cut depend on its place in the batch, equality is up to the rounding
    of the merge (well inside one bf16 step of an O(1) value), not bit for bit."""
    cfg = cfg_small(1, B=24, S=333)
    co = wl.coarse_inputs(cfg)
    co["len"] = wl.uniform_int(5, "lens", cfg.B, 0, 333)
    scale = cfg.dh ** -0.5
    perm = np.random.default_rng(0).permutation(cfg.B)
    cp = dict(co, k=co["k"][perm], v=co["v"][perm], q=co["q"][perm], len=co["len"][perm])
    with Ctx(cfg) as c:
        _, _, b1 = run_coarse(c, co, scale)
        _, _, b2 = run_coarse(c, co, scale)
        _, _, b3 = run_coarse(c, cp, scale)
    assert np.array_equal(b1, b2)
    d = np.abs(wl.bf16_bits_to_f64(b3) - wl.bf16_bits_to_f64(b1[perm]))
    assert d.max() <= 2.0 ** -7 and (d > 0).mean() < 0.05


def test_flat_attention_on_a_token_level_cache(oracle):
    cfg = cfg_small(1, B=3, S=4096 + 5)       # token-level cache: one row per token
    co = wl.coarse_inputs(cfg, poison=True)
    scale = cfg.dh ** -0.5
    want, _ = oracle.attention(co["q"], co["k"], co["v"], co["len"], scale, n_threads=NT)
    with Ctx(cfg) as c:
        got, _, _ = run_coarse(c, co, scale, flat=True)
    assert_close(got, want, "flat")


# ------------------------------------------------------------------ converter

@pytest.mark.parametrize("idx,rows", [(0, None), (1, None), (2, None), (3, 24), (4, 24)])
@pytest.mark.parametrize("layout", [ph.PHOTON_W_IN_MAJOR, ph.PHOTON_W_OUT_MAJOR])
def test_converter_matches_oracle(oracle, idx, rows, layout):
    """Full batch on the device; at the two large batches the oracle recomputes a
    seeded sample of batch rows (each output row depends on its own x row only)."""
    cfg = wl.CONFIGS[idx]
    cv = wl.converter_inputs(cfg, with_bias=(idx == 0))
    out_major = layout == ph.PHOTON_W_OUT_MAJOR
    w = cv["w_out_major"] if out_major else cv["w_in_major"]
    pick = np.arange(cfg.B) if rows is None else np.sort(
        np.random.default_rng(idx).choice(cfg.B, rows, replace=False))
    want = oracle.converter(cv["x"][pick], w, cv["bias"], w_out_major=out_major, n_threads=NT)
    with Ctx(cfg) as c:
        U = torch.empty(cfg.B, cfg.P, cfg.D, dtype=torch.bfloat16, device="cuda")
        bias = None if cv["bias"] is None else dev_bf16(cv["bias"])
        ph.photon_converter(c.h, dev_bf16(cv["x"]), dev_bf16(w), layout, bias, U)
        torch.cuda.synchronize()
    assert_close(host_f64(U)[pick], want, f"converter cfg{idx}")


def test_converter_for_thousands_of_latents(oracle):
    """A batch large enough for the persistent large-tile kernel (more than two tiles of
    128 x 256 per SM), ragged last row tile, with bias; the oracle recomputes a sample of rows."""
    cfg = cfg_small(4, B=5000)                                  # D 1024, P 8: 40 x 32 tiles
    cv = wl.converter_inputs(cfg, with_bias=True)
    pick = np.sort(np.random.default_rng(8).choice(cfg.B, 96, replace=False))
    pick[-1] = cfg.B - 1
    want = oracle.converter(cv["x"][pick], cv["w_out_major"], cv["bias"], w_out_major=True, n_threads=NT)
    with Ctx(cfg) as c:
        U = torch.empty(cfg.B, cfg.P, cfg.D, dtype=torch.bfloat16, device="cuda")
        ph.photon_converter(c.h, dev_bf16(cv["x"]), dev_bf16(cv["w_out_major"]), ph.PHOTON_W_OUT_MAJOR,
                            dev_bf16(cv["bias"]), U)
        assert c.status() == 0
    assert_close(host_f64(U)[pick], want, "converter, 5000 latents")


def test_converter_one_hot_rows_are_bit_exact_and_ragged_batches_work():
    cfg = cfg_small(0, B=37)
    cv = wl.converter_inputs(cfg)
    x = np.zeros((cfg.B, cfg.D), np.uint16)
    hot = (np.arange(cfg.B) * 7) % cfg.D
    x[np.arange(cfg.B), hot] = 0x3F80                           # 1.0
    with Ctx(cfg) as c:
        U = torch.empty(cfg.B, cfg.P, cfg.D, dtype=torch.bfloat16, device="cuda")
        ph.photon_converter(c.h, dev_bf16(x), dev_bf16(cv["w_out_major"]), ph.PHOTON_W_OUT_MAJOR, None, U)
        torch.cuda.synchronize()
    assert np.array_equal(host_bits(U).reshape(cfg.B, -1), cv["w_in_major"][hot])


# ------------------------------------------------------------------ chunk attention

@pytest.mark.parametrize("idx", [0, 1, 2, 3])
def test_chunk_attention_matches_oracle(oracle, idx):
    cfg = wl.CONFIGS[idx]
    ch = wl.chunk_inputs(cfg, poison=True)
    scale = cfg.dh ** -0.5
    want, _ = oracle.chunk_attention(ch["q"], ch["kc"], ch["vc"], ch["len"], scale, n_threads=NT)
    with Ctx(cfg) as c:
        d = chunks_to_dev(ch)
        out = torch.empty_like(d["q"])
        ph.photon_chunk_attn(c.h, d["kv"], d["q"], None, out, scale=scale)
        assert c.status() == 0
    assert_close(host_f64(out), want, f"chunk cfg{idx}")


def test_chunk_attention_full_size_chunk_parallel_config_sampled(oracle):
    """All 16 384 chunks on the device in the benchmark's launch shape; the
    oracle recomputes a seeded sample of chunks (each is independent of all others)."""
    cfg = wl.CONFIGS[4]
    ch = wl.chunk_inputs(cfg, poison=True)
    scale = cfg.dh ** -0.5
    pick = np.sort(np.random.default_rng(4).choice(cfg.Nc, 600, replace=False)).astype(np.int32)
    pick[:3] = [0, 1, 2]
    pick[-1] = cfg.Nc - 1
    want, _ = oracle.chunk_attention(ch["q"][pick], ch["kc"], ch["vc"], ch["len"], scale, slot=pick,
                                     n_threads=NT)
    with Ctx(cfg) as c:
        d = chunks_to_dev(ch)
        out = torch.empty_like(d["q"])
        ph.photon_chunk_attn(c.h, d["kv"], d["q"], None, out, scale=scale)
        assert c.status() == 0
    assert_close(host_f64(out)[pick], want, "chunk cfg4 sample")


def test_chunk_attention_strict_positions_gather_and_bad_slots(oracle):
    """n_in = j - 1 (query is the latent before in-chunk position j, incl. the
    prefix-only case), a gather through `slot`, and an out-of-range slot."""
    cfg = cfg_small(4, B=4)
    ch = wl.chunk_inputs(cfg, poison=True, strict_paper=True)
    assert ch["len"].min() == cfg.P
    scale = cfg.dh ** -0.5
    slot = np.random.default_rng(1).permutation(cfg.Nc).astype(np.int32)[:100]
    slot[17] = cfg.Nc + 3
    q = ch["q"][:100]
    want, _, flags = oracle.attention(q, ch["kc"], ch["vc"], ch["len"], scale, slot=slot, want_flags=True)
    with Ctx(cfg) as c:
        d = chunks_to_dev(ch)
        dq = dev_bf16(q)
        out = torch.full_like(dq, 7.0)
        ph.photon_chunk_attn(c.h, d["kv"], dq, dev_i32(slot), out, scale=scale)
        assert c.status() == flags == ph.PHOTON_DEV_BAD_INDEX
    got = host_f64(out)
    assert np.all(got[17] == 0)
    assert_close(got, want, "chunk gather")


@pytest.mark.parametrize("idx,B", [(1, 2048), (0, 1024)])
def test_chunk_attention_large_batches_with_gather(oracle, idx, B):
    """Thousands of chunks, grouped query heads, a gather through `slot` with one bad entry,
    strict (prefix-only) positions and poisoned rows."""
    cfg = cfg_small(idx, B=B)
    ch = wl.chunk_inputs(cfg, poison=True, strict_paper=True)
    scale = cfg.dh ** -0.5
    slot = np.random.default_rng(idx).permutation(cfg.Nc).astype(np.int32)
    slot[123] = -5
    pick = np.sort(np.random.default_rng(9).choice(cfg.Nc, 400, replace=False))
    pick[0] = 123
    pick.sort()
    want, _, flags = oracle.attention(ch["q"][pick], ch["kc"], ch["vc"], ch["len"], scale,
                                      slot=slot[pick], n_threads=NT, want_flags=True)
    with Ctx(cfg) as c:
        d = chunks_to_dev(ch)
        out = torch.full_like(d["q"], 3.0)
        ph.photon_chunk_attn(c.h, d["kv"], d["q"], dev_i32(slot), out, scale=scale)
        assert c.status() == flags == ph.PHOTON_DEV_BAD_INDEX
    got = host_f64(out)
    assert np.all(got[123] == 0)
    assert_close(got[pick], want, "chunk gather, large batch")


@pytest.mark.parametrize("dh,Hq,Hkv", [(128, 8, 2), (64, 6, 2), (64, 3, 3)])
def test_chunk_attention_at_the_largest_window(oracle, dh, Hq, Hkv):
    """P + C = 64, the widest window a context accepts (several passes over the rows), every length
    from 0 to 64, group sizes 4, 3 and 1, poisoned rows past the end."""
    cfg = cfg_small(4, B=5, chunks_per_seq=13, P=16, C=48, Hq=Hq, Hkv=Hkv, dh=dh, D=Hq * dh)
    ch = wl.chunk_inputs(cfg, poison=True)
    lens = (np.arange(cfg.Nc) % 65).astype(np.int32)
    cap = cfg.P + cfg.C
    bad = np.arange(cap)[None, :] >= lens[:, None]
    ch["kc"][np.broadcast_to(bad[:, None, :, None], ch["kc"].shape)] = 0x7FC1
    ch["vc"][np.broadcast_to(bad[:, None, :, None], ch["vc"].shape)] = 0xFFC1
    # rows that are valid now but were poisoned by the generator: give them values again
    fresh_k = wl.normal_bf16(11, "k", ch["kc"].shape)
    fresh_v = wl.normal_bf16(12, "v", ch["vc"].shape)
    ok = np.broadcast_to(~bad[:, None, :, None], ch["kc"].shape)
    ch["kc"][ok] = fresh_k[ok]
    ch["vc"][ok] = fresh_v[ok]
    ch["len"] = lens
    scale = cfg.dh ** -0.5
    want, _ = oracle.chunk_attention(ch["q"], ch["kc"], ch["vc"], lens, scale, n_threads=NT)
    with Ctx(cfg) as c:
        d = chunks_to_dev(ch)
        out = torch.full_like(d["q"], 5.0)
        ph.photon_chunk_attn(c.h, d["kv"], d["q"], None, out, scale=scale)
        assert c.status() == 0
    got = host_f64(out)
    assert np.all(got[lens == 0] == 0)
    assert_close(got, want, f"chunk cap 64 dh={dh} G={Hq // Hkv}")


@pytest.mark.parametrize("dh,Hq,Hkv,P,C", [(128, 8, 8, 8, 16), (128, 8, 2, 8, 24), (64, 6, 2, 8, 16), (64, 3, 3, 4, 4)])
def test_chunk_attention_through_the_ring_of_bulk_copies(oracle, dh, Hq, Hkv, P, C):
    """Enough (chunk, KV head) pairs for the persistent kernel whose warps keep their next items on their way
    into shared memory: every length from 0 to the capacity (empty items take no slot turn), a number of items
    that is no multiple of the grid, a gather through a permutation with two bad entries, poisoned rows past
    the end, group sizes 1, 3 and 4.  Every output is compared."""
    n_chunks = (8 * 148 * 8 + Hkv - 1) // Hkv + 37
    cfg = cfg_small(4, B=n_chunks, chunks_per_seq=1, P=P, C=C, Hq=Hq, Hkv=Hkv, dh=dh, D=Hq * dh)
    assert cfg.Nc == n_chunks
    ch = wl.chunk_inputs(cfg, poison=True)
    cap = P + C
    lens = ((np.arange(cfg.Nc) * 7) % (cap + 1)).astype(np.int32)
    bad = np.arange(cap)[None, :] >= lens[:, None]
    fresh_k = wl.normal_bf16(21, "k", ch["kc"].shape)
    fresh_v = wl.normal_bf16(22, "v", ch["vc"].shape)
    gone = np.broadcast_to(bad[:, None, :, None], ch["kc"].shape)
    ch["kc"] = np.where(gone, np.uint16(0x7FC1), fresh_k)
    ch["vc"] = np.where(gone, np.uint16(0xFFC1), fresh_v)
    ch["len"] = lens
    scale = cfg.dh ** -0.5
    slot = np.random.default_rng(dh + Hq).permutation(cfg.Nc).astype(np.int32)
    slot[5] = -1
    slot[cfg.Nc - 2] = cfg.Nc
    want, _, flags = oracle.attention(ch["q"], ch["kc"], ch["vc"], lens, scale, slot=slot, n_threads=NT, want_flags=True)
    with Ctx(cfg) as c:
        d = chunks_to_dev(ch)
        out = torch.full_like(d["q"], 5.0)
        ph.photon_chunk_attn(c.h, d["kv"], d["q"], dev_i32(slot), out, scale=scale)
        assert c.status() == flags == ph.PHOTON_DEV_BAD_INDEX
    got = host_f64(out)
    assert np.all(got[5] == 0) and np.all(got[cfg.Nc - 2] == 0)
    empty = lens[np.clip(slot, 0, cfg.Nc - 1)] == 0
    assert np.all(got[empty] == 0)
    assert_close(got, want, f"chunk ring dh={dh} G={Hq // Hkv} cap={cap}")


@pytest.mark.parametrize("idx,lengths,B", [(1, (2, 2), 16), (1, (4, 4, 4), 64), (3, (2, 2), 64), (4, (2, 2), 8)])
def test_decode_step_under_other_hierarchies(oracle, idx, lengths, B):
    """The whole step on the shapes another hierarchy gives the same model: (2, 2) makes
    the coarse stream four times longer and the token chunks two long; three levels
    make it four times shorter."""
    cfg = wl.with_hierarchy(cfg_small(idx, B=B), lengths)
    s = wl.step_inputs(cfg, poison=True)
    co, cv, ch = s["coarse"], s["converter"], s["chunks"]
    scale = cfg.dh ** -0.5
    with Ctx(cfg) as c:
        d, dc = coarse_to_dev(co), chunks_to_dev(ch)
        out = torch.empty_like(d["q"])
        U = torch.empty(cfg.B, cfg.P, cfg.D, dtype=torch.bfloat16, device="cuda")
        oc = torch.empty_like(dc["q"])
        args = ph.make_step_args(d["kv"], d["k_new"], d["v_new"], d["q"], out, scale, dev_bf16(cv["w_in_major"]),
                                 ph.PHOTON_W_IN_MAJOR, U, cfg.B, chunks=dc["kv"], q_chunk=dc["q"], out_chunk=oc,
                                 Nc=cfg.Nc, scale_chunk=scale)
        ph.photon_decode_step(c.h, args)
        assert c.status() == 0
    want = oracle.decode_step(co, cv, ch, scale, scale, chain=True, n_threads=NT)
    assert_close(host_f64(out), want["out"], f"coarse {cfg.name}")
    assert_close(host_f64(oc), want["chunk_out"], f"chunk {cfg.name}")
    assert_close(host_f64(U), want["U"], f"U {cfg.name}")


def test_calls_larger_than_the_context_was_made_for_are_refused():
    cfg = cfg_small(1, B=8, S=70)
    co = wl.coarse_inputs(cfg)
    with Ctx(cfg, max_queries=4) as c:
        d = coarse_to_dev(co)
        out = torch.empty_like(d["q"])
        n0 = ph.photon_launch_count(c.h)
        with pytest.raises(ph.PhotonError) as e:
            ph.photon_coarse_attn(c.h, d["kv"], d["q"], out, None, 1.0)
        assert e.value.code == ph.PHOTON_ERR_WORKSPACE
        assert ph.photon_launch_count(c.h) == n0 and c.status() == 0


def test_chunk_attention_ignores_other_chunks_bit_exactly():
    cfg = cfg_small(4, B=2)
    ch = wl.chunk_inputs(cfg)
    scale = cfg.dh ** -0.5
    ch2 = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in ch.items()}
    other = np.arange(cfg.Nc) != 11
    ch2["kc"][other] = wl.normal_bf16(77, "a", ch2["kc"][other].shape)
    ch2["vc"][other] = wl.normal_bf16(78, "a", ch2["vc"][other].shape)
    ch2["q"][other] = wl.normal_bf16(79, "a", ch2["q"][other].shape)
    with Ctx(cfg) as c:
        outs = []
        for x in (ch, ch2):
            d = chunks_to_dev(x)
            out = torch.empty_like(d["q"])
            ph.photon_chunk_attn(c.h, d["kv"], d["q"], None, out, scale=scale)
            outs.append(host_bits(out))
    assert np.array_equal(outs[0][11], outs[1][11]) and not np.array_equal(outs[0][10], outs[1][10])


# ------------------------------------------------------------------ the step

@pytest.mark.parametrize("idx", [0, 1, 3])
@pytest.mark.parametrize("layout", [ph.PHOTON_W_IN_MAJOR, ph.PHOTON_W_OUT_MAJOR])
def test_decode_step_chain_matches_oracle(oracle, idx, layout):
    cfg = wl.CONFIGS[idx] if idx != 3 else cfg_small(3, B=48, shared_S=512)
    s = wl.step_inputs(cfg, poison=True)
    co, cv, chk = s["coarse"], s["converter"], s["chunks"]
    out_major = layout == ph.PHOTON_W_OUT_MAJOR
    scale = cfg.dh ** -0.5
    with Ctx(cfg) as c:
        d, dc = coarse_to_dev(co), chunks_to_dev(chk)
        out = torch.empty_like(d["q"])
        lse = torch.empty(cfg.B, cfg.Hq, dtype=torch.float32, device="cuda")
        U = torch.empty(cfg.B, cfg.P, cfg.D, dtype=torch.bfloat16, device="cuda")
        oc = torch.empty_like(dc["q"])
        w = dev_bf16(cv["w_out_major"] if out_major else cv["w_in_major"])
        args = ph.make_step_args(d["kv"], d["k_new"], d["v_new"], d["q"], out, scale, w, layout, U,
                                 cfg.B, chunks=dc["kv"], q_chunk=dc["q"], out_chunk=oc, Nc=cfg.Nc,
                                 scale_chunk=scale, lse_coarse=lse)
        n0 = ph.photon_launch_count(c.h)
        ph.photon_decode_step(c.h, args)
        assert c.status() == 0
        assert ph.photon_launch_count(c.h) > n0
        r = oracle.decode_step(co, cv, chk, scale, scale, chain=True, w_out_major=out_major,
                               n_threads=NT)
        assert np.array_equal(host_bits(d["k"]), co["k"]) and np.array_equal(host_bits(d["v"]), co["v"])
        assert np.array_equal(d["len"].cpu().numpy(), co["len"])
        assert_close(host_f64(out), r["out"], "step: coarse out")
        assert_close(host_f64(U), r["U"], "step: U")
        assert_close(host_f64(oc), r["chunk_out"], "step: chunk out")
        assert np.abs(lse.cpu().numpy() - r["lse"]).max() < 2e-3


@pytest.mark.parametrize("shared", [False, True])
def test_step_with_the_append_folded_into_the_attention_equals_append_then_attention(oracle, shared):
    """For a contiguous cache the step installs the new row inside the attention kernel instead of launching the
    append first.  Cache, lengths, status bits and the attention output must be what photon_kv_append followed
    by photon_coarse_attn gives, bit for bit: lengths that open a new tile (64, 128), that fill the last slot, and
    a unit without room, which is flagged and attends its full cache unchanged."""
    cfg = cfg_small(3, B=13, S=330, shared_S=200) if shared else cfg_small(1, B=13, S=330)
    s = wl.step_inputs(cfg, poison=True)
    co, cv, chk = s["coarse"], s["converter"], s["chunks"]
    lens = np.array([0, 1, 63, 64, 65, 127, 128, 300, 328, 329, 330, 200, 5], np.int32)
    co["k"] = wl.normal_bf16(9, "k", co["k"].shape)
    co["v"] = wl.normal_bf16(9, "v", co["v"].shape)
    for u, n in enumerate(lens):
        if n < 330:                                      # the slot the new row goes to, and everything behind it
            co["k"][u, :, n:] = 0x7FC1
            co["v"][u, :, n:] = 0xFFC1
    co["len"] = lens
    scale = cfg.dh ** -0.5
    with Ctx(cfg) as c:
        # append, then attention, as two calls
        d1 = coarse_to_dev(co)
        out1 = torch.empty_like(d1["q"])
        lse1 = torch.empty(cfg.B, cfg.Hq, dtype=torch.float32, device="cuda")
        n0 = ph.photon_launch_count(c.h)
        ph.photon_kv_append(c.h, d1["kv"], d1["k_new"], d1["v_new"])
        ph.photon_coarse_attn(c.h, d1["kv"], d1["q"], out1, lse1, scale)
        two_calls = ph.photon_launch_count(c.h) - n0
        assert c.status() == ph.PHOTON_DEV_CAPACITY
        # the step
        d2, dc = coarse_to_dev(co), chunks_to_dev(chk)
        out2 = torch.empty_like(d2["q"])
        lse2 = torch.empty_like(lse1)
        U = torch.empty(cfg.B, cfg.P, cfg.D, dtype=torch.bfloat16, device="cuda")
        oc = torch.empty_like(dc["q"])
        args = ph.make_step_args(d2["kv"], d2["k_new"], d2["v_new"], d2["q"], out2, scale, dev_bf16(cv["w_out_major"]),
                                 ph.PHOTON_W_OUT_MAJOR, U, cfg.B, chunks=dc["kv"], q_chunk=dc["q"], out_chunk=oc,
                                 Nc=cfg.Nc, scale_chunk=scale, lse_coarse=lse2)
        n0 = ph.photon_launch_count(c.h)
        ph.photon_decode_step(c.h, args)
        assert ph.photon_launch_count(c.h) - n0 == two_calls - 1 + 2       # no append launch; converter and chunk attention
        assert c.status() == ph.PHOTON_DEV_CAPACITY
        ph.photon_decode_step(c.h, args)                                    # the counters are back at zero: a second step works
        assert c.status() == ph.PHOTON_DEV_CAPACITY
        for name in ("k", "v"):
            got1 = host_bits(d1[name])
        assert np.array_equal(d1["len"].cpu().numpy(), np.minimum(lens + 1, 330))
        assert np.array_equal(d2["len"].cpu().numpy(), np.minimum(lens + 2, 330))
    # first step of the folded path against the two calls: redo it on fresh buffers (the second step above moved on)
    with Ctx(cfg) as c:
        d3, dc = coarse_to_dev(co), chunks_to_dev(chk)
        out3 = torch.empty_like(d3["q"])
        lse3 = torch.empty_like(lse1)
        args = ph.make_step_args(d3["kv"], d3["k_new"], d3["v_new"], d3["q"], out3, scale, dev_bf16(cv["w_out_major"]),
                                 ph.PHOTON_W_OUT_MAJOR, U, cfg.B, chunks=dc["kv"], q_chunk=dc["q"], out_chunk=oc,
                                 Nc=cfg.Nc, scale_chunk=scale, lse_coarse=lse3)
        ph.photon_decode_step(c.h, args)
        assert c.status() == ph.PHOTON_DEV_CAPACITY
        assert np.array_equal(host_bits(d3["k"]), host_bits(d1["k"])) and np.array_equal(host_bits(d3["v"]), host_bits(d1["v"]))
        assert np.array_equal(d3["len"].cpu().numpy(), d1["len"].cpu().numpy())
        assert np.array_equal(host_bits(out3), host_bits(out1))
        assert np.array_equal(lse3.cpu().numpy(), lse1.cpu().numpy())
    flags = oracle.kv_append(co["k"], co["v"], co["len"], co["k_new"], co["v_new"])
    assert flags == ph.PHOTON_DEV_CAPACITY
    assert np.array_equal(host_bits(d3["k"]), co["k"]) and np.array_equal(host_bits(d3["v"]), co["v"])
    want, _ = oracle.attention(co["q"], co["k"], co["v"], co["len"], scale, shared=shared_of(co), n_threads=NT)
    assert_close(host_f64(out3), want, "folded append")


@pytest.mark.parametrize("idx", [2, 3, 4])
def test_decode_step_chain_at_full_size(oracle, idx):
    """The step as the benchmark times it on the long-context, shared-prefix and chunk-parallel workloads: one
    call at full size.  The append is checked in full and bit for bit, the coarse attention in full; of the
    converter and the chunk attention the oracle recomputes a seeded sample of rows / chunks (every row of U
    depends on its own latent only, every chunk on its own buffer only)."""
    cfg = wl.CONFIGS[idx]
    s = wl.step_inputs(cfg, poison=True)
    co, cv, chk = s["coarse"], s["converter"], s["chunks"]
    scale = cfg.dh ** -0.5
    rng = np.random.default_rng(40 + idx)
    rows = np.sort(rng.choice(cfg.B, min(cfg.B, 24), replace=False))
    pick = np.sort(rng.choice(cfg.Nc, min(cfg.Nc, 400), replace=False)).astype(np.int32)
    pick[0], pick[-1] = 0, cfg.Nc - 1
    with Ctx(cfg) as c:
        d, dc = coarse_to_dev(co), chunks_to_dev(chk)
        out = torch.empty_like(d["q"])
        lse = torch.empty(cfg.B, cfg.Hq, dtype=torch.float32, device="cuda")
        U = torch.empty(cfg.B, cfg.P, cfg.D, dtype=torch.bfloat16, device="cuda")
        oc = torch.empty_like(dc["q"])
        args = ph.make_step_args(d["kv"], d["k_new"], d["v_new"], d["q"], out, scale, dev_bf16(cv["w_out_major"]),
                                 ph.PHOTON_W_OUT_MAJOR, U, cfg.B, chunks=dc["kv"], q_chunk=dc["q"], out_chunk=oc,
                                 Nc=cfg.Nc, scale_chunk=scale, lse_coarse=lse)
        ph.photon_decode_step(c.h, args)
        assert c.status() == 0
        assert oracle.kv_append(co["k"], co["v"], co["len"], co["k_new"], co["v_new"]) == 0
        assert np.array_equal(host_bits(d["k"]), co["k"]) and np.array_equal(host_bits(d["v"]), co["v"])
        assert np.array_equal(d["len"].cpu().numpy(), co["len"])
        want, want_lse = oracle.attention(co["q"], co["k"], co["v"], co["len"], scale, shared=shared_of(co),
                                          n_threads=NT)
        assert_close(host_f64(out), want, f"step cfg{idx}: coarse out")
        assert np.abs(lse.cpu().numpy() - want_lse).max() < 2e-3
        x = oracle.round_bf16(want).reshape(cfg.B, -1)[rows]
        want_U = oracle.converter(x, cv["w_out_major"], None, w_out_major=True, n_threads=NT)
        assert_close(host_f64(U)[rows], want_U.reshape(len(rows), cfg.P, cfg.D), f"step cfg{idx}: U rows")
        want_c, _ = oracle.chunk_attention(chk["q"][pick], chk["kc"], chk["vc"], chk["len"], scale, slot=pick,
                                           n_threads=NT)
        assert_close(host_f64(oc)[pick], want_c, f"step cfg{idx}: chunk sample")


# chunk attention beside the coarse part with little / with more than 1 MiB to move, and in line after it
@pytest.mark.parametrize("idx,B,S", [(1, 24, 300), (1, 130, 200), (4, 12, 128), (4, 40, 64)])
@pytest.mark.parametrize("pinned,split", [(True, True), (True, False), (False, True), (False, False)])
def test_decode_step_from_host_buffers(oracle, pinned, split, idx, B, S):
    """The step whose inputs (new K/V rows, both query tensors, the lengths) start in host memory and
    whose results end there: one packed buffer each way through the staging areas the arguments look into;
    with the split declared, the chunk attention's half of either buffer travels beside the coarse part."""
    cfg = cfg_small(idx, B=B, S=S)
    s = wl.step_inputs(cfg, poison=True)
    co, cv, chk = s["coarse"], s["converter"], s["chunks"]
    scale = cfg.dh ** -0.5
    assert (cfg.Nc * cfg.Hkv * chk["cap"] * cfg.dh * 4 <= 32 << 20) == (idx == 1)
    with Ctx(cfg) as c:
        d, dc = coarse_to_dev(co), chunks_to_dev(chk)
        lens0 = co["len"].copy()                                             # before the append
        ins = [co["k_new"], co["v_new"], co["q"], lens0, chk["q"]]              # the chunk attention's input last
        offs, total = [], 0
        for a in ins:
            offs.append(total)
            total += (a.nbytes + 255) // 256 * 256
        h_in = torch.zeros(total, dtype=torch.uint8)
        for a, o in zip(ins, offs):
            h_in[o:o + a.nbytes] = torch.from_numpy(np.ascontiguousarray(a).view(np.uint8).reshape(-1))
        d_in = torch.full((total,), 0xEE, dtype=torch.uint8, device="cuda")

        def view(j, like, dtype):
            return d_in[offs[j]:offs[j] + ins[j].nbytes].view(dtype).view(like.shape)
        k_new, v_new, q = (view(j, t, torch.bfloat16) for j, t in enumerate((d["k_new"], d["v_new"], d["q"])))
        ln, qc = view(3, d["len"], torch.int32), view(4, dc["q"], torch.bfloat16)
        n_out, n_oc = d["q"].numel() * 2, dc["q"].numel() * 2
        d_out = torch.full((n_out + n_oc,), 0xEE, dtype=torch.uint8, device="cuda")
        h_out = torch.zeros(n_out + n_oc, dtype=torch.uint8)
        if pinned:
            h_in, h_out = h_in.pin_memory(), h_out.pin_memory()
        out = d_out[:n_out].view(torch.bfloat16).view(d["q"].shape)
        oc = d_out[n_out:].view(torch.bfloat16).view(dc["q"].shape)
        U = torch.empty(cfg.B, cfg.P, cfg.D, dtype=torch.bfloat16, device="cuda")
        # the cache as it was before the newest row: the lengths come from the host with everything else
        co0 = wl.coarse_inputs(cfg, poison=True)
        kv = ph.make_kv(dev_bf16(co0["k"]), dev_bf16(co0["v"]), ln, max_len=cfg.S)
        args = ph.make_step_args(kv, k_new, v_new, q, out, scale, dev_bf16(cv["w_in_major"]), ph.PHOTON_W_IN_MAJOR, U,
                                 cfg.B, chunks=dc["kv"], q_chunk=qc, out_chunk=oc, Nc=cfg.Nc, scale_chunk=scale)
        io = ph.HostIO(h_in, d_in, d_out, h_out, in_split=offs[4], out_split=n_out) if split else ph.HostIO(h_in, d_in, d_out, h_out)
        ph.photon_decode_step_host(c.h, args, io)                              # returns with the results on the host
        got = h_out.numpy().copy()
        assert c.status() == 0
        # page-locked buffers with the split declared: the chunk attention wrote to the host buffer itself and its
        # half of the staging area was never touched; in every other case the results passed through it
        staged = d_out[n_out:].cpu().numpy()
        direct = pinned and split and (idx == 4 or n_oc <= 1 << 20)
        assert bool((staged == 0xEE).all()) if direct else np.array_equal(staged, got[n_out:])
        assert np.array_equal(ln.cpu().numpy(), lens0 + 1)
        # the same step from device tensors gives the same bits
        out2, oc2, U2 = torch.empty_like(d["q"]), torch.empty_like(dc["q"]), torch.empty_like(U)
        args2 = ph.make_step_args(d["kv"], d["k_new"], d["v_new"], d["q"], out2, scale, dev_bf16(cv["w_in_major"]),
                                  ph.PHOTON_W_IN_MAJOR, U2, cfg.B, chunks=dc["kv"], q_chunk=dc["q"], out_chunk=oc2,
                                  Nc=cfg.Nc, scale_chunk=scale)
        ph.photon_decode_step(c.h, args2)
        assert np.array_equal(got[:n_out].view(np.uint16).reshape(out2.shape), host_bits(out2))
        assert np.array_equal(got[n_out:].view(np.uint16).reshape(oc2.shape), host_bits(oc2))
        n0 = ph.photon_launch_count(c.h)
        assert ph.load().photon_decode_step_host(c.h, None, None, None, 0, 0, None, None, 0, 0, None) == ph.PHOTON_ERR_INVALID_ARG
        with pytest.raises(ph.PhotonError) as e:                               # a split beyond the buffer
            ph.photon_decode_step_host(c.h, args, ph.HostIO(h_in, d_in, d_out, h_out, in_split=total + 1))
        assert e.value.code == ph.PHOTON_ERR_INVALID_ARG
        with pytest.raises(ValueError):
            ph.HostIO(h_in, d_in, d_out, h_out[:-1])
        assert ph.photon_launch_count(c.h) == n0
    r = oracle.decode_step(co, cv, chk, scale, scale, chain=True, n_threads=NT)
    assert_close(wl.bf16_bits_to_f64(got[:n_out].view(np.uint16)).reshape(r["out"].shape), r["out"], "host step: coarse out")
    assert_close(wl.bf16_bits_to_f64(got[n_out:].view(np.uint16)).reshape(r["chunk_out"].shape), r["chunk_out"], "host step: chunk out")


def test_decode_step_with_given_x_and_no_chunks(oracle):
    cfg = wl.CONFIGS[0]
    s = wl.step_inputs(cfg)
    co, cv = s["coarse"], s["converter"]
    scale = cfg.dh ** -0.5
    with Ctx(cfg) as c:
        d = coarse_to_dev(co)
        out = torch.empty_like(d["q"])
        U = torch.empty(cfg.B, cfg.P, cfg.D, dtype=torch.bfloat16, device="cuda")
        args = ph.make_step_args(d["kv"], d["k_new"], d["v_new"], d["q"], out, scale,
                                 dev_bf16(cv["w_in_major"]), ph.PHOTON_W_IN_MAJOR, U, cfg.B,
                                 x=dev_bf16(cv["x"]))
        ph.photon_decode_step(c.h, args)
        assert c.status() == 0
    want = oracle.converter(cv["x"], cv["w_in_major"])
    assert_close(host_f64(U), want, "step: U from x")


# ------------------------------------------------------------------ argument checks on a live context

def test_invalid_arguments_launch_nothing():
    cfg = wl.CONFIGS[0]
    co = wl.coarse_inputs(cfg)
    with Ctx(cfg) as c:
        d = coarse_to_dev(co)
        out = torch.empty_like(d["q"])
        n0 = ph.photon_launch_count(c.h)
        with pytest.raises(ph.PhotonError) as e:              # misaligned q
            ph.photon_coarse_attn(c.h, d["kv"], d["q"].data_ptr() + 2, out, None, 1.0)
        assert e.value.code == ph.PHOTON_ERR_INVALID_ARG
        with pytest.raises(ph.PhotonError):                   # NULL out
            ph.photon_coarse_attn(c.h, d["kv"], d["q"], None, None, 1.0)
        with pytest.raises(ph.PhotonError):                   # NaN scale
            ph.photon_coarse_attn(c.h, d["kv"], d["q"], out, None, float("nan"))
        with pytest.raises(ph.PhotonError):                   # bad layout code
            ph.photon_converter(c.h, d["q"], d["q"], 5, None, out, 2)
        with pytest.raises(ph.PhotonError):                   # chunk cache wider than P + C
            ph.photon_chunk_attn(c.h, d["kv"], d["q"], None, out, 2, 1.0)
        with pytest.raises(ph.PhotonError):                   # append more rows than capacity
            ph.photon_kv_append(c.h, d["kv"], d["k_new"], d["v_new"], n_rows=cfg.S + 1)
        assert ph.photon_launch_count(c.h) == n0 and c.status() == 0
    with pytest.raises(ph.PhotonError) as e:
        ph.photon_create(4, 2, 96, 256, 4, 4, 16)
    assert e.value.code == ph.PHOTON_ERR_UNSUPPORTED
