"""Parity of the whole-chunk causal attention (the local decoder at many
positions of a chunk at once) with the CPU oracle, through the C boundary.
bf16 outputs: max abs error 2e-2, mean abs error 2e-3 against the fp64 oracle;
rows that do not exist yet must be exactly zero."""
import numpy as np
import pytest
import torch

import paper_2512_20687_b200 as ph
from paper_2512_20687_b200 import workloads as wl

from gpu_util import Ctx, assert_close, chunks_to_dev, dev_bf16, dev_i32, host_bits, host_f64

pytestmark = pytest.mark.gpu

NT = 16     # oracle threads


def cfg_small(i, **kw):
    return wl.scaled(wl.CONFIGS[i], **kw)


def run(c, d, q, slot=None, row0=0, scale=1.0, fill=9.0):
    out = torch.full_like(q, fill)
    ph.photon_chunk_causal_attn(c.h, d["kv"], q, slot, out, row0=row0, scale=scale)
    return out


def missing_rows(lens, row0, R):
    return (row0 + np.arange(R))[None, :] >= np.asarray(lens)[:, None]        # [n, R]


@pytest.mark.parametrize("idx", [0, 1, 2, 3])
@pytest.mark.parametrize("full", [False, True])
def test_whole_chunks_match_oracle(oracle, idx, full):
    """Every position of every in-flight chunk: ragged lengths with poisoned rows
    past the end, and complete chunks (the teacher-forced case)."""
    cfg = wl.CONFIGS[idx]
    ch = wl.chunk_causal_inputs(cfg, poison=True, full=full)
    scale = cfg.dh ** -0.5
    want = oracle.chunk_causal_attention(ch["q"], ch["kc"], ch["vc"], ch["len"], scale, n_threads=NT)
    with Ctx(cfg) as c:
        d = chunks_to_dev(ch)
        out = run(c, d, d["q"], scale=scale)
        assert c.status() == 0
    got = host_f64(out)
    assert np.all(got[missing_rows(ch["len"], 0, ch["rows"])] == 0)
    assert_close(got, want, f"causal chunk cfg{idx} full={full}")


def test_full_size_chunk_parallel_config_sampled(oracle):
    """All 16 384 chunks of the chunk-parallel configuration in one launch; the
    oracle recomputes a seeded sample of chunks (each is independent of the rest)."""
    cfg = wl.CONFIGS[4]
    ch = wl.chunk_causal_inputs(cfg, poison=True)
    scale = cfg.dh ** -0.5
    pick = np.sort(np.random.default_rng(5).choice(cfg.Nc, 300, replace=False)).astype(np.int32)
    pick[:2] = [0, 1]
    pick[-1] = cfg.Nc - 1
    want = oracle.chunk_causal_attention(ch["q"][pick], ch["kc"], ch["vc"], ch["len"], scale,
                                         slot=pick, n_threads=NT)
    with Ctx(cfg) as c:
        d = chunks_to_dev(ch)
        out = run(c, d, d["q"], scale=scale)
        assert c.status() == 0
    got = host_f64(out[torch.from_numpy(pick).long().cuda()])
    assert np.all(got[missing_rows(ch["len"][pick], 0, ch["rows"])] == 0)
    assert_close(got, want, "causal chunk cfg4 sample")


@pytest.mark.parametrize("row0,rows", [(0, 8), (8, 16), (5, 7), (23, 1), (0, 1), (3, 20)])
def test_row_windows(oracle, row0, rows):
    """The prefix-only pass (rows 0..P-1), the in-chunk rows only, single rows and
    windows that straddle the 16-row tiles, on ragged chunks."""
    cfg = cfg_small(4, B=6)                                   # P = 8, C = 16: 24 rows
    ch = wl.chunk_causal_inputs(cfg, poison=True, row0=row0, rows=rows)
    scale = cfg.dh ** -0.5
    want = oracle.chunk_causal_attention(ch["q"], ch["kc"], ch["vc"], ch["len"], scale, row0=row0,
                                         n_threads=NT)
    with Ctx(cfg) as c:
        d = chunks_to_dev(ch)
        out = run(c, d, d["q"], row0=row0, scale=scale)
        assert c.status() == 0
    got = host_f64(out)
    assert np.all(got[missing_rows(ch["len"], row0, rows)] == 0)
    assert_close(got, want, f"causal chunk rows {row0}+{rows}")


@pytest.mark.parametrize("dh,Hq,Hkv,P,C", [(128, 8, 2, 16, 48), (64, 6, 2, 16, 48), (64, 3, 3, 8, 40),
                                           (128, 4, 4, 4, 29), (64, 16, 1, 2, 9)])
def test_every_length_up_to_the_widest_window(oracle, dh, Hq, Hkv, P, C):
    """Buffers of up to 64 rows (1 to 4 key tiles), every length from 0 to the
    capacity, group sizes 1, 3, 4 and 16, both head sizes, NaN patterns past the end."""
    cfg = cfg_small(4, B=5, chunks_per_seq=14, P=P, C=C, Hq=Hq, Hkv=Hkv, dh=dh, D=Hq * dh)
    cap = P + C
    ch = wl.chunk_causal_inputs(cfg, full=True)
    lens = (np.arange(cfg.Nc) % (cap + 1)).astype(np.int32)
    gone = np.arange(cap)[None, :] >= lens[:, None]
    ch["kc"][np.broadcast_to(gone[:, None, :, None], ch["kc"].shape)] = 0x7FC1
    ch["vc"][np.broadcast_to(gone[:, None, :, None], ch["vc"].shape)] = 0xFFC1
    ch["len"] = lens
    scale = dh ** -0.5
    want = oracle.chunk_causal_attention(ch["q"], ch["kc"], ch["vc"], lens, scale, n_threads=NT)
    with Ctx(cfg) as c:
        d = chunks_to_dev(ch)
        out = run(c, d, d["q"], scale=scale)
        assert c.status() == 0
    got = host_f64(out)
    assert np.all(got[missing_rows(lens, 0, cap)] == 0)
    assert_close(got, want, f"causal chunk cap {cap} dh={dh} G={Hq // Hkv}")


def test_gather_through_slots_and_bad_slots(oracle):
    cfg = cfg_small(1, B=512)                                 # 16 query / 4 KV heads, 8-row buffers
    ch = wl.chunk_causal_inputs(cfg, poison=True)
    scale = cfg.dh ** -0.5
    n = 700
    slot = np.random.default_rng(2).integers(0, cfg.Nc, n).astype(np.int32)
    slot[41], slot[n - 1] = cfg.Nc, -1
    q = ch["q"][:n]
    want, flags = oracle.chunk_causal_attention(q, ch["kc"], ch["vc"], ch["len"], scale, slot=slot,
                                                n_threads=NT, want_flags=True)
    with Ctx(cfg) as c:
        d = chunks_to_dev(ch)
        out = run(c, d, dev_bf16(q), slot=dev_i32(slot), scale=scale)
        assert c.status() == flags == ph.PHOTON_DEV_BAD_INDEX
    got = host_f64(out)
    assert np.all(got[41] == 0) and np.all(got[n - 1] == 0)
    assert_close(got, want, "causal chunk gather")


def test_many_chunks_through_slots_handed_out_from_the_counter(oracle):
    """Enough items for the kernel to hand them out from its global counter (more than 16
    per warp), gathered through a random slot array with repeats and two bad entries;
    twice, so that the counters are seen to be back at zero."""
    cfg = cfg_small(4, B=64)                                  # 2048 chunk buffers, 8 KV heads
    ch = wl.chunk_causal_inputs(cfg, poison=True)
    scale = cfg.dh ** -0.5
    n = 6000                                                  # 48 000 items over at most 1184 warps
    slot = np.random.default_rng(6).integers(0, cfg.Nc, n).astype(np.int32)
    slot[17], slot[n - 2] = -3, cfg.Nc
    q = wl.normal_bf16(4, "qrows_many", (n, ch["rows"], cfg.Hq, cfg.dh))
    pick = np.sort(np.random.default_rng(7).choice(n, 150, replace=False))
    pick[0], pick[1], pick[-1] = 17, n - 2, n - 1
    pick.sort()
    want, flags = oracle.chunk_causal_attention(q[pick], ch["kc"], ch["vc"], ch["len"], scale, slot=slot[pick],
                                                n_threads=NT, want_flags=True)
    with Ctx(cfg, max_queries=n) as c:
        d = chunks_to_dev(ch)
        dq, ds = dev_bf16(q), dev_i32(slot)
        a = run(c, d, dq, slot=ds, scale=scale)
        assert c.status() == flags == ph.PHOTON_DEV_BAD_INDEX
        b = run(c, d, dq, slot=ds, scale=scale, fill=3.0)
        assert c.status() == ph.PHOTON_DEV_BAD_INDEX
    got = host_f64(a)
    assert np.array_equal(host_bits(a), host_bits(b))
    assert np.all(got[17] == 0) and np.all(got[n - 2] == 0)
    assert_close(got[pick], want, "causal chunk, handed out from the counter")


def test_last_row_agrees_with_the_single_query_kernel():
    """The row at position len-1 is what the decode step's chunk attention computes
    for the newest position; two different kernels, same bf16 result up to rounding."""
    cfg = cfg_small(4, B=16)
    ch = wl.chunk_causal_inputs(cfg, poison=True)
    scale = cfg.dh ** -0.5
    last = np.stack([ch["q"][c, ch["len"][c] - 1] for c in range(cfg.Nc)])
    with Ctx(cfg) as c:
        d = chunks_to_dev(ch)
        out = run(c, d, d["q"], scale=scale)
        single = torch.empty(cfg.Nc, cfg.Hq, cfg.dh, dtype=torch.bfloat16, device="cuda")
        ph.photon_chunk_attn(c.h, d["kv"], dev_bf16(last), None, single, scale=scale)
        assert c.status() == 0
    got = host_f64(out)
    rows = np.stack([got[c, ch["len"][c] - 1] for c in range(cfg.Nc)])
    assert np.abs(rows - host_f64(single)).max() <= 2e-2


def test_later_rows_never_reach_earlier_positions_bit_exactly():
    """Causality on the device: overwriting rows > t (and growing len) leaves the
    bf16 outputs of positions <= t bit-identical."""
    cfg = cfg_small(4, B=2)
    ch = wl.chunk_causal_inputs(cfg, full=True)
    scale = cfg.dh ** -0.5
    t = 10
    short = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in ch.items()}
    short["len"] = np.full(cfg.Nc, t + 1, np.int32)
    short["kc"][:, :, t + 1:] = 0x7FC1
    short["vc"][:, :, t + 1:] = 0xFFFF
    with Ctx(cfg) as c:
        a = chunks_to_dev(ch)
        b = chunks_to_dev(short)
        oa, ob = run(c, a, a["q"], scale=scale), run(c, b, b["q"], scale=scale)
        assert c.status() == 0
    ha, hb = host_bits(oa), host_bits(ob)
    assert np.array_equal(ha[:, : t + 1], hb[:, : t + 1])
    assert not hb[:, t + 1:].any()


def test_bad_arguments_are_refused():
    cfg = cfg_small(4, B=1)
    ch = wl.chunk_causal_inputs(cfg)
    with Ctx(cfg) as c:
        d = chunks_to_dev(ch)
        out = torch.empty_like(d["q"])
        for row0, rows in [(-1, 4), (0, 0), (20, 5), (0, 25)]:
            with pytest.raises(ph.PhotonError) as e:
                ph.photon_chunk_causal_attn(c.h, d["kv"], d["q"], None, out, row0=row0, rows=rows)
            assert e.value.code == ph.PHOTON_ERR_INVALID_ARG
        with pytest.raises(ph.PhotonError):
            ph.photon_chunk_causal_attn(c.h, d["kv"], d["q"], None, out, Nc=cfg.Nc + 1)
        ph.photon_chunk_causal_attn(c.h, d["kv"], d["q"], None, out, Nc=0)          # nothing to do
        assert c.status() == 0
