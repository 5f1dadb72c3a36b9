"""A paged coarse cache gives the results of the contiguous cache it stands for:
append bit-exactly, attention within the usual bar of the CPU oracle (which sees the
contiguous cache; a paged cache is a storage layout, not another computation)."""
import numpy as np
import pytest
import torch

import paper_2512_20687_b200 as ph
from paper_2512_20687_b200 import workloads as wl

from gpu_util import Ctx, assert_close, dev_bf16, dev_i32, host_bits, host_f64

pytestmark = pytest.mark.gpu

NT = 16


def cfg_small(i, **kw):
    return wl.scaled(wl.CONFIGS[i], **kw)


def to_pages(a, table, page_rows, n_pages, fill):
    """Contiguous [n_units, Hkv, cap, dh] -> pool [n_pages, Hkv, page_rows, dh] through the table."""
    n_units, Hkv, cap, dh = a.shape
    pool = np.full((n_pages, Hkv, page_rows, dh), fill, np.uint16)
    for u in range(n_units):
        for j in range(table.shape[1]):
            pool[table[u, j]] = a[u, :, j * page_rows:(j + 1) * page_rows]
    return pool


def from_pages(pool, table, page_rows):
    n_units, ppu = table.shape
    return np.concatenate([pool[table[:, j]] for j in range(ppu)], axis=2)


@pytest.mark.parametrize("idx,B,S,page_rows", [(1, 9, 701, 64), (1, 64, 512, 128), (4, 40, 128, 64), (0, 2, 16, 64)])
def test_paged_append_and_attention(oracle, idx, B, S, page_rows):
    cfg = cfg_small(idx, B=B, S=S)
    co = wl.coarse_inputs(cfg, poison=True)
    ppu = -(-S // page_rows)
    cap = ppu * page_rows
    lens = np.array([max(0, S - 1 - 37 * (u % 5)) for u in range(B)], np.int32)
    lens[0] = S - 1
    if B > 2:
        lens[1], lens[2] = 0, page_rows - 1                      # an empty unit; an append that fills a page
    pad = lambda a: np.concatenate([a, np.full(a.shape[:2] + (cap - S, a.shape[3]), 0x7FC1, np.uint16)], axis=2)
    k, v = pad(co["k"]), pad(co["v"])
    for u, n in enumerate(lens):
        k[u, :, n:] = 0x7FC1
        v[u, :, n:] = 0xFFC1
    n_pages = B * ppu + 3
    table = np.random.default_rng(idx).permutation(n_pages)[: B * ppu].reshape(B, ppu).astype(np.int32)
    scale = cfg.dh ** -0.5
    ok, ov, ol = k.copy(), v.copy(), lens.copy()
    assert oracle.kv_append(ok, ov, ol, co["k_new"], co["v_new"]) == 0
    want, want_lse = oracle.attention(co["q"], ok, ov, ol, scale, n_threads=NT)
    with Ctx(cfg) as c:
        pk, pv = dev_bf16(to_pages(k, table, page_rows, n_pages, 0x7FC1)), dev_bf16(to_pages(v, table, page_rows, n_pages, 0x7FC1))
        dl = dev_i32(lens)
        kv = ph.make_kv(pk, pv, dl, page_table=dev_i32(table))
        assert kv.cap == cap and kv.n_units == B
        ph.photon_kv_append(c.h, kv, dev_bf16(co["k_new"]), dev_bf16(co["v_new"]))
        q = dev_bf16(co["q"])
        out = torch.empty_like(q)
        lse = torch.empty(B, cfg.Hq, dtype=torch.float32, device="cuda")
        ph.photon_coarse_attn(c.h, kv, q, out, lse, scale)
        out2 = torch.empty_like(q)
        ph.photon_flat_attn(c.h, kv, q, out2, None, scale)
        assert c.status() == 0
        assert np.array_equal(dl.cpu().numpy(), ol)
        gk, gv = from_pages(host_bits(pk), table, page_rows), from_pages(host_bits(pv), table, page_rows)
        assert np.array_equal(gk, ok) and np.array_equal(gv, ov)         # the append wrote the right page, bit-exactly
    assert_close(host_f64(out), want, "paged coarse attention")
    assert np.array_equal(host_bits(out), host_bits(out2))
    fin = np.isfinite(want_lse)
    assert np.abs(lse.cpu().numpy()[fin] - want_lse[fin]).max() < 2e-3


def test_paged_and_contiguous_give_the_same_bits():
    cfg = cfg_small(1, B=16, S=8192)
    co = wl.coarse_inputs(cfg)
    page_rows, ppu = 256, 32
    n_pages = cfg.B * ppu
    table = np.random.default_rng(7).permutation(n_pages).reshape(cfg.B, ppu).astype(np.int32)
    scale = cfg.dh ** -0.5
    with Ctx(cfg) as c:
        q = dev_bf16(co["q"])
        a, b = torch.empty_like(q), torch.empty_like(q)
        dl = dev_i32(co["len"])
        ph.photon_coarse_attn(c.h, ph.make_kv(dev_bf16(co["k"]), dev_bf16(co["v"]), dl), q, a, None, scale)
        pk, pv = dev_bf16(to_pages(co["k"], table, page_rows, n_pages, 0)), dev_bf16(to_pages(co["v"], table, page_rows, n_pages, 0))
        ph.photon_coarse_attn(c.h, ph.make_kv(pk, pv, dl, page_table=dev_i32(table)), q, b, None, scale)
        assert c.status() == 0
    assert np.array_equal(host_bits(a), host_bits(b))                    # the same tiles in the same order


def test_bad_pages_and_calls_that_do_not_take_pages():
    cfg = cfg_small(0, B=2, S=16)
    co = wl.coarse_inputs(cfg)
    pool = np.zeros((3, cfg.Hkv, 64, cfg.dh), np.uint16)
    with Ctx(cfg) as c:
        pk, pv, dl = dev_bf16(pool), dev_bf16(pool), dev_i32(co["len"])
        kv = ph.make_kv(pk, pv, dl, page_table=dev_i32(np.array([[1], [5]], np.int32)))
        ph.photon_kv_append(c.h, kv, dev_bf16(co["k_new"]), dev_bf16(co["v_new"]))
        assert c.status() == ph.PHOTON_DEV_BAD_INDEX                      # unit 1 names page 5 of 3
        assert list(dl.cpu().numpy()) == [co["len"][0] + 1, co["len"][1]]
        q = dev_bf16(co["q"])
        out = torch.empty_like(q)
        ph.photon_coarse_attn(c.h, kv, q, out, None, 1.0)
        assert c.status() == ph.PHOTON_DEV_BAD_INDEX and np.isfinite(host_f64(out)).all()
        q1, o1 = q.unsqueeze(1).contiguous(), out.unsqueeze(1).contiguous()
        for call in (lambda: ph.photon_chunk_attn(c.h, kv, q, None, out),
                     lambda: ph.photon_chunk_causal_attn(c.h, kv, q1, None, o1)):
            with pytest.raises(ph.PhotonError) as e:
                call()
            assert e.value.code == ph.PHOTON_ERR_INVALID_ARG
        kv.page_rows = 48                                                 # not a multiple of 64
        with pytest.raises(ph.PhotonError):
            ph.photon_coarse_attn(c.h, kv, q, out, None, 1.0)
