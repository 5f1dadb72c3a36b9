"""photon_coarse_attn_noalloc: the context-free coarse attention for callers that cannot allocate
device memory (its workspace is an array inside the library image).  Called through the C boundary
twice in a row and compared with photon_coarse_attn and with the CPU oracle on the same inputs.
Collected last on purpose."""
import numpy as np
import pytest
import torch

import paper_2512_20687_b200 as ph
from paper_2512_20687_b200 import workloads as wl

from gpu_util import Ctx, assert_close, coarse_to_dev, host_f64

pytestmark = pytest.mark.gpu


def _inputs(seed_shift):
    cfg = wl.scaled(wl.CONFIGS[1], B=11, S=900, seed=100 + seed_shift)
    co = wl.coarse_inputs(cfg, poison=True)
    lens = np.array([899, 0, 1, 63, 64, 65, 300, 512, 700, 128, 898], np.int32)
    for u, n in enumerate(lens):
        co["k"][u, :, n:] = 0x7FC1
        co["v"][u, :, n:] = 0x7FC1
    co["len"] = lens
    return cfg, co


def test_no_alloc_entry_point_matches_the_context_one_twice_in_a_row(oracle):
    for call in range(2):                                  # second call finds the first one's leftovers
        cfg, co = _inputs(call)
        scale = cfg.dh ** -0.5
        d = coarse_to_dev(co)
        want = torch.empty_like(d["q"])
        want_lse = torch.empty(cfg.B, cfg.Hq, dtype=torch.float32, device="cuda")
        with Ctx(cfg) as c:
            ph.photon_coarse_attn(c.h, d["kv"], d["q"], want, want_lse, scale)
            assert c.status() == 0
        got = torch.full_like(d["q"], 7.0)
        got_lse = torch.full_like(want_lse, 7.0)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        ph.photon_coarse_attn_noalloc(cfg.Hq, cfg.Hkv, cfg.dh, d["kv"], d["q"], got, got_lse, scale, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert_close(host_f64(got), host_f64(want), f"no-alloc call {call}")
        a, b = got_lse.cpu().numpy(), want_lse.cpu().numpy()
        assert np.array_equal(np.isneginf(a), np.isneginf(b))
        fin = np.isfinite(b)
        assert np.abs(a[fin] - b[fin]).max() < 2e-3
        assert np.all(host_f64(got)[1] == 0)               # the empty unit
        ref, ref_lse = oracle.attention(co["q"], co["k"], co["v"], co["len"], scale, n_threads=16)
        assert_close(host_f64(got), ref, f"no-alloc call {call} against the oracle")
        assert np.abs(a[fin] - ref_lse[fin]).max() < 2e-3


def test_no_alloc_entry_point_allocates_nothing_and_takes_wide_groups(oracle):
    """Sixteen query heads per KV head of 64 features and one long unit among short ones, so that many CTAs
    hold a piece of the same cache and both partial slots of a CTA are in use; the status word is the one
    inside the array (dev_status = None).  Once the first call has looked up the array, a call leaves the
    device's free memory and torch's own counters where they were."""
    Hkv, G, dh = 2, 16, 64
    cfg = wl.scaled(wl.CONFIGS[1], B=6, S=6000, Hq=G * Hkv, Hkv=Hkv, dh=dh, D=G * Hkv * dh, seed=321)
    co = wl.coarse_inputs(cfg, poison=True)
    lens = np.array([5999, 3, 70, 0, 129, 640], np.int32)
    for u, n in enumerate(lens):
        co["k"][u, :, n:] = 0x7FC1
        co["v"][u, :, n:] = 0x7FC1
    co["len"] = lens
    scale = dh ** -0.5
    d = coarse_to_dev(co)
    got = torch.empty_like(d["q"])
    ph.photon_coarse_attn_noalloc(cfg.Hq, Hkv, dh, d["kv"], d["q"], got, None, scale)      # looks the array up
    torch.cuda.synchronize()
    free0, alloc0, reserved0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    got.fill_(7.0)
    ph.photon_coarse_attn_noalloc(cfg.Hq, Hkv, dh, d["kv"], d["q"], got, None, scale)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
    want, _ = oracle.attention(co["q"], co["k"], co["v"], lens, scale, n_threads=16)
    assert_close(host_f64(got), want, "no-alloc, G = 16, dh = 64")


def test_no_alloc_entry_point_rejects_sizes_beyond_its_array():
    cfg, co = _inputs(0)
    d = coarse_to_dev(co)
    out = torch.empty_like(d["q"])
    kv = d["kv"]
    real = kv.n_units
    kv.n_units = 16384 // cfg.Hkv + 1                      # one (unit, KV head) pair too many
    with pytest.raises(ph.PhotonError) as e:
        ph.photon_coarse_attn_noalloc(cfg.Hq, cfg.Hkv, cfg.dh, kv, d["q"], out, None, 1.0)
    assert e.value.code == ph.PHOTON_ERR_WORKSPACE
    kv.n_units = real
