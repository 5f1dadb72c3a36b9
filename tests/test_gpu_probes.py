"""The two aids beside the decode step: the read-ceiling probe must bring in every byte it is asked for, and
the wait probe must show that a bounded wait which runs out ends in a status bit, not in a hung kernel, and
that the context is usable afterwards."""
import numpy as np
import pytest
import torch

import paper_2512_20687_b200 as ph
from paper_2512_20687_b200 import workloads as wl

from gpu_util import Ctx, assert_close, coarse_to_dev, host_f64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("nbytes,ctas", [(16, 0), (32768, 1), (32768 * 5 + 4096 + 16, 3), (70 * 1000 * 1000 - 1000 * 1000 % 16, 0),
                                         (64 << 20, 296), (64 << 20, 148)])
def test_read_probe_sees_every_byte(nbytes, ctas):
    cfg = wl.CONFIGS[0]
    nbytes -= nbytes % 16
    g = torch.Generator(device="cuda")
    g.manual_seed(nbytes % 1000 + ctas)
    buf = torch.randint(-2 ** 31, 2 ** 31 - 1, (nbytes // 4 + 64,), dtype=torch.int32, device="cuda", generator=g)
    total = torch.zeros(1, dtype=torch.int32, device="cuda")
    with Ctx(cfg) as c:
        ph.photon_read_probe(c.h, buf, nbytes, ctas, total)
        ph.photon_read_probe(c.h, buf, nbytes, ctas, total)          # twice: the sum doubles
        assert c.status() == 0
    words = buf[:nbytes // 4][::32].to(torch.int64).sum().item()       # first word of every 128 bytes
    assert (int(total.item()) - 2 * words) % 2 ** 32 == 0


def test_read_probe_rejects_bad_arguments():
    cfg = wl.CONFIGS[0]
    buf = torch.zeros(1024, dtype=torch.int32, device="cuda")
    with Ctx(cfg) as c:
        for args in ((buf, 24, 0), (buf, 32, -1)):
            with pytest.raises(ph.PhotonError) as e:
                ph.photon_read_probe(c.h, *args)
            assert e.value.code == ph.PHOTON_ERR_INVALID_ARG
        with pytest.raises(ph.PhotonError):
            ph.photon_read_probe(c.h, buf.view(torch.uint8)[4:], 32, 0)     # misaligned
        assert c.status() == 0


def test_a_wait_that_runs_out_sets_the_status_bit_and_leaves_the_context_usable(oracle):
    cfg = wl.scaled(wl.CONFIGS[1], B=5, S=700)
    co = wl.coarse_inputs(cfg, poison=True)
    co["len"] = np.array([699, 0, 64, 300, 513], np.int32)
    for u, n in enumerate(co["len"]):
        co["k"][u, :, n:] = 0x7FC1
        co["v"][u, :, n:] = 0x7FC1
    scale = cfg.dh ** -0.5
    want, _ = oracle.attention(co["q"], co["k"], co["v"], co["len"], scale, n_threads=16)
    with Ctx(cfg) as c:
        ph.photon_set_attention_ctas(c.h, 37)                            # unit 0 is cut: its ticket is used
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        ph.photon_wait_probe(c.h, 1_000_000)                             # gives up after a millisecond
        t1.record()
        assert c.status(clear=False) == ph.PHOTON_DEV_TIMEOUT            # the kernel came back by itself
        assert 0.5 < t0.elapsed_time(t1) < 500.0
        assert c.status() == ph.PHOTON_DEV_TIMEOUT                       # read and cleared, tickets back to zero
        assert c.status() == 0
        d = coarse_to_dev(co)
        out = torch.empty_like(d["q"])
        ph.photon_coarse_attn(c.h, d["kv"], d["q"], out, None, scale)
        assert c.status() == 0
        assert_close(host_f64(out), want, "after a wait that ran out")
        with pytest.raises(ph.PhotonError):
            ph.photon_wait_probe(c.h, 10 ** 9)                           # limits beyond a tenth of a second are refused
