"""The public entry points called the way a host loop without graphs calls them: one call at a
time, each on an idle device, many times over.  Kernels that overlap their predecessor's tail
(programmatic dependent launch) start under other conditions here than inside a replayed graph
or a tight sequence of launches, and a fault that shows once in some tens of such calls does not
show in a parity test that calls once.  Every call must leave the status word clear and, where
the inputs are put back, give the first call's bits."""
import numpy as np
import pytest
import torch

import paper_2512_20687_b200 as ph
from paper_2512_20687_b200 import workloads as wl

from gpu_util import Ctx, chunks_to_dev, coarse_to_dev, dev_bf16

pytestmark = pytest.mark.gpu

CALLS = 120


def bits(t):
    return t.view(torch.int16)


def test_layer_steps_one_at_a_time_on_the_default_workload():
    """STEP of an encoder layer on the coarse caches and of a decoder layer on the chunk buffers
    (64 and 128 rows: the shapes of the default workload), the lengths put back before every call."""
    cfg = wl.CONFIGS[1]
    s = wl.step_inputs(cfg)
    co, chk = s["coarse"], s["chunks"]
    scale = cfg.dh ** -0.5
    li = wl.encoder_layer_inputs(cfg)
    names = ("g1", "wqkv", "wo", "g2", "wgu", "wdown")
    with Ctx(cfg) as c:
        d, dc = coarse_to_dev(co), chunks_to_dev(chk)
        layer = ph.make_layer(*(dev_bf16(li[n]) for n in names), ph.PHOTON_W_IN_MAJOR, li["F"])
        scr = ph.make_layer_scratch(max(cfg.B, cfg.Nc), cfg.Hq, cfg.Hkv, cfg.dh, li["F"], torch.device("cuda"),
                                    torch.bfloat16)
        ex = dev_bf16(li["x"])
        ey, ey0 = torch.empty_like(ex), None
        len0 = d["len"].clone()
        for it in range(CALLS):
            d["len"].copy_(len0)
            torch.cuda.synchronize()
            ph.photon_encoder_step(c.h, layer, scr, ex, d["kv"], ey, scale=scale)
            torch.cuda.synchronize()
            assert c.status() == 0, f"encoder step, call {it}"
            if ey0 is None:
                ey0 = ey.clone()
            assert torch.equal(bits(ey), bits(ey0)), f"encoder step, call {it}"
        gen = torch.Generator(device="cuda")
        gen.manual_seed(5)
        dx = torch.empty(cfg.Nc, cfg.D, dtype=torch.bfloat16, device="cuda").normal_(generator=gen)
        dy, dy0 = torch.empty_like(dx), None
        clen0 = (dc["len"] - 1).clamp(min=0)
        for it in range(CALLS):
            dc["len"].copy_(clen0)
            torch.cuda.synchronize()
            ph.photon_decoder_step(c.h, layer, scr, dx, dc["kv"], dy, scale=scale)
            torch.cuda.synchronize()
            assert c.status() == 0, f"decoder step, call {it}"
            if dy0 is None:
                dy0 = dy.clone()
            assert torch.equal(bits(dy), bits(dy0)), f"decoder step, call {it}"


@pytest.mark.parametrize("idx", [1, 3])
def test_decode_steps_one_at_a_time(idx):
    """The four-part decode step (append folded in or not, a shared prefix with the own keys riding along on
    workload 3), the lengths put back before every call."""
    cfg = wl.CONFIGS[idx]
    s = wl.step_inputs(cfg)
    co, cv, chk = s["coarse"], s["converter"], s["chunks"]
    scale = cfg.dh ** -0.5
    with Ctx(cfg) as c:
        d, dc = coarse_to_dev(co), chunks_to_dev(chk)
        len0 = d["len"].clone()
        out = torch.empty_like(d["q"])
        U = torch.empty(cfg.B, cfg.P, cfg.D, dtype=torch.bfloat16, device="cuda")
        oc = torch.empty_like(dc["q"])
        args = ph.make_step_args(d["kv"], d["k_new"], d["v_new"], d["q"], out, scale, dev_bf16(cv["w_in_major"]),
                                 ph.PHOTON_W_IN_MAJOR, U, cfg.B, chunks=dc["kv"], q_chunk=dc["q"], out_chunk=oc,
                                 Nc=cfg.Nc, scale_chunk=scale)
        first = None
        for it in range(CALLS):
            d["len"].copy_(len0)
            torch.cuda.synchronize()
            ph.photon_decode_step(c.h, args)
            torch.cuda.synchronize()
            assert c.status() == 0, f"decode step, call {it}"
            if first is None:
                first = (out.clone(), U.clone(), oc.clone())
            for got, want in zip((out, U, oc), first):
                assert torch.equal(bits(got), bits(want)), f"decode step, call {it}"
        assert np.array_equal(d["len"].cpu().numpy(), len0.cpu().numpy() + 1)
