"""Helpers for the GPU parity tests: move seeded numpy inputs to the device,
call the library through its binding, bring results back as float64."""
import numpy as np
import torch

import paper_2512_20687_b200 as ph
from paper_2512_20687_b200 import workloads as wl

MAX_ABS, MEAN_ABS = 2e-2, 2e-3          # bf16 output vs fp64 oracle on bf16-rounded inputs


def dev_bf16(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda().view(torch.bfloat16)


def dev_i32(a) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()


def host_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def host_f64(t: torch.Tensor) -> np.ndarray:
    return wl.bf16_bits_to_f64(host_bits(t))


def assert_close(got_f64: np.ndarray, want_f64: np.ndarray, what: str = ""):
    assert got_f64.shape == want_f64.shape, (got_f64.shape, want_f64.shape)
    assert np.isfinite(got_f64).all(), f"{what}: non-finite output"
    err = np.abs(got_f64 - want_f64)
    assert err.max() <= MAX_ABS, f"{what}: max abs err {err.max():.4g} > {MAX_ABS}"
    assert err.mean() <= MEAN_ABS, f"{what}: mean abs err {err.mean():.4g} > {MEAN_ABS}"


def assert_close_scaled(got_f64: np.ndarray, want_f64: np.ndarray, what: str = "", slack: float = 1.0):
    """The same bar for values that leave the range the bar was set for: 2e-2 covers the
    bf16 rounding of magnitudes up to 2 with a margin; a value of magnitude m > 2 has a bf16
    step m/2 times larger, so its bound grows by that factor.  Rounding a value to bf16 alone
    costs a quarter of its bf16 step on average (about 2e-3 already for magnitudes between 1
    and 2), so the mean bound is the usual 2e-3 or twice that pure-rounding mean, whichever
    is larger: chained roundings may cost as much again as the last one.  `slack` widens
    both bounds for the outputs of a chain of kernels, where a one-step difference in an
    intermediate of magnitude m moves what depends on it by up to m * 2^-7."""
    assert got_f64.shape == want_f64.shape, (got_f64.shape, want_f64.shape)
    assert np.isfinite(got_f64).all(), f"{what}: non-finite output"
    err = np.abs(got_f64 - want_f64)
    bound = slack * MAX_ABS * np.maximum(1.0, np.abs(want_f64) / 2.0)
    worst = (err / bound).max()
    assert worst <= 1.0, f"{what}: abs err reaches {worst:.3g} of its bound"
    step = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(want_f64), 2.0 ** -20))) - 7)
    mean_bound = slack * max(MEAN_ABS, 0.5 * float(step.mean()))
    assert err.mean() <= mean_bound, f"{what}: mean abs err {err.mean():.4g} > {mean_bound:.4g}"


class Ctx:
    def __init__(self, cfg, max_queries=None, max_splits=0):
        self.cfg = cfg
        mq = max_queries or max(cfg.B, cfg.Nc)
        self.h = ph.photon_create(cfg.Hq, cfg.Hkv, cfg.dh, cfg.D, cfg.P, cfg.C, mq, max_splits)

    def __enter__(self):
        return self

    def __exit__(self, *a):
        torch.cuda.synchronize()
        ph.photon_destroy(self.h)

    def status(self, clear=True):
        return ph.photon_device_status(self.h, clear)


def coarse_to_dev(co: dict):
    d = {k: (dev_bf16(v) if isinstance(v, np.ndarray) and v.dtype == np.uint16 else v) for k, v in co.items()}
    d["len"] = dev_i32(co["len"])
    kw = {}
    if "k_shared" in co:
        d["shared_len"], d["shared_id"] = dev_i32(co["shared_len"]), dev_i32(co["shared_id"])
        kw = dict(k_shared=d["k_shared"], v_shared=d["v_shared"], shared_len=d["shared_len"],
                  shared_id=d["shared_id"])
    d["kv"] = ph.make_kv(d["k"], d["v"], d["len"], **kw)
    return d


def chunks_to_dev(ch: dict):
    d = {"kc": dev_bf16(ch["kc"]), "vc": dev_bf16(ch["vc"]), "q": dev_bf16(ch["q"]),
         "len": dev_i32(ch["len"])}
    d["kv"] = ph.make_kv(d["kc"], d["vc"], d["len"])
    return d


def shared_of(co: dict):
    if "k_shared" not in co:
        return None
    return {"k": co["k_shared"], "v": co["v_shared"], "len": co["shared_len"], "id": co["shared_id"]}
