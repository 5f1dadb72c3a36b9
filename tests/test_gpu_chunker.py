"""Parity of the context chunker's two kernels (row normalisation, linear map on
the tensor cores incl. its split of K over a cluster) with the CPU oracle, through
the C boundary.  bf16 outputs: max abs error 2e-2, mean abs error 2e-3 against the
fp64 oracle on the same bf16 inputs."""
import numpy as np
import pytest
import torch

import paper_2512_20687_b200 as ph
from paper_2512_20687_b200 import workloads as wl

from gpu_util import Ctx, assert_close, dev_bf16, host_bits, host_f64

pytestmark = pytest.mark.gpu

NT = 16     # oracle threads


def cfg_small(i, **kw):
    return wl.scaled(wl.CONFIGS[i], **kw)


@pytest.mark.parametrize("rows,cols,with_gamma", [(64, 8192, True), (5, 4096, False), (3, 8, True), (130, 1032, True),
                                                  (3000, 1032, True), (1025, 2048, False), (1500, 8, True)])
def test_rmsnorm_matches_oracle(oracle, rows, cols, with_gamma):
    x = wl.normal_bf16(21, "x", (rows, cols), std=3.0)
    g = wl.f32_to_bf16_bits((wl.bf16_bits_to_f64(wl.normal_bf16(21, "g", (cols,), std=0.2)) + 1.0).astype(np.float32))
    want = oracle.rmsnorm(x, g if with_gamma else None, eps=1e-5)
    with Ctx(cfg_small(0)) as c:
        dx = dev_bf16(x)
        out = torch.full_like(dx, 9.0)
        ph.photon_rmsnorm(c.h, dx, dev_bf16(g) if with_gamma else None, 1e-5, out)
        assert c.status() == 0
        inplace = dx.clone()
        ph.photon_rmsnorm(c.h, inplace, dev_bf16(g) if with_gamma else None, 1e-5, inplace)
        assert c.status() == 0
    assert_close(host_f64(out), want, f"rmsnorm {rows}x{cols}")
    assert np.array_equal(host_bits(out), host_bits(inplace))
    # bf16 rounding of an O(1) value: within one bf16 step of the oracle's own rounding
    assert np.abs(host_f64(out) - wl.bf16_bits_to_f64(oracle.round_bf16(want))).max() <= 2.0 ** -6


# (B, K, N): the 1B-class chunker (4 CTAs share a tile), the chunk-parallel one (wide batch),
# a tile count that needs no split, odd batch sizes, the smallest K that is still split, K too short to split
# and more narrow tiles than SMs (wider slabs, one wave)
SHAPES = [(64, 8192, 2048), (512, 4096, 1024), (64, 2048, 8192), (1, 1024, 64), (130, 1024, 128),
          (17, 512, 64), (200, 4096, 256), (64, 1024, 11264), (130, 512, 6400),
          # thousands of rows: the persistent kernel (one to several tiles per CTA, a ragged last row tile)
          (9000, 512, 1280), (16384, 256, 768), (4100, 192, 2816)]


@pytest.mark.parametrize("B,K,N", SHAPES)
@pytest.mark.parametrize("out_major", [False, True])
def test_linear_matches_oracle(oracle, B, K, N, out_major):
    x = wl.normal_bf16(22, "x", (B, K))
    w = wl.normal_bf16(22, "w", (K, N), std=K ** -0.5)
    bias = wl.normal_bf16(22, "b", (N,), std=0.5)
    wm = np.ascontiguousarray(w.T) if out_major else w
    want = oracle.linear(x, wm, bias, w_out_major=out_major, n_threads=NT)
    with Ctx(cfg_small(0)) as c:
        y = torch.full((B, N), 7.0, dtype=torch.bfloat16, device="cuda")
        layout = ph.PHOTON_W_OUT_MAJOR if out_major else ph.PHOTON_W_IN_MAJOR
        ph.photon_linear(c.h, dev_bf16(x), dev_bf16(wm), layout, dev_bf16(bias), y)
        y2 = torch.empty_like(y)
        ph.photon_linear(c.h, dev_bf16(x), dev_bf16(wm), layout, dev_bf16(bias), y2)
        assert c.status() == 0
    assert np.array_equal(host_bits(y), host_bits(y2))                  # the split of K adds in a fixed order
    assert_close(host_f64(y), want, f"linear {B}x{K}x{N}")


def test_linear_with_more_tiles_than_sms_repeated_on_an_idle_device():
    """128 rows and 176 slabs of 64 output columns (the gate/up projection of a layer step on 128 chunks): 200 calls, each on
    an idle device with another kernel run in between, as a caller that launches one operation at a time does.
    Every call gives the first call's bits and leaves the status word clear.  (A form of this kernel that put
    two CTAs on an SM for such tile counts gave up on a wait, or failed, once in some tens of such calls.)"""
    B, K, N = 128, 2048, 11264
    x = dev_bf16(wl.normal_bf16(25, "x", (B, K)))
    w = dev_bf16(wl.normal_bf16(25, "w", (K, N), std=K ** -0.5))
    with Ctx(cfg_small(0)) as c:
        y0 = torch.empty((B, N), dtype=torch.bfloat16, device="cuda")
        ph.photon_linear(c.h, x, w, ph.PHOTON_W_IN_MAJOR, None, y0)
        torch.cuda.synchronize()
        y, n = torch.empty_like(y0), torch.empty_like(x)
        for _ in range(200):
            ph.photon_rmsnorm(c.h, x, None, 1e-5, n)
            torch.cuda.synchronize()
            ph.photon_linear(c.h, x, w, ph.PHOTON_W_IN_MAJOR, None, y)
            torch.cuda.synchronize()
            assert c.status() == 0
            assert torch.equal(y.view(torch.int16), y0.view(torch.int16))


def test_large_tile_kernel_adds_bias_and_residual_and_is_deterministic(oracle):
    """Thousands of rows with bias and a residual that aliases the output; the oracle
    recomputes a sample of rows; two calls give the same bits."""
    B, K, N = 6000, 320, 1792
    x = wl.normal_bf16(24, "x", (B, K))
    w = wl.normal_bf16(24, "w", (K, N), std=K ** -0.5)
    bias, res = wl.normal_bf16(24, "b", (N,), std=0.5), wl.normal_bf16(24, "r", (B, N))
    pick = np.sort(np.random.default_rng(3).choice(B, 200, replace=False))
    pick[0], pick[-1] = 0, B - 1
    want = oracle.linear(x[pick], w, bias, n_threads=NT) + wl.bf16_bits_to_f64(res[pick])
    with Ctx(cfg_small(0)) as c:
        dx, dw, db = dev_bf16(x), dev_bf16(w), dev_bf16(bias)
        y1, y2 = dev_bf16(res).clone(), dev_bf16(res).clone()
        ph.photon_linear(c.h, dx, dw, ph.PHOTON_W_IN_MAJOR, db, y1, residual=y1)
        ph.photon_linear(c.h, dx, dw, ph.PHOTON_W_IN_MAJOR, db, y2, residual=y2)
        assert c.status() == 0
    assert np.array_equal(host_bits(y1), host_bits(y2))
    assert_close(host_f64(y1)[pick], want, "large tiles, bias + residual")


def test_linear_one_hot_rows_return_weight_rows_bit_exactly():
    K, N = 4096, 128                                                     # split over a cluster
    w = wl.normal_bf16(23, "w", (K, N))
    x = np.zeros((64, K), np.float32)
    ks = np.arange(64) * 61 % K
    x[np.arange(64), ks] = 1.0
    with Ctx(cfg_small(0)) as c:
        y = torch.empty((64, N), dtype=torch.bfloat16, device="cuda")
        ph.photon_linear(c.h, dev_bf16(wl.f32_to_bf16_bits(x)), dev_bf16(w), ph.PHOTON_W_IN_MAJOR, None, y)
        assert c.status() == 0
    assert np.array_equal(host_bits(y), w[ks])


@pytest.mark.parametrize("idx", [0, 1, 4])
def test_chunker_matches_oracle(oracle, idx):
    """Normalise, then project: the two calls in a row on the workload's shapes."""
    cfg = wl.CONFIGS[idx]
    ci = wl.chunker_inputs(cfg)
    xn_want, want = oracle.chunker(ci["x"], ci["gamma"], ci["eps"], ci["w_in_major"], ci["bias"], n_threads=NT)
    with Ctx(cfg) as c:
        x = dev_bf16(ci["x"])
        xn = torch.empty_like(x)
        y = torch.empty((cfg.B, cfg.D), dtype=torch.bfloat16, device="cuda")
        ph.photon_rmsnorm(c.h, x, dev_bf16(ci["gamma"]), ci["eps"], xn)
        ph.photon_linear(c.h, xn, dev_bf16(ci["w_in_major"]), ph.PHOTON_W_IN_MAJOR, dev_bf16(ci["bias"]), y)
        assert c.status() == 0
    assert_close(host_f64(y), want, f"chunker cfg{idx}")
    assert np.abs(host_f64(xn) - wl.bf16_bits_to_f64(xn_want)).max() <= 2.0 ** -6


def test_bad_arguments_are_refused():
    with Ctx(cfg_small(0)) as c:
        x = torch.zeros((4, 128), dtype=torch.bfloat16, device="cuda")
        w = torch.zeros((128, 64), dtype=torch.bfloat16, device="cuda")
        y = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
        for K, N in [(100, 64), (128, 32), (0, 64)]:
            with pytest.raises(ph.PhotonError) as e:
                ph.photon_linear(c.h, x, w, ph.PHOTON_W_IN_MAJOR, None, y, K=K, N=N)
            assert e.value.code == ph.PHOTON_ERR_INVALID_ARG
        with pytest.raises(ph.PhotonError):
            ph.photon_linear(c.h, x, w, 7, None, y)
        with pytest.raises(ph.PhotonError):
            ph.photon_rmsnorm(c.h, x, None, 1e-5, x, cols=12)
        with pytest.raises(ph.PhotonError):
            ph.photon_rmsnorm(c.h, x, None, -1.0, x)
        ph.photon_linear(c.h, x, w, ph.PHOTON_W_IN_MAJOR, None, y, B=0)
        ph.photon_rmsnorm(c.h, x, None, 0.0, x, rows=0)
        assert c.status() == 0
