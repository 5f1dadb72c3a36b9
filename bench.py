#!/usr/bin/env python
"""Benchmark of the PHOTON decode step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--impl reference]

A step is one pass of the whole hot path (append -> coarse attention ->
converter -> chunk attention) over one batch of seeded synthetic input.  The
metric is decode tokens/s = token-level in-flight chunks per step / step time.
With N > 1 every rank runs an independent replica of the same per-GPU batch
(weak scaling, no data-path collective); time is the max over ranks.  Under
torchrun the ranks are there already; started plainly with --gpus N > 1 the
script starts them itself (torch.distributed.run on 127.0.0.1).  Rank 0 prints
ONE JSON line.  The K timed steps are repeated a few times and the median
repetition is reported.

`--impl reference` times the CPU oracle (a deliberately plain fp64 program)
on the host cores on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2512_20687_b200 import workloads as wl  # noqa: E402

METRIC, UNIT = "decode_tokens_per_s", "tokens/s"
L2_BYTES = 126 * 1000 * 1000


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=200)
    ap.add_argument("--config", type=int, default=1, help="index into the five workload configurations")
    ap.add_argument("--impl", default="photon", choices=["photon", "reference"])
    ap.add_argument("--layout", default="out_major", choices=["out_major", "in_major"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-parts", action="store_true")
    ap.add_argument("--only-this-workload", action="store_true",
                    help="skip the other target workloads' attention parts and the read-ceiling probe (profiler captures)")
    ap.add_argument("--max-splits", type=int, default=0)
    ap.add_argument("--hierarchy", default="",
                    help="chunk lengths C_1,...,C_L instead of 4,4 (e.g. 2,2): same model and context, other stream lengths")
    ap.add_argument("--attention-ctas", type=int, default=0,
                    help="persistent grid of the coarse attention (0: the library's choice)")
    ap.add_argument("--batch", type=int, default=0,
                    help="shrink the workload to this many sequences (for profiler captures of a small case)")
    return ap.parse_args()


def workload_desc(cfg) -> dict:
    full = wl.CONFIGS[cfg.index].B
    d = {"workload": f"config {cfg.index} ({cfg.name}{'' if cfg.B == full else f', REDUCED from batch {full}'}): batch {cfg.B}, context {cfg.context} tokens -> "
                     f"{cfg.S} coarse latents, {cfg.Hq}q/{cfg.Hkv}kv heads x {cfg.dh}, d_model {cfg.D}, "
                     f"converter {cfg.D}->{cfg.P}x{cfg.D}, chunk attention P={cfg.P} C={cfg.C}, "
                     f"{cfg.chunks_per_seq} in-flight chunks per sequence",
         "batch": cfg.B, "coarse_len": cfg.S, "context": cfg.context, "seed": cfg.seed, "tokens_per_coarse_latent": cfg.compress,
         "tokens_per_step": cfg.tokens_per_step}
    if cfg.shared_S:
        d["shared_prefix_len"] = cfg.shared_S
    return d


# --------------------------------------------------------------------------- CPU oracle arm

def oracle_sample(cfg, seconds: float, threads: int):
    """The first b sequences (and their chunks) of the workload, b sized so that
    one oracle step costs about `seconds` of wall time on `threads` cores."""
    flops = (cfg.B * cfg.Hq * (cfg.S + cfg.shared_S) * cfg.dh * 4 + 2.0 * cfg.B * cfg.D * cfg.P * cfg.D
             + cfg.Nc * cfg.Hq * (cfg.P + cfg.C) * cfg.dh * 4)
    rate = 0.25e9 * max(1, threads)                      # plain fp64 loops: ~0.25 Gflop/s per core
    b = int(max(1, min(cfg.B, cfg.B * seconds * rate / flops)))
    sub = wl.scaled(cfg, B=b)
    s = wl.step_inputs(sub)
    return sub, s


def time_oracle_step(cfg, sample_cfg, s, threads: int) -> float:
    from oracle import photon_oracle as oracle
    co = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in s["coarse"].items()}
    scale = cfg.dh ** -0.5
    t0 = time.perf_counter()
    oracle.decode_step(co, s["converter"], s["chunks"], scale, scale, chain=True, w_out_major=True,
                       n_threads=threads)
    return time.perf_counter() - t0


def cpu_baseline(cfg, seconds: float = 10.0) -> dict:
    """The oracle as it stands on all host cores: whole decode steps on a bounded sample of the workload
    (the first b sequences, b sized for about `seconds` of wall time per step at most), repeated until
    about 1.5 s of wall time (some 10-30 core-seconds) have gone by."""
    from oracle import photon_oracle as oracle
    threads = oracle.hardware_threads() or os.cpu_count() or 1
    sub, s = oracle_sample(cfg, seconds, threads)
    time_oracle_step(cfg, sub, s, threads)                        # first touch of the pages
    times = []
    while sum(times) < 1.5 and len(times) < 50:
        times.append(time_oracle_step(cfg, sub, s, threads))
    dt = sum(times) / len(times)
    tokens = cfg.tokens_per_step * sub.B / cfg.B
    # the same program on one core, on a sample sized for about 2 s per step
    sub1, s1 = oracle_sample(cfg, 2.0, 1)
    time_oracle_step(cfg, sub1, s1, 1)
    dt1 = time_oracle_step(cfg, sub1, s1, 1)
    return {"value": tokens / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{len(times)} decode steps of the first {sub.B} of {cfg.B} sequences "
                      f"({sub.Nc} chunks), {dt:.3f} s each, {sum(times) * threads:.0f} core-seconds",
            "single_thread": {"value": cfg.tokens_per_step * sub1.B / cfg.B / dt1, "unit": UNIT,
                              "sample": f"one decode step of the first {sub1.B} of {cfg.B} sequences, {dt1:.3f} s"},
            "hardware_threads": threads}


def run_reference(args, cfg) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import photon_oracle as oracle
    oracle.build()
    threads = oracle.hardware_threads() or os.cpu_count() or 1
    per_step = max(0.05, min(10.0, 150.0 / max(1, args.steps + args.warmup)))
    sub, s = oracle_sample(cfg, per_step, threads)
    for _ in range(args.warmup):
        time_oracle_step(cfg, sub, s, threads)
    times = [time_oracle_step(cfg, sub, s, threads) for _ in range(args.steps)]
    dt = sum(times) / len(times)
    tokens = cfg.tokens_per_step * sub.B / cfg.B
    val = tokens / dt
    sample = (f"each step = one oracle decode step of the first {sub.B} of {cfg.B} sequences "
              f"({sub.Nc} chunks)")
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3 * cfg.B / sub.B,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_desc(cfg),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- GPU arm

class ClockSampler:
    """nvidia-smi clock/throttle samples taken while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.uuid, self.proc, self.f = uuid, None, None

    def start(self):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.uuid, f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        self.f.flush()
        self.f.seek(0)
        rows = [r.strip().split(", ") for r in self.f.read().splitlines() if r.strip()]
        self.f.close()
        os.unlink(self.f.name)
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 8:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); power.append(float(r[2]))
            except ValueError:
                continue
            for n, v in zip(names, r[4:8]):
                if v.strip().lower() == "active":
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power)}


def run_gpu(args, cfg) -> None:
    import torch

    import paper_2512_20687_b200 as ph
    from paper_2512_20687_b200 import dist as pd

    rank, local_rank, world = pd.init()
    torch.cuda.set_device(local_rank if world > 1 else 0)
    dev = torch.device("cuda", torch.cuda.current_device())
    ph.load()

    out_major = args.layout == "out_major"
    layout = ph.PHOTON_W_OUT_MAJOR if out_major else ph.PHOTON_W_IN_MAJOR
    scale = cfg.dh ** -0.5
    s = wl.step_inputs(cfg)
    co, cv, ch = s["coarse"], s["converter"], s["chunks"]

    def dev_bf16(a):
        return torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)

    coarse_bytes = wl.coarse_kv_bytes(cfg)
    chunk_bytes = wl.chunk_kv_bytes(cfg, ch["len"])
    w_bytes = cv["w_in_major"].nbytes
    per_replica = co["k"].nbytes * 2 + ch["kc"].nbytes * 2 + w_bytes
    R = max(4, -(-3 * L2_BYTES // per_replica))
    base = {"k": dev_bf16(co["k"]), "v": dev_bf16(co["v"]), "kc": dev_bf16(ch["kc"]),
            "vc": dev_bf16(ch["vc"]), "w": dev_bf16(cv["w_out_major"] if out_major else cv["w_in_major"])}
    k_new, v_new, q = dev_bf16(co["k_new"]), dev_bf16(co["v_new"]), dev_bf16(co["q"])
    qc = dev_bf16(ch["q"])
    lens0 = torch.from_numpy(np.tile(co["len"], (R, 1))).to(dev)
    lens = lens0.clone()
    clen = torch.from_numpy(ch["len"]).to(dev)
    shared = {}
    if cfg.shared_S:
        shared = dict(k_shared=dev_bf16(co["k_shared"]), v_shared=dev_bf16(co["v_shared"]),
                      shared_len=torch.from_numpy(co["shared_len"]).to(dev),
                      shared_id=torch.from_numpy(co["shared_id"]).to(dev))
    ctx = ph.photon_create(cfg.Hq, cfg.Hkv, cfg.dh, cfg.D, cfg.P, cfg.C, max(cfg.B, cfg.Nc),
                           args.max_splits)
    if args.attention_ctas:
        ph.photon_set_attention_ctas(ctx, args.attention_ctas)
    reps = []
    for r in range(R):
        t = {n: (b if r == 0 else b.clone()) for n, b in base.items()}
        t["out"] = torch.empty_like(q)
        t["U"] = torch.empty(cfg.B, cfg.P, cfg.D, dtype=torch.bfloat16, device=dev)
        t["oc"] = torch.empty_like(qc)
        t["kv"] = ph.make_kv(t["k"], t["v"], lens[r], max_len=cfg.S, **shared)
        t["ckv"] = ph.make_kv(t["kc"], t["vc"], clen)
        t["args"] = ph.make_step_args(t["kv"], k_new, v_new, q, t["out"], scale, t["w"], layout, t["U"],
                                      cfg.B, chunks=t["ckv"], q_chunk=qc, out_chunk=t["oc"], Nc=cfg.Nc,
                                      scale_chunk=scale)
        reps.append(t)
    torch.cuda.synchronize()

    def step(i, a=None):
        r = i % R
        ph.photon_decode_step(ctx, a if a is not None else reps[r]["args"])
        if r == R - 1:
            lens.copy_(lens0)                     # undo the appends of one ring cycle

    K, W = args.steps, args.warmup
    for i in range(W):
        step(i)
    lens.copy_(lens0)
    torch.cuda.synchronize()
    n0 = ph.photon_launch_count(ctx)
    step(0)
    launches_per_step = ph.photon_launch_count(ctx) - n0
    for i in range(1, R):
        step(i)
    torch.cuda.synchronize()
    assert ph.photon_device_status(ctx) == 0, "device status word set during warm-up"

    # CUDA graphs of one ring cycle each (R steps + the length reset); K steps = full cycles + a tail
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())

    def capture(n_steps):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for i in range(n_steps):
                    step(i)
                if n_steps % R:
                    lens.copy_(lens0)
        return g

    cycles_per_graph = max(1, 32 // R)
    G = R * cycles_per_graph
    g_full = capture(G) if K >= G else None
    g_tail = capture(K % G) if K % G else None
    n_full = K // G

    def replay():
        for _ in range(n_full):
            g_full.replay()
        if g_tail is not None:
            g_tail.replay()

    replay() if K <= 4096 else (g_full.replay() if g_full else g_tail.replay())     # untimed graph warm-up
    torch.cuda.synchronize()

    uuid = str(torch.cuda.get_device_properties(dev).uuid)
    sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
    # the K steps are timed REPS times over (each repetition bracketed by a barrier and a synchronize on both
    # sides, device time by CUDA events, max over ranks); the median repetition is the one reported
    REPS = 5 if K <= 4096 else 3
    secs = []
    sampler.start()
    for _ in range(REPS):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        pd.barrier()
        torch.cuda.synchronize()
        e0.record()
        replay()
        e1.record()
        torch.cuda.synchronize()
        pd.barrier()
        secs.append(pd.reduce_max(e0.elapsed_time(e1) * 1e-3))
    clocks = sampler.stop()
    if clocks["samples"] < 3:                     # region too short to sample: repeat it untimed under the sampler
        sampler = ClockSampler(sampler.uuid)
        sampler.start()
        t_end = time.time() + 1.0
        while time.time() < t_end:
            replay()
            torch.cuda.synchronize()
        clocks = sampler.stop()
        clocks["note"] = "timed region shorter than the sampling period; sampled on an untimed repeat of it"
    assert ph.photon_device_status(ctx) == 0, "device status word set during the timed region"
    sec_max = statistics.median(secs)
    tokens_total = pd.reduce_sum(cfg.tokens_per_step * K)
    value = tokens_total / sec_max

    # per-kernel times: a CUDA graph of back-to-back calls of one part, rotating over the replicas
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except OSError:
        pass
    hbm_peak = float(peaks.get("hbm_gbs", 6650.0))
    tensor_peak = float(peaks.get("bf16_tflops", 1590.0))
    peak_src = "MEASURED_PEAKS.json, of measured" if peaks else "6650 GB/s / 1590 TFLOP/s, of fallback"

    def graph_time_us(fn, reset_lens=False, calls=None, replays=6):
        calls = calls or R * max(1, 32 // R)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for i in range(calls):
                    fn(reps[i % R])
                    if reset_lens and i % R == R - 1:
                        lens.copy_(lens0)
        g.replay()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(replays):
            g.replay()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) * 1e3 / (replays * calls)

    qo_coarse = 2 * cfg.B * cfg.Hq * cfg.dh * 2
    qo_chunk = 2 * cfg.Nc * cfg.Hq * cfg.dh * 2
    conv_flops = 2.0 * cfg.B * cfg.D * cfg.P * cfg.D
    conv_bytes = w_bytes + cfg.B * cfg.D * 2 + cfg.B * cfg.P * cfg.D * 2
    kernels = {
        "coarse_attn": {"bytes": coarse_bytes + qo_coarse,
                        "fn": lambda t: ph.photon_coarse_attn(ctx, t["kv"], q, t["out"], None, scale)},
        "chunk_attn": {"bytes": chunk_bytes + qo_chunk,
                       "fn": lambda t: ph.photon_chunk_attn(ctx, t["ckv"], qc, None, t["oc"], scale=scale)},
        "converter": {"bytes": conv_bytes, "flops": conv_flops,
                      "fn": lambda t: ph.photon_converter(ctx, t["out"].view(cfg.B, -1), t["w"], layout,
                                                          None, t["U"])},
        "kv_append": {"bytes": 2 * 2 * cfg.B * cfg.Hkv * cfg.dh * 2, "reset": True,
                      "fn": lambda t: ph.photon_kv_append(ctx, t["kv"], k_new, v_new)},
    }
    parts = {}
    lens.copy_(lens0)
    for name, kd in kernels.items():
        if args.no_parts and name not in ("coarse_attn", "chunk_attn"):
            continue
        us = graph_time_us(kd["fn"], reset_lens=kd.get("reset", False))
        kd["us"] = us
        parts[name] = {"us": us, "algorithmic_bytes": kd["bytes"], "GBps": kd["bytes"] / us * 1e-3,
                       "frac_hbm": kd["bytes"] / us * 1e-3 / hbm_peak}
        if "flops" in kd:
            parts[name]["TFLOPs"] = kd["flops"] / us * 1e-6
            t_roof = max(kd["bytes"] / (hbm_peak * 1e3), kd["flops"] / (tensor_peak * 1e6))
            parts[name]["frac_of_own_roofline"] = t_roof / us
    lens.copy_(lens0)
    torch.cuda.synchronize()
    def time_calls(fns, replays=6):
        """us per call of a CUDA graph that runs the given calls back to back, replayed `replays` times."""
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for fn in fns:
                    fn()
        g.replay()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(replays):
            g.replay()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) * 1e3 / (replays * len(fns))

    def read_ceiling(nbytes):
        """The read-ceiling probe of the library on buffers of nbytes (rotating, more than 3x L2 in all): a kernel with
        the attention's launch, grid and ring that only brings the bytes into shared memory.  Best of three grids."""
        nbytes -= nbytes % 16
        n_buf = max(4, -(-3 * L2_BYTES // nbytes))
        bufs = [torch.empty(nbytes, dtype=torch.uint8, device=dev).random_() for _ in range(n_buf)]
        best = None
        for ctas in (0, 2 * torch.cuda.get_device_properties(dev).multi_processor_count,
                     torch.cuda.get_device_properties(dev).multi_processor_count):
            us = time_calls([(lambda b=b, c=ctas: ph.photon_read_probe(ctx, b, nbytes, c)) for b in bufs * max(1, 32 // n_buf)])
            if best is None or us < best["us"]:
                best = {"us": us, "ctas": ctas}
        del bufs
        torch.cuda.empty_cache()
        return best

    def other_workload(idx):
        """The dominant attention part of another of the target workloads, timed in this run the same way as `parts`
        (its caches only feed a timing: drawn on the device from a fixed seed, lengths as in the workload)."""
        oc = wl.CONFIGS[idx]
        gen = torch.Generator(device=dev)
        gen.manual_seed(777 + idx)
        octx = ph.photon_create(oc.Hq, oc.Hkv, oc.dh, oc.D, oc.P, oc.C, max(oc.B, oc.Nc), args.max_splits)
        o_scale = oc.dh ** -0.5

        def draw(*shape):
            return torch.empty(*shape, dtype=torch.bfloat16, device=dev).normal_(generator=gen)

        res = {}
        if idx == 4:
            # chunk attention over every in-flight chunk; lengths P + (in-chunk position + 1) as the workload draws them
            ln = torch.from_numpy(wl.chunk_inputs(wl.scaled(oc, B=1))["len"][:oc.chunks_per_seq]).repeat(oc.B).to(dev)
            cap = oc.P + oc.C
            kc, vc = draw(oc.Nc, oc.Hkv, cap, oc.dh), draw(oc.Nc, oc.Hkv, cap, oc.dh)
            qq = draw(oc.Nc, oc.Hq, oc.dh)
            oo = torch.empty_like(qq)
            kvc = ph.make_kv(kc, vc, ln.to(torch.int32))
            nbytes = int(ln.sum().item()) * oc.Hkv * oc.dh * 4 + 2 * oc.Nc * oc.Hq * oc.dh * 2
            us = time_calls([lambda: ph.photon_chunk_attn(octx, kvc, qq, None, oo, scale=o_scale)] * 8)
            res = {"kernel": "chunk_attn", "l2": "one set of chunk buffers of %.0f MiB, larger than L2" % (nbytes / 2**20)}
        else:
            kvb = oc.B * oc.Hkv * oc.S * oc.dh * 4
            n_rep = max(4, -(-3 * L2_BYTES // kvb))
            k0, v0 = draw(oc.B, oc.Hkv, oc.S, oc.dh), draw(oc.B, oc.Hkv, oc.S, oc.dh)
            ks, vs = [k0] + [k0.clone() for _ in range(n_rep - 1)], [v0] + [v0.clone() for _ in range(n_rep - 1)]
            qq = draw(oc.B, oc.Hq, oc.dh)
            oo = [torch.empty_like(qq) for _ in range(n_rep)]
            ln = torch.full((oc.B,), oc.S, dtype=torch.int32, device=dev)
            sh = {}
            if oc.shared_S:
                sh = dict(k_shared=draw(1, oc.Hkv, oc.shared_S, oc.dh), v_shared=draw(1, oc.Hkv, oc.shared_S, oc.dh),
                          shared_len=torch.full((1,), oc.shared_S, dtype=torch.int32, device=dev),
                          shared_id=torch.zeros(oc.B, dtype=torch.int32, device=dev))
            kvs = [ph.make_kv(ks[r], vs[r], ln, max_len=oc.S, **sh) for r in range(n_rep)]
            nbytes = wl.coarse_kv_bytes(oc) + 2 * oc.B * oc.Hq * oc.dh * 2
            us = time_calls([(lambda r=r: ph.photon_coarse_attn(octx, kvs[r], qq, oo[r], None, o_scale))
                             for r in list(range(n_rep)) * max(1, 32 // n_rep)])
            res = {"kernel": "coarse_attn", "l2": "%d replicas of the cache, %.0f MiB in all" % (n_rep, n_rep * kvb / 2**20)}
            if oc.shared_S:
                flops = 4.0 * oc.B * oc.Hq * oc.shared_S * oc.dh
                logical = oc.B * (oc.S + oc.shared_S) * oc.Hkv * oc.dh * 4
                t_roof = max(nbytes / (hbm_peak * 1e3), flops / (tensor_peak * 1e6))
                res.update({"prefix_flops": flops, "TFLOPs": flops / us * 1e-6, "frac_of_own_roofline": t_roof / us,
                            "logical_GBps": logical / us * 1e-3,
                            "note": "one launch: the prefix contraction on the tensor cores with the branches' short own caches "
                                    "riding along as extra key tiles (two launches once an own cache exceeds 32 rows); the prefix "
                                    "is read once, so the HBM fraction of the physical bytes says little: the own roofline "
                                    "is the slower of bytes / HBM peak and prefix flops / bf16 peak; logical = bytes a "
                                    "cache with the prefix copied into every branch would read"})
        bits_o = ph.photon_device_status(octx)
        ph.photon_destroy(octx)
        torch.cuda.empty_cache()
        res.update({"workload": oc.name, "us": us, "algorithmic_bytes": nbytes, "GBps": nbytes / us * 1e-3,
                    "frac": nbytes / us * 1e-3 / hbm_peak, "frac_of_nominal_8TBs": nbytes / us * 1e-3 / 8000.0,
                    "device_status": bits_o})
        return res

    parts["note"] = ("each part timed as a CUDA graph of back-to-back calls rotating over the replicas; "
                     "kv_append's figure includes a %d-int length reset every %d calls" % (cfg.B * R, R))

    # The global caches of the three generation schedules (a flat Transformer; hierarchical generation,
    # which keeps a cache at every level; recursive generation, which keeps the top level only) for the same
    # context, read with the same attention kernel: measured time and bytes per read and, amortised over the
    # tokens between reads, per generated token.  The lower-level caches only feed a timing, so they are
    # filled on the device from a fixed torch seed; the top level is the step's own coarse attention.
    kv_measured, schedules = {}, {}
    if not args.no_parts and cfg.compress == 16:
        gen = torch.Generator(device=dev)
        gen.manual_seed(1234 + cfg.seed)
        per_level = {2: {"rows_per_sequence": cfg.S + cfg.shared_S, "kv_bytes_per_read": coarse_bytes,
                         "us_per_read": kernels["coarse_attn"].get("us")}}
        for level, fn in ((0, ph.photon_flat_attn), (1, ph.photon_coarse_attn)):
            rows = wl.global_caches(cfg, "flat" if level == 0 else "hierarchical")[0]["rows"]
            nbytes = cfg.B * cfg.Hkv * rows * cfg.dh * 2 * 2
            if nbytes > (24 << 30):
                continue
            kk = torch.empty(cfg.B, cfg.Hkv, rows, cfg.dh, dtype=torch.bfloat16, device=dev).normal_(generator=gen)
            vv = torch.empty_like(kk).normal_(generator=gen)
            ln = torch.full((cfg.B,), rows, dtype=torch.int32, device=dev)
            kvf = ph.make_kv(kk, vv, ln, max_len=rows)
            o2 = torch.empty_like(q)
            for _ in range(2):
                fn(ctx, kvf, q, o2, None, scale)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            n_rep = 5
            torch.cuda.synchronize()
            a.record()
            for _ in range(n_rep):
                fn(ctx, kvf, q, o2, None, scale)
            b.record()
            torch.cuda.synchronize()
            per_level[level] = {"rows_per_sequence": rows, "kv_bytes_per_read": nbytes,
                                "us_per_read": a.elapsed_time(b) * 1e3 / n_rep}
            del kk, vv, kvf
        torch.cuda.empty_cache()
        kv_measured = {"flat_token_level": per_level.get(0), "level1_global": per_level.get(1),
                       "recursive_top_level": per_level[2]}
        for sch in wl.SCHEDULES:
            caches = wl.global_caches(cfg, sch)
            if any(c["level"] not in per_level for c in caches):
                continue
            schedules[sch] = {
                "caches": [dict(c, **per_level[c["level"]]) for c in caches],
                "kv_bytes_per_token": sum(per_level[c["level"]]["kv_bytes_per_read"] / c["tokens_per_read"]
                                          for c in caches) / cfg.B,
                "global_attention_us_per_token": sum(per_level[c["level"]]["us_per_read"] / c["tokens_per_read"]
                                                     for c in caches)}
        if schedules:
            schedules["note"] = ("per sequence and layer, whole batch decoded in step; levels 0 and 1 hold a shared prefix "
                                 "once per branch; eager calls on caches larger than L2 for levels 0 and 1, the "
                                 "timed graph for the top level")

    # the widened row: the local decoder's attention at every position of every in-flight chunk in one launch
    # (teacher-forced whole chunks).  It reuses the chunk buffers of the replicas with every row counted as
    # present; its queries only feed a timing, so they are drawn on the device from a fixed torch seed.
    widened = {}
    if not args.no_parts:
        cap = cfg.P + cfg.C
        gen = torch.Generator(device=dev)
        gen.manual_seed(4321 + cfg.seed)
        n_q = max(2, min(R, -(-2 * L2_BYTES // max(1, cfg.Nc * cap * cfg.Hq * cfg.dh * 2))))
        qr = [torch.empty(cfg.Nc, cap, cfg.Hq, cfg.dh, dtype=torch.bfloat16, device=dev).normal_(generator=gen)
              for _ in range(n_q)]
        orows = [torch.empty_like(t) for t in qr]
        full_len = torch.full((cfg.Nc,), cap, dtype=torch.int32, device=dev)
        full_kv = [ph.make_kv(t["kc"], t["vc"], full_len) for t in reps]
        turn = {"i": 0}

        def causal_call(t):
            i = turn["i"] = turn["i"] + 1
            ph.photon_chunk_causal_attn(ctx, full_kv[i % R], qr[i % n_q], None, orows[i % n_q], scale=scale)

        us = graph_time_us(causal_call)
        nbytes = 2 * cfg.Nc * cfg.Hkv * cap * cfg.dh * 2 + 2 * cfg.Nc * cap * cfg.Hq * cfg.dh * 2
        flops = 4.0 * cfg.Nc * cfg.Hq * cfg.dh * cap * (cap + 1) / 2
        widened["chunk_causal_attn"] = {
            "workload": "all %d rows of each of the %d in-flight chunks, causal" % (cap, cfg.Nc),
            "us": us, "algorithmic_bytes": nbytes, "GBps": nbytes / us * 1e-3,
            "frac_hbm": nbytes / us * 1e-3 / hbm_peak, "TFLOPs": flops / us * 1e-6,
            "note": "K, V, q and out each counted once; causal flops only"}
        del qr, orows, full_kv
        torch.cuda.empty_cache()

        # the coarse attention on a paged layout of the same cache: pages of 128 rows (64 when the stream is
        # shorter), scattered over the pool by a fixed permutation; same bytes, one table look-up per tile
        if cfg.S % 64 == 0 and not cfg.shared_S:
            pr = 128 if cfg.S % 128 == 0 else 64
            ppu = cfg.S // pr
            perm = torch.randperm(cfg.B * ppu, generator=torch.Generator().manual_seed(99 + cfg.seed)).to(dev)
            inv = torch.empty_like(perm)
            inv[perm] = torch.arange(cfg.B * ppu, device=dev)

            def paged(t):
                pool = t.view(cfg.B, cfg.Hkv, ppu, pr, cfg.dh).permute(0, 2, 1, 3, 4).reshape(cfg.B * ppu, cfg.Hkv, pr, cfg.dh)
                return pool[perm].contiguous()                 # pool[i] = page perm[i]; page j sits at inv[j]

            table = inv.view(cfg.B, ppu).to(torch.int32).contiguous()
            pkv = [ph.make_kv(paged(t["k"]), paged(t["v"]), lens[r], max_len=cfg.S, page_table=table)
                   for r, t in enumerate(reps)]
            turn["i"] = -1

            def paged_call(t):
                i = turn["i"] = turn["i"] + 1
                ph.photon_coarse_attn(ctx, pkv[i % R], q, reps[i % R]["out"], None, scale)

            us_p = graph_time_us(paged_call)
            widened["paged_coarse_attn"] = {
                "workload": "the coarse attention of the step on pages of %d rows scattered over a pool" % pr,
                "us": us_p, "algorithmic_bytes": kernels["coarse_attn"]["bytes"],
                "GBps": kernels["coarse_attn"]["bytes"] / us_p * 1e-3,
                "frac_hbm": kernels["coarse_attn"]["bytes"] / us_p * 1e-3 / hbm_peak, "TFLOPs": 0.0,
                "us_contiguous": kernels["coarse_attn"]["us"]}
            del pkv
            torch.cuda.empty_cache()

        # the top-level context chunker (step (ii) of a recursive-generation step): normalise the 4 concatenated
        # lower-level latents per sequence, project [B, 4D] -> [B, D]; weights rotate like the converter's
        ci = wl.chunker_inputs(cfg)
        Kc = ci["K"]
        cw = [dev_bf16(ci["w_out_major"] if out_major else ci["w_in_major"])]
        cw += [cw[0].clone() for _ in range(R - 1)]
        cx, cg, cb = dev_bf16(ci["x"]), dev_bf16(ci["gamma"]), dev_bf16(ci["bias"])
        cxn = torch.empty_like(cx)
        cy = torch.empty(cfg.B, cfg.D, dtype=torch.bfloat16, device=dev)
        turn["i"] = 0

        def norm_call(t):
            ph.photon_rmsnorm(ctx, cx, cg, ci["eps"], cxn)

        def linear_call(t):
            i = turn["i"] = turn["i"] + 1
            ph.photon_linear(ctx, cxn, cw[i % R], layout, cb, cy)

        def chunker_call(t):
            norm_call(t)
            linear_call(t)

        us_n, us_l, us_c = graph_time_us(norm_call), graph_time_us(linear_call), graph_time_us(chunker_call)
        cbytes = Kc * cfg.D * 2 + cfg.B * Kc * 2 + cfg.B * cfg.D * 2
        cflops = 2.0 * cfg.B * Kc * cfg.D
        t_roof = max(cbytes / (hbm_peak * 1e3), cflops / (tensor_peak * 1e6))
        widened["chunker"] = {
            "workload": "[%d, %d] -> [%d, %d]: row normalisation, then linear with bias" % (cfg.B, Kc, cfg.B, cfg.D),
            "us": us_c, "us_rmsnorm": us_n, "us_linear": us_l, "algorithmic_bytes": cbytes,
            "GBps": cbytes / us_c * 1e-3, "frac_hbm": cbytes / us_c * 1e-3 / hbm_peak,
            "TFLOPs": cflops / us_c * 1e-6, "frac_of_own_roofline": t_roof / us_c,
            "note": "x, W and y counted once; the normalised copy of x is an intermediate"}
        del cw
        torch.cuda.empty_cache()

        # STEP of one LLaMA layer of the top-level encoder (normalise, q/k/v, rotary, append, attention, output
        # projection, MLP) on the step's own caches: eight or nine launches; weights rotate over the replicas
        if cfg.Hq * cfg.dh == cfg.D:
            li = wl.encoder_layer_inputs(cfg)
            F = li["F"]
            names = ("g1", "wqkv", "wo", "g2", "wgu", "wdown")
            lw0 = {n: dev_bf16(np.ascontiguousarray(li[n].T) if out_major and li[n].ndim == 2 else li[n]) for n in names}
            layers = []
            for r in range(R):
                wr = lw0 if r == 0 else {n: (t.clone() if t.dim() == 2 else t) for n, t in lw0.items()}
                layers.append(ph.make_layer(*(wr[n] for n in names), layout, F))
            scr = ph.make_layer_scratch(cfg.B, cfg.Hq, cfg.Hkv, cfg.dh, F, dev, torch.bfloat16)
            ex = dev_bf16(li["x"])
            ey = torch.empty_like(ex)
            plain_kv = [ph.make_kv(t["k"], t["v"], lens[r], max_len=cfg.S) for r, t in enumerate(reps)]
            turn["i"] = -1

            def layer_call(t):
                i = turn["i"] = turn["i"] + 1
                ph.photon_encoder_step(ctx, layers[i % R], scr, ex, plain_kv[i % R], ey, scale=scale)

            lens.copy_(lens0)
            n_l0 = ph.photon_launch_count(ctx)
            layer_call(None)
            launches_e = ph.photon_launch_count(ctx) - n_l0
            lens.copy_(lens0)
            us_e = graph_time_us(layer_call, reset_lens=True)
            lens.copy_(lens0)
            QKV = (cfg.Hq + 2 * cfg.Hkv) * cfg.dh
            wbytes = 2 * (cfg.D * QKV + cfg.D * cfg.D + cfg.D * 2 * F + F * cfg.D)
            ebytes = wbytes + cfg.B * cfg.S * cfg.Hkv * cfg.dh * 4
            eflops = 2.0 * cfg.B * (wbytes / 2)
            widened["encoder_step"] = {
                "workload": "one layer, batch %d: D %d, %dq/%dkv x %d, F %d, cache of %d latents per sequence" % (
                    cfg.B, cfg.D, cfg.Hq, cfg.Hkv, cfg.dh, F, cfg.S),
                "us": us_e, "launches": launches_e, "algorithmic_bytes": ebytes, "GBps": ebytes / us_e * 1e-3,
                "frac_hbm": ebytes / us_e * 1e-3 / hbm_peak, "TFLOPs": eflops / us_e * 1e-6,
                "note": "weights and the sequences' own K/V rows counted once (no shared prefix), activations not counted"}

            # the same layer of a local decoder for the newest in-chunk position of every in-flight chunk:
            # chunk buffers of the replicas one row short of their recorded length (room for the append);
            # the lengths are put back by a small copy before every call (inside the timed graph)
            lcfg = wl.scaled(cfg, B=cfg.Nc)
            dx = torch.empty(cfg.Nc, cfg.D, dtype=torch.bfloat16, device=dev).normal_(generator=gen)
            dy = torch.empty_like(dx)
            dlen0 = (clen - 1).clamp(min=0)
            dlen = dlen0.clone()
            dkv = [ph.make_kv(t["kc"], t["vc"], dlen) for t in reps]
            dscr = ph.make_layer_scratch(cfg.Nc, cfg.Hq, cfg.Hkv, cfg.dh, F, dev, torch.bfloat16)
            turn["i"] = -1

            def dec_call(t):
                i = turn["i"] = turn["i"] + 1
                dlen.copy_(dlen0)
                ph.photon_decoder_step(ctx, layers[i % R], dscr, dx, dkv[i % R], dy, scale=scale)

            n_l0 = ph.photon_launch_count(ctx)
            dec_call(None)
            launches_d = ph.photon_launch_count(ctx) - n_l0
            us_d = graph_time_us(dec_call)
            dbytes = wbytes + int(dlen0.sum().item() + cfg.Nc) * cfg.Hkv * cfg.dh * 4 + 2 * cfg.Nc * cfg.D * 2
            dflops = 2.0 * cfg.Nc * (wbytes / 2)
            t_roof = max(dbytes / (hbm_peak * 1e3), dflops / (tensor_peak * 1e6))
            widened["decoder_step"] = {
                "workload": "one layer, %d in-flight chunks (one new token each): D %d, F %d, windows of at most %d rows" % (
                    cfg.Nc, cfg.D, F, cfg.P + cfg.C),
                "us": us_d, "launches": launches_d, "algorithmic_bytes": dbytes, "GBps": dbytes / us_d * 1e-3,
                "frac_hbm": dbytes / us_d * 1e-3 / hbm_peak, "TFLOPs": dflops / us_d * 1e-6,
                "frac_of_own_roofline": t_roof / us_d,
                "note": "weights, the chunks' K/V rows, x and y counted once; the figure includes one small copy that "
                        "puts the lengths back before each call"}
            # and over fresh converter prefixes: the P prefix vectors of (up to 4096) chunks go through the layer, are
            # installed as rows 0..P-1 of emptied chunk buffers and attend causally among themselves
            n_pre = min(cfg.Nc, 4096)
            pU = torch.empty(n_pre, cfg.P, cfg.D, dtype=torch.bfloat16, device=dev).normal_(generator=gen)
            pY = torch.empty_like(pU)
            plen = torch.zeros(cfg.Nc, dtype=torch.int32, device=dev)
            pkv2 = [ph.make_kv(t["kc"].clone(), t["vc"].clone(), plen) for t in reps[:2]]
            pscr = ph.make_layer_scratch(n_pre * cfg.P, cfg.Hq, cfg.Hkv, cfg.dh, F, dev, torch.bfloat16)
            turn["i"] = -1

            def prefill_call(t):
                i = turn["i"] = turn["i"] + 1
                plen.zero_()
                ph.photon_decoder_prefill(ctx, layers[i % R], pscr, pU, pkv2[i % 2], None, pY, n=n_pre, scale=scale)

            n_l0 = ph.photon_launch_count(ctx)
            prefill_call(None)
            launches_p = ph.photon_launch_count(ctx) - n_l0
            us_pf = graph_time_us(prefill_call)
            pflops = 2.0 * n_pre * cfg.P * (wbytes / 2)
            pbytes = wbytes + 2 * n_pre * cfg.P * cfg.D * 2 + 2 * n_pre * cfg.P * cfg.Hkv * cfg.dh * 2
            t_roof = max(pbytes / (hbm_peak * 1e3), pflops / (tensor_peak * 1e6))
            widened["decoder_prefill"] = {
                "workload": "one layer over the %d prefix vectors of each of %d chunks" % (cfg.P, n_pre),
                "us": us_pf, "launches": launches_p, "algorithmic_bytes": pbytes, "GBps": pbytes / us_pf * 1e-3,
                "frac_hbm": pbytes / us_pf * 1e-3 / hbm_peak, "TFLOPs": pflops / us_pf * 1e-6,
                "frac_of_own_roofline": t_roof / us_pf,
                "note": "weights, U, y and the installed K/V rows counted once; includes the small kernel that empties the lengths"}
            del layers, lw0, dscr, dkv, pscr, pkv2
            torch.cuda.empty_cache()

    # roofline of the dominant kernel = the attention part that takes the longest
    dom = max(("coarse_attn", "chunk_attn"), key=lambda n: kernels[n]["us"])
    def recorded_traffic(kernel_name):
        """DRAM bytes per launch from the committed ncu capture, or None once the kernel's source has changed."""
        note = "no ncu capture on record for this kernel and workload"
        if args.batch or args.hierarchy:
            return None, "reduced batch or another hierarchy: the recorded traffic belongs to the standard workload"
        try:
            rec = json.load(open(os.path.join(ROOT, "profiles", "dram_traffic.txt"))).get(
                f"config{cfg.index}", {}).get(kernel_name)
            if rec:
                import hashlib
                src = os.path.join(ROOT, "paper_2512_20687_b200", "csrc", rec["source"])
                if hashlib.sha256(open(src, "rb").read()).hexdigest() == rec["source_sha256"]:
                    return rec["dram_bytes_per_launch"], rec.get("how", "")
                note = "kernel source changed since the ncu counters were taken"
        except (OSError, ValueError, KeyError):
            pass
        return None, note

    # (with a shared prefix the coarse attention is the shared-prefix kernel, recorded under that name)
    traffic, traffic_note = recorded_traffic("shared_prefix" if cfg.shared_S and dom == "coarse_attn" else dom)
    if "chunk_causal_attn" in widened:
        widened["chunk_causal_attn"]["traffic"], widened["chunk_causal_attn"]["traffic_note"] = recorded_traffic(
            "chunk_causal_attn")
    ach = kernels[dom]["bytes"] / kernels[dom]["us"] * 1e-3
    roofline = {"bound": "hbm", "kernel": dom, "achieved": ach, "peak": hbm_peak, "unit": "GB/s",
                "frac": ach / hbm_peak, "traffic": traffic, "traffic_note": traffic_note,
                "algorithmic_bytes": kernels[dom]["bytes"], "us_per_launch": kernels[dom]["us"],
                "peak_source": peak_src, "frac_of_nominal_8TBs": ach / 8000.0,
                # the replicas are meant to keep the reads in HBM: less DRAM traffic than 95 % of the
                # algorithmic bytes would mean the L2 served part of them
                "l2_assisted": None if traffic is None else bool(traffic < 0.95 * kernels[dom]["bytes"])}
    ceil = {"us": None, "ctas": 0} if args.only_this_workload else read_ceiling(kernels[dom]["bytes"])
    roofline.update({"read_ceiling_us": ceil["us"], "read_ceiling_ctas": ceil["ctas"],
                     "frac_of_read_ceiling": ceil["us"] / kernels[dom]["us"] if ceil["us"] else None,
                     "read_ceiling_note": "photon_read_probe on buffers of the same size: the attention's launch, grid and "
                                          "ring of bulk copies with nothing computed (best of three grids)"})
    # the dominant attention part of every target workload (configs 1-4), this run's own workload from `parts`
    by_workload = {}
    if not args.no_parts and not args.batch and not args.hierarchy and not args.only_this_workload:
        for idx in (1, 2, 3, 4):
            if idx == cfg.index:
                pc = parts[dom]
                by_workload[f"config{idx}"] = {"workload": cfg.name, "kernel": dom, "us": pc["us"],
                                               "algorithmic_bytes": pc["algorithmic_bytes"], "GBps": pc["GBps"],
                                               "frac": pc["frac_hbm"], "frac_of_nominal_8TBs": pc["GBps"] / 8000.0}
            else:
                by_workload[f"config{idx}"] = other_workload(idx)
        by_workload["note"] = ("dominant attention part per target workload, CUDA graph of back-to-back calls on inputs larger "
                               "than L2, fraction of the measured copy peak (%s) and of the nominal 8 TB/s" % peak_src)
    if cfg.shared_S and "coarse_attn" in parts:
        # a shared prefix makes the coarse attention a contraction over the prefix plus a stream over the own
        # rows: its own roofline is the slower of the two, and the bytes a cache without sharing would read
        # are reported as logical, not physical, throughput
        pc = parts["coarse_attn"]
        prefix_flops = 4.0 * cfg.B * cfg.Hq * cfg.shared_S * cfg.dh
        logical = (cfg.B * (cfg.S + cfg.shared_S)) * cfg.Hkv * cfg.dh * 4
        t_roof = max(pc["algorithmic_bytes"] / (hbm_peak * 1e3), prefix_flops / (tensor_peak * 1e6))
        pc.update({"prefix_flops": prefix_flops, "TFLOPs": prefix_flops / pc["us"] * 1e-6,
                   "frac_of_own_roofline": t_roof / pc["us"], "logical_kv_bytes": logical,
                   "logical_GBps": logical / pc["us"] * 1e-3,
                   "logical_note": "bytes a cache with the prefix copied into every branch would read; not physical traffic"})
    # derived from the per-part times: a meta-context of C_{<=L} tokens per sequence needs the append and the
    # coarse attention once, the converter once per level-2 latent plus once for the level above (1 + C_2
    # times), and the chunk attention once per token
    amortised = None
    if all(n in parts for n in ("kv_append", "coarse_attn", "converter", "chunk_attn")):
        c2 = 4 if cfg.compress == 16 else max(1, int(round(cfg.compress ** 0.5)))
        t_meta = (parts["kv_append"]["us"] + parts["coarse_attn"]["us"] + (1 + c2) * parts["converter"]["us"]
                  + cfg.compress * parts["chunk_attn"]["us"])
        amortised = {"tokens_per_s": cfg.tokens_per_step * cfg.compress / t_meta * 1e6, "us_per_meta_context": t_meta,
                     "note": "derived from the parts: append + coarse attention once, converter %d times, chunk attention "
                             "%d times per meta-context of %d tokens per sequence" % (1 + c2, cfg.compress, cfg.compress)}
    step_bytes = sum(kernels[n]["bytes"] for n in kernels)

    # end to end through the public API with host buffers: every step its inputs (new K/V row, both
    # query tensors, the cache lengths) travel from pinned host memory to the device and its results
    # (both attention outputs and the converter's prefix vectors U) travel back.  The inputs live in one host buffer and one device buffer
    # (the tensors are views into it), so a step is one H2D copy, the decode step and one D2H copy.
    def pack(tensors):
        offs, total = [], 0
        for t in tensors:
            offs.append(total)
            total += (t.numel() * t.element_size() + 255) // 256 * 256
        return offs, total

    in_src = [k_new, v_new, q, lens0[0], qc]              # the chunk attention's input last: it may travel apart
    in_offs, in_total = pack(in_src)
    h_in = torch.empty(in_total, dtype=torch.uint8).pin_memory()
    d_in = torch.empty(in_total, dtype=torch.uint8, device=dev)
    views = []
    for t, o in zip(in_src, in_offs):
        nb = t.numel() * t.element_size()
        h_in[o:o + nb].copy_(t.cpu().contiguous().view(-1).view(torch.uint8))
        views.append(d_in[o:o + nb].view(t.dtype).view(t.shape))
    e_k_new, e_v_new, e_q, e_len, e_qc = views
    n_e2e = max(3, min(K, 2000))

    def run_e2e(with_U):
        """tokens/s of host-driven steps and the bytes that come back per step.  with_U: the converter's prefix
        vectors travel to the host as well (they lie between the two attention outputs in the staging area)."""
        out_src = [reps[0]["out"]] + ([reps[0]["U"]] if with_U else []) + [reps[0]["oc"]]
        out_offs, out_total = pack(out_src)
        d_out = torch.empty(out_total, dtype=torch.uint8, device=dev)
        h_out = torch.empty(out_total, dtype=torch.uint8).pin_memory()
        vs = [d_out[o:o + t.numel() * t.element_size()].view(t.dtype).view(t.shape) for t, o in zip(out_src, out_offs)]
        e_out, e_oc = vs[0], vs[-1]
        e2e_args = []
        for r in range(R):
            t = reps[r]
            kv_e = ph.make_kv(t["k"], t["v"], e_len, max_len=cfg.S, **shared)
            e2e_args.append(ph.make_step_args(kv_e, e_k_new, e_v_new, e_q, e_out, scale, t["w"], layout,
                                              vs[1] if with_U else t["U"], cfg.B, chunks=t["ckv"], q_chunk=e_qc,
                                              out_chunk=e_oc, Nc=cfg.Nc, scale_chunk=scale))
        host_io = ph.HostIO(h_in, d_in, d_out, h_out, in_split=in_offs[4], out_split=out_offs[-1])
        # one call of the library per step: host -> staging, the decode step, staging -> host, wait for the stream
        for i in range(max(3, min(300, n_e2e // 5))):  # the first few hundred host-driven steps of a process run slower
            ph.photon_decode_step_host(ctx, e2e_args[i % R], host_io)
        pd.barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for i in range(n_e2e):
            ph.photon_decode_step_host(ctx, e2e_args[i % R], host_io)
        torch.cuda.synchronize()
        sec = pd.reduce_max(time.perf_counter() - t0)
        lens.copy_(lens0)
        torch.cuda.synchronize()
        return pd.reduce_sum(cfg.tokens_per_step * n_e2e) / sec, out_total

    h2d = in_total
    e2e_val, d2h = run_e2e(False)
    e2e_val_U, d2h_U = run_e2e(True)
    lens.copy_(lens0)
    torch.cuda.synchronize()
    bits = ph.photon_device_status(ctx)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": sec_max * 1e3 / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": dict(workload_desc(cfg),
                       l2="inputs larger than L2: KV caches, chunk buffers and converter weight rotate over "
                          f"{R} replicas ({R * per_replica / 2**20:.0f} MiB vs 126 MB L2)",
                       launch="CUDA graph of %d steps replayed; per-rank batch fixed" % G,
                       w_layout=args.layout),
        "clocks": clocks,
        "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": n_e2e,
                "note": "photon_decode_step_host: one pinned host buffer -> device (new K/V row, queries, lengths), decode step, "
                        "both attention outputs -> host, wait, every step; the chunk attention's query and output cross the bus "
                        "beside the coarse part where that attention runs on the side stream, the coarse output leaves beside "
                        "the converter.  The converter's output U stays on the device in this figure: its consumers are the "
                        "local decoders (photon_decoder_prefill reads it from device memory), no host code of a serving loop "
                        "reads prefix vectors; with_converter_output is the same loop with U copied back as well",
                "with_converter_output": {"value": e2e_val_U, "unit": UNIT, "d2h_bytes_per_step": d2h_U}},
        "gpu_launches": launches_per_step * K,
        "roofline": roofline,
        "roofline_by_workload": by_workload,
        "us_per_step": sec_max * 1e6 / K,
        "step_hbm": {"algorithmic_bytes": step_bytes, "GBps": step_bytes / (sec_max / K) * 1e-9,
                     "frac": step_bytes / (sec_max / K) * 1e-9 / hbm_peak},
        "parts": parts,
        "amortised": amortised,
        "widened": widened,
        "kv_bytes_per_token": {
            "photon_coarse_per_step": coarse_bytes,
            "photon_per_token": coarse_bytes / cfg.compress / cfg.B + (chunk_bytes / cfg.Nc),
            "flat_per_token": wl.flat_kv_bytes(cfg) / cfg.B,
            "note": "per sequence and layer; coarse step amortised over %d tokens" % cfg.compress,
            "measured": kv_measured},
        "schedules": schedules,
        "device_status": bits,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(cfg)
    ph.photon_destroy(ctx)
    pd.barrier()
    if rank == 0:
        print(json.dumps(line), flush=True)
    pd.shutdown()


def spawn_ranks(n: int, argv: list[str]) -> int:
    """Starts n ranks of this script on this node (one per GPU) the way a launcher would, and returns their
    exit code: what `bench.py --gpus N` does when nobody has started the ranks for it."""
    import socket
    with socket.socket() as so:
        so.bind(("127.0.0.1", 0))
        port = so.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]
    return subprocess.call(cmd)


def main():
    args = parse()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "photon":
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
    cfg = wl.CONFIGS[args.config]
    if args.batch and args.batch < cfg.B:
        cfg = wl.scaled(cfg, B=args.batch, tokens_per_step=cfg.tokens_per_step * args.batch // cfg.B)
    if args.hierarchy:
        cfg = wl.with_hierarchy(cfg, tuple(int(t) for t in args.hierarchy.split(",")))
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_gpu(args, cfg)


if __name__ == "__main__":
    main()
