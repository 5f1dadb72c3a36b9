"""Seeded input generator and the closed-form byte counts (no GPU)."""
import numpy as np
import torch

from paper_2512_20687_b200 import workloads as wl


def test_streams_are_deterministic_and_sliceable():
    a = wl.normal_bf16(3, "t", (1000,))
    b = wl.normal_bf16(3, "t", (1000,))
    assert np.array_equal(a, b)
    assert np.array_equal(wl.normal_bf16(3, "t", (100,), offset=250), a[250:350])
    assert not np.array_equal(a, wl.normal_bf16(4, "t", (1000,)))
    assert not np.array_equal(a, wl.normal_bf16(3, "u", (1000,)))
    big = wl.normal_bf16(5, "big", (3, 1 << 22))          # crosses the threaded block size
    assert np.array_equal(big.reshape(-1)[(1 << 22) - 5:(1 << 22) + 5],
                          wl.normal_bf16(5, "big", (10,), offset=(1 << 22) - 5))


def test_distribution_and_bf16_rounding():
    x = wl.bf16_bits_to_f64(wl.normal_bf16(0, "m", (1 << 20,)))
    assert abs(x.mean()) < 5e-3 and abs(x.std() - 1.0) < 5e-3 and np.isfinite(x).all()
    w = wl.bf16_bits_to_f64(wl.normal_bf16(0, "w", (1 << 18,), std=256 ** -0.5))
    assert abs(w.var() * 256 - 1.0) < 2e-2
    r = np.random.default_rng(0).standard_normal(50000).astype(np.float32)
    t = torch.from_numpy(r).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(wl.f32_to_bf16_bits(r), t)
    assert np.array_equal(wl.bf16_bits_to_f64(t), torch.from_numpy(r).to(torch.bfloat16).double().numpy())


def test_config_table_matches_the_hierarchy():
    """Cached coarse length is T / C_{<=L} (Section 2.3.3, inference cost)."""
    for c in wl.CONFIGS:
        assert c.S == c.context // c.compress and c.D == c.Hq * c.dh and c.Hq % c.Hkv == 0
        if c.shared_S:
            assert c.shared_S == c.shared_context // c.compress
    assert [c.S for c in wl.CONFIGS] == [16, 512, 8192, 32, 128]
    assert [c.Nc for c in wl.CONFIGS] == [16, 128, 32, 512, 16384]


def test_kv_bytes_closed_forms():
    """Per step the coarse cache is C_{<=L} times smaller than a token-level
    cache; a coarse step happens once per C_{<=L} tokens, so per generated
    token the ratio is C_{<=L}^2 (takeaway table of Section 2.3.3)."""
    mib = 1 << 20
    assert [wl.coarse_kv_bytes(c) // 1024 for c in wl.CONFIGS[:1]] == [16]
    assert [wl.coarse_kv_bytes(c) / mib for c in wl.CONFIGS[1:]] == [64, 256, 20, 256]
    assert [wl.flat_kv_bytes(c) / mib for c in wl.CONFIGS[1:]] == [1024, 4096, 320, 4096]
    for c in wl.CONFIGS:
        assert wl.flat_kv_bytes(c) == c.compress * wl.coarse_kv_bytes(c)
        per_token_coarse = wl.coarse_kv_bytes(c) / c.compress
        assert wl.flat_kv_bytes(c) / per_token_coarse == c.compress ** 2 == 256


def test_generation_schedules_against_a_decode_loop():
    """Count, token by token, the rows each schedule's global attention reads
    (a level advances when its chunk fills and its newest row attends itself and
    everything before it) and compare with the closed forms; the orders of
    Section 2.3.2 / 2.3.3 follow: recursive generation reads C_{<=L}^2 times fewer
    rows than a flat Transformer, hierarchical generation is dominated by level 1."""
    C1, C2 = 4, 4
    for T in (16, 64, 1024):
        rows = {"flat": 0, "hierarchical": 0, "recursive": 0}
        n1 = n2 = 0
        for t in range(1, T + 1):
            rows["flat"] += t                              # the new token sees t rows
            if t % C1 == 0:
                n1 += 1
                rows["hierarchical"] += n1
            if t % (C1 * C2) == 0:
                n2 += 1
                rows["hierarchical"] += n2
                rows["recursive"] += n2
        for sch in wl.SCHEDULES:
            assert wl.cumulative_global_rows(T, sch) == rows[sch], (T, sch)
    big = 1 << 20
    flat, hier, rec = (wl.cumulative_global_rows(big, s) for s in wl.SCHEDULES)
    assert abs(flat / rec / 256 - 1) < 1e-4               # (C1 C2)^2
    assert abs(hier / rec / 17 - 1) < 1e-4                # 1 + C2^2
    cfg = wl.CONFIGS[1]
    per_row = cfg.Hkv * cfg.dh * 4
    caches = wl.global_caches(cfg, "hierarchical")
    assert [(c["rows"], c["reads_per_meta"]) for c in caches] == [(2048, 4), (512, 1)]
    assert wl.global_caches(cfg, "recursive") == caches[-1:]
    assert wl.global_caches(cfg, "flat")[0]["rows"] == 8192
    assert wl.global_kv_bytes_per_token(cfg, "flat") == 8192 * per_row
    assert wl.global_kv_bytes_per_token(cfg, "hierarchical") == (2048 / 4 + 512 / 16) * per_row
    assert wl.global_kv_bytes_per_token(cfg, "recursive") == 512 / 16 * per_row
    assert wl.global_kv_bytes_per_token(cfg, "recursive") * cfg.B == wl.coarse_kv_bytes(cfg) / cfg.compress


def test_other_hierarchies():
    """(2, 2), the paper's other ablation point, and three levels: the derived
    configurations, and the closed forms against a decode loop that advances level l
    once per C_{<=l} tokens."""
    c22 = wl.with_hierarchy(wl.CONFIGS[1], (2, 2))
    assert (c22.S, c22.compress, c22.C) == (2048, 4, 2) and wl.coarse_kv_bytes(c22) == 4 * wl.coarse_kv_bytes(wl.CONFIGS[1])
    c444 = wl.with_hierarchy(wl.CONFIGS[2], (4, 4, 4))
    assert (c444.S, c444.compress) == (2048, 64)
    c3 = wl.with_hierarchy(wl.CONFIGS[3], (2, 2))
    assert (c3.S, c3.shared_S) == (128, 8192)
    for lengths in ((2, 2), (4, 4, 4), (2, 4, 8)):
        T = 1024
        upto = np.cumprod(lengths)
        n = [0] * len(lengths)
        hier = rec = 0
        for t in range(1, T + 1):
            for l, u in enumerate(upto):
                if t % u == 0:
                    n[l] += 1
                    hier += n[l]
                    if l == len(lengths) - 1:
                        rec += n[l]
        assert wl.cumulative_global_rows(T, "hierarchical", lengths) == hier
        assert wl.cumulative_global_rows(T, "recursive", lengths) == rec
        caches = wl.global_caches(c444 if len(lengths) == 3 and lengths == (4, 4, 4) else
                                  wl.with_hierarchy(wl.CONFIGS[2], lengths), "hierarchical", lengths)
        assert [c["tokens_per_read"] for c in caches] == list(upto)
        assert [c["rows"] for c in caches] == [131072 // u for u in upto]


def test_chunk_inputs_structure():
    cfg = wl.CONFIGS[0]
    ch = wl.chunk_inputs(cfg, poison=True)
    assert ch["kc"].shape == (16, 2, 8, 64) and ch["len"].min() >= cfg.P + 1 and ch["len"].max() <= 8
    for c in range(cfg.Nc):
        assert np.all(ch["kc"][c, :, ch["len"][c]:] == 0x7FC1)
        assert not np.any(ch["kc"][c, :, : ch["len"][c]] == 0x7FC1)
    strict = wl.chunk_inputs(cfg, strict_paper=True)
    assert np.array_equal(strict["len"], ch["len"] - 1) and strict["len"].min() >= cfg.P
    big = wl.chunk_inputs(wl.scaled(wl.CONFIGS[4], B=8))
    assert set(np.unique(big["n_in"])) == set(range(1, 17))
    assert wl.chunk_kv_bytes(cfg, ch["len"]) == int(ch["len"].sum()) * 2 * 64 * 4


def test_shard_units_partitions_exactly():
    for n in (0, 1, 7, 64, 16384):
        for ws in (1, 2, 3, 8):
            parts = [wl.shard_units(n, ws, r) for r in range(ws)]
            assert parts[0][0] == 0 and parts[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(parts, parts[1:]))
            sizes = [b - a for a, b in parts]
            assert max(sizes) - min(sizes) <= 1
