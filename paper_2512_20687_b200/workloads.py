"""Seeded synthetic inputs for the PHOTON decode step (numpy only).

This module serves both the CUDA path and the CPU oracle and therefore holds
none of the method's arithmetic: it only draws numbers and lays them out.
Every tensor is a pure function of (seed, tensor name, element index) through
a counter-based generator, so any slice can be regenerated independently and
the oracle and the GPU always see identical bits.

Generator: element i of stream s under seed k is
    z  = splitmix64(key(k, s) + i)
    u1 = (top 24 bits of z + 0.5) / 2^24,  u2 = (low 24 bits of z + 0.5) / 2^24
    x  = std * sqrt(-2 ln u1) * cos(2 pi u2)            (Box-Muller)
computed in float64, cast to float32, then rounded to bf16 (round to nearest
even) and stored as raw uint16 bits.

Shapes follow the five benchmark configurations: a coarse KV cache of
S = T / (C1*C2) latents per sequence (hierarchy of Section 2.1, cache of
Eq. 12), a converter weight mapping one latent to P prefix vectors
(Section 2.1.2), and chunk-local caches of P + C rows (Eq. 6-7).
"""
from __future__ import annotations

import dataclasses
import zlib
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_GOLD = np.uint64(0x9E3779B97F4A7C15)
_MIX1 = np.uint64(0xBF58476D1CE4E5B9)
_MIX2 = np.uint64(0x94D049BB133111EB)


def _splitmix64(x: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = x + _GOLD
        z = (z ^ (z >> np.uint64(30))) * _MIX1
        z = (z ^ (z >> np.uint64(27))) * _MIX2
        return z ^ (z >> np.uint64(31))


def stream_key(seed: int, name: str) -> np.uint64:
    """64-bit key of a named tensor stream under a seed."""
    h = zlib.crc32(name.encode()) & 0xFFFFFFFF
    k = np.array([(int(seed) << 32) ^ h], dtype=np.uint64)
    return _splitmix64(_splitmix64(k))[0]


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 raw bits, round to nearest even (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """bf16 raw bits -> float64 (exact)."""
    u = np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def _normal_block(key: np.uint64, start: int, count: int, std: float) -> np.ndarray:
    idx = np.arange(start, start + count, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = _splitmix64(idx + key)
    u1 = ((z >> np.uint64(40)).astype(np.float64) + 0.5) * (1.0 / 16777216.0)
    u2 = ((z & np.uint64(0xFFFFFF)).astype(np.float64) + 0.5) * (1.0 / 16777216.0)
    x = np.sqrt(-2.0 * np.log(u1)) * np.cos((2.0 * np.pi) * u2)
    return f32_to_bf16_bits((x * std).astype(np.float32))


def normal_bf16(seed: int, name: str, shape, std: float = 1.0, offset: int = 0) -> np.ndarray:
    """bf16 bits of N(0, std^2) samples for the named stream, elements
    [offset, offset + prod(shape)) of that stream, in C order."""
    n = int(np.prod(shape, dtype=np.int64))
    key = stream_key(seed, name)
    out = np.empty(n, dtype=np.uint16)
    block = 1 << 22
    starts = list(range(0, n, block))

    def work(s):
        c = min(block, n - s)
        out[s:s + c] = _normal_block(key, offset + s, c, std)

    if len(starts) <= 1:
        for s in starts:
            work(s)
    else:
        with ThreadPoolExecutor(max_workers=8) as ex:
            list(ex.map(work, starts))
    return out.reshape(shape)


def uniform_int(seed: int, name: str, n: int, lo: int, hi: int) -> np.ndarray:
    """n int32 values uniform in [lo, hi] (inclusive)."""
    key = stream_key(seed, name)
    with np.errstate(over="ignore"):
        z = _splitmix64(np.arange(n, dtype=np.uint64) + key)
    span = np.uint64(hi - lo + 1)
    return (lo + ((z >> np.uint64(16)) % span).astype(np.int64)).astype(np.int32)


@dataclasses.dataclass(frozen=True)
class DecodeConfig:
    """One benchmark configuration of the decode step.

    B sequences; S coarse latents per sequence after the step's append
    (S = context / (C1*C2)); Hq/Hkv/dh attention heads; D model width
    (= Hq*dh); P prefix vectors and C chunk length of the local decoders;
    chunks_per_seq in-flight chunks per sequence; shared_S > 0 adds one
    shared document prefix of that many coarse latents stored once.
    tokens_per_step = number of token-level in-flight chunks.
    """
    name: str
    index: int
    B: int
    context: int
    S: int
    Hq: int
    Hkv: int
    dh: int
    D: int
    P: int
    C: int
    chunks_per_seq: int
    seed: int
    compress: int            # C_{<=L}: tokens per coarse latent
    shared_S: int = 0
    shared_context: int = 0
    tokens_per_step: int = 0

    @property
    def Nc(self) -> int:
        return self.B * self.chunks_per_seq

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv


CONFIGS = (
    DecodeConfig("tiny", 0, B=2, context=256, S=16, Hq=4, Hkv=2, dh=64, D=256, P=4, C=4,
                 chunks_per_seq=8, seed=0, compress=16, tokens_per_step=16),
    DecodeConfig("1b_class", 1, B=64, context=8192, S=512, Hq=16, Hkv=4, dh=128, D=2048, P=4, C=4,
                 chunks_per_seq=2, seed=1, compress=16, tokens_per_step=64),
    DecodeConfig("long_context", 2, B=16, context=131072, S=8192, Hq=16, Hkv=4, dh=128, D=2048,
                 P=4, C=4, chunks_per_seq=2, seed=2, compress=16, tokens_per_step=16),
    DecodeConfig("shared_prefix", 3, B=256, context=512, S=32, Hq=16, Hkv=4, dh=128, D=2048,
                 P=4, C=4, chunks_per_seq=2, seed=3, compress=16, shared_S=2048,
                 shared_context=32768, tokens_per_step=256),
    DecodeConfig("chunk_parallel", 4, B=512, context=2048, S=128, Hq=8, Hkv=8, dh=128, D=1024,
                 P=8, C=16, chunks_per_seq=32, seed=4, compress=16, tokens_per_step=512 * 32),
)


def scaled(cfg: DecodeConfig, **kw) -> DecodeConfig:
    """A copy of cfg with some fields replaced (for reduced-size test cases)."""
    return dataclasses.replace(cfg, **kw)


def with_hierarchy(cfg: DecodeConfig, chunk_lengths) -> DecodeConfig:
    """The same model shapes and context under another hierarchy (C_1, ..., C_L): the
    coarse stream holds context / prod(C_l) latents per sequence (a shared prefix
    likewise) and the token-level chunks are C_1 long.  (4, 4) is the hierarchy of the
    five configurations; the paper's ablation also runs (2, 2)."""
    total = int(np.prod(chunk_lengths))
    assert cfg.context % total == 0 and cfg.shared_context % total == 0
    return dataclasses.replace(
        cfg, name=f"{cfg.name}/{'x'.join(str(c) for c in chunk_lengths)}", compress=total,
        S=cfg.context // total, shared_S=cfg.shared_context // total, C=int(chunk_lengths[0]))


def coarse_inputs(cfg: DecodeConfig, replica: int = 0, poison: bool = False) -> dict:
    """Coarse-stream tensors for one decode step.

    The cache holds S-1 valid rows per sequence; the step appends row S-1
    and attends over S rows.  Rows >= len are zero, or NaN bit patterns
    when poison=True (they must never influence a result).
    Layout: k, v [B, Hkv, cap, dh] with cap = S; len [B].
    """
    tag = f"r{replica}"
    cap = cfg.S
    shape = (cfg.B, cfg.Hkv, cap, cfg.dh)
    k = normal_bf16(cfg.seed, f"coarse_k/{tag}", shape)
    v = normal_bf16(cfg.seed, f"coarse_v/{tag}", shape)
    fill = np.uint16(0x7FC1) if poison else np.uint16(0)
    k[:, :, cfg.S - 1:, :] = fill
    v[:, :, cfg.S - 1:, :] = fill
    out = {
        "k": k, "v": v, "cap": cap,
        "len": np.full(cfg.B, cfg.S - 1, dtype=np.int32),
        "k_new": normal_bf16(cfg.seed, f"k_new/{tag}", (cfg.B, cfg.Hkv, cfg.dh)),
        "v_new": normal_bf16(cfg.seed, f"v_new/{tag}", (cfg.B, cfg.Hkv, cfg.dh)),
        "q": normal_bf16(cfg.seed, f"coarse_q/{tag}", (cfg.B, cfg.Hq, cfg.dh)),
    }
    if cfg.shared_S:
        sshape = (1, cfg.Hkv, cfg.shared_S, cfg.dh)
        out.update({
            "k_shared": normal_bf16(cfg.seed, f"shared_k/{tag}", sshape),
            "v_shared": normal_bf16(cfg.seed, f"shared_v/{tag}", sshape),
            "shared_len": np.array([cfg.shared_S], dtype=np.int32),
            "shared_id": np.zeros(cfg.B, dtype=np.int32),
            "cap_shared": cfg.shared_S,
        })
    return out


def converter_inputs(cfg: DecodeConfig, replica: int = 0, with_bias: bool = False) -> dict:
    """Converter tensors: x [B, D] ~ N(0,1); weight ~ N(0, 1/D) drawn as the
    logical matrix W[k, n] (k input feature, n = r*D + j output column) and
    returned in both storage orders: w_in_major [D, P*D] and
    w_out_major [P*D, D] (its transpose)."""
    tag = f"r{replica}"
    w = normal_bf16(cfg.seed, f"conv_w/{tag}", (cfg.D, cfg.P * cfg.D), std=cfg.D ** -0.5)
    out = {
        "x": normal_bf16(cfg.seed, f"conv_x/{tag}", (cfg.B, cfg.D)),
        "w_in_major": w,
        "w_out_major": np.ascontiguousarray(w.T),
        "bias": None,
    }
    if with_bias:
        out["bias"] = normal_bf16(cfg.seed, f"conv_b/{tag}", (cfg.P * cfg.D,))
    return out


def chunker_inputs(cfg: DecodeConfig, replica: int = 0, block: int = 4) -> dict:
    """Level-L context chunker: per sequence the `block` reconstructed level-(L-1)
    latents of the meta-context just decoded, concatenated (x [B, block*D], N(0,1)),
    a per-feature scale around 1, a weight [block*D, D] of variance 1/(block*D) in
    both storage orders, and a bias."""
    tag = f"r{replica}"
    K = block * cfg.D
    w = normal_bf16(cfg.seed, f"chunker_w/{tag}", (K, cfg.D), std=K ** -0.5)
    g = bf16_bits_to_f64(normal_bf16(cfg.seed, f"chunker_g/{tag}", (K,), std=0.1)) + 1.0
    return {
        "x": normal_bf16(cfg.seed, f"chunker_x/{tag}", (cfg.B, K)),
        "gamma": f32_to_bf16_bits(g.astype(np.float32)),
        "w_in_major": w, "w_out_major": np.ascontiguousarray(w.T),
        "bias": normal_bf16(cfg.seed, f"chunker_b/{tag}", (cfg.D,), std=0.1),
        "eps": 1e-5, "K": K, "N": cfg.D,
    }


def encoder_layer_inputs(cfg: DecodeConfig, F: int | None = None, replica: int = 0) -> dict:
    """Weights of one LLaMA layer of the top-level encoder (in-major, variance 1/K
    each, norm scales around 1) and the step's input x [B, D].  F defaults to the
    multiple of 64 nearest to 2.75 D (5632 for D = 2048, the usual 1B-class width)."""
    tag = f"r{replica}"
    D, dh, Hq, Hkv = cfg.D, cfg.dh, cfg.Hq, cfg.Hkv
    F = F or max(64, int(round(2.75 * D / 64)) * 64)
    one = lambda name, n: f32_to_bf16_bits(
        (bf16_bits_to_f64(normal_bf16(cfg.seed, f"{name}/{tag}", (n,), std=0.1)) + 1.0).astype(np.float32))
    mat = lambda name, k, n: normal_bf16(cfg.seed, f"{name}/{tag}", (k, n), std=k ** -0.5)
    return {
        "x": normal_bf16(cfg.seed, f"enc_x/{tag}", (cfg.B, D)), "F": F,
        "g1": one("enc_g1", D), "wqkv": mat("enc_wqkv", D, (Hq + 2 * Hkv) * dh), "wo": mat("enc_wo", Hq * dh, D),
        "g2": one("enc_g2", D), "wgu": mat("enc_wgu", D, 2 * F), "wdown": mat("enc_wdown", F, D),
    }


def chunk_inputs(cfg: DecodeConfig, replica: int = 0, poison: bool = False,
                 strict_paper: bool = False) -> dict:
    """Chunk-local tensors: Nc in-flight chunks, each a cache of cap = P + C
    rows, layout kc, vc [Nc, Hkv, P+C, dh]; rows 0..P-1 are the prefix, rows
    P.. the in-chunk positions.  The in-chunk position p ~ U{0..C-1}; the
    query is in-chunk token p and sees itself, so n_in = p + 1 in-chunk rows
    are valid (len = P + n_in).  strict_paper=True gives n_in = p instead
    (the query is the latent before position p+1; Eq. 6 with j = p + 1)."""
    tag = f"r{replica}"
    Nc, cap = cfg.Nc, cfg.P + cfg.C
    p = uniform_int(cfg.seed, f"chunk_pos/{tag}", Nc, 0, cfg.C - 1)
    n_in = p if strict_paper else p + 1
    ln = (cfg.P + n_in).astype(np.int32)
    shape = (Nc, cfg.Hkv, cap, cfg.dh)
    kc = normal_bf16(cfg.seed, f"chunk_k/{tag}", shape)
    vc = normal_bf16(cfg.seed, f"chunk_v/{tag}", shape)
    fill = np.uint16(0x7FC1) if poison else np.uint16(0)
    invalid = np.arange(cap, dtype=np.int32)[None, :] >= ln[:, None]      # [Nc, cap]
    kc[np.broadcast_to(invalid[:, None, :, None], shape)] = fill
    vc[np.broadcast_to(invalid[:, None, :, None], shape)] = fill
    return {
        "kc": kc, "vc": vc, "cap": cap, "len": ln, "n_in": n_in.astype(np.int32),
        "q": normal_bf16(cfg.seed, f"chunk_q/{tag}", (Nc, cfg.Hq, cfg.dh)),
    }


def chunk_causal_inputs(cfg: DecodeConfig, replica: int = 0, poison: bool = False,
                        full: bool = False, row0: int = 0, rows: int | None = None) -> dict:
    """The chunk buffers of chunk_inputs with a query for `rows` consecutive
    positions of every chunk, starting at row `row0` (default: all P + C rows):
    q [Nc, rows, Hq, dh].  full=True makes every chunk complete (len = P + C),
    the teacher-forced whole-chunk case; otherwise the lengths are the ragged
    ones of chunk_inputs and positions >= len do not exist yet."""
    tag = f"r{replica}"
    a = chunk_inputs(cfg, replica=replica, poison=poison and not full)
    cap = a["cap"]
    rows = cap - row0 if rows is None else rows
    if full:
        shape = (cfg.Nc, cfg.Hkv, cap, cfg.dh)
        a["kc"] = normal_bf16(cfg.seed, f"chunk_k/{tag}", shape)
        a["vc"] = normal_bf16(cfg.seed, f"chunk_v/{tag}", shape)
        a["len"] = np.full(cfg.Nc, cap, np.int32)
        a["n_in"] = np.full(cfg.Nc, cfg.C, np.int32)
    a["q"] = normal_bf16(cfg.seed, f"chunk_qrows/{tag}", (cfg.Nc, rows, cfg.Hq, cfg.dh))
    a["row0"], a["rows"] = row0, rows
    return a


def step_inputs(cfg: DecodeConfig, replica: int = 0, poison: bool = False) -> dict:
    """Everything one decode step consumes."""
    return {
        "coarse": coarse_inputs(cfg, replica, poison),
        "converter": converter_inputs(cfg, replica),
        "chunks": chunk_inputs(cfg, replica, poison),
    }


# ---- algorithmic byte counts (what the method itself must move) -----------

def coarse_kv_bytes(cfg: DecodeConfig) -> int:
    """K+V bytes the coarse attention must read in one step: every valid row
    of every sequence once, a shared prefix once for all branches."""
    per_row = cfg.Hkv * cfg.dh * 2 * 2
    return (cfg.B * cfg.S + cfg.shared_S) * per_row


def flat_kv_bytes(cfg: DecodeConfig) -> int:
    """K+V bytes a token-level cache of the same context would need."""
    per_row = cfg.Hkv * cfg.dh * 2 * 2
    return (cfg.B * cfg.context + cfg.shared_context) * per_row


# ---- global caches of the generation schedules (Sections 2.3.2 and 2.3.3) ----

SCHEDULES = ("flat", "hierarchical", "recursive")


def global_caches(cfg: DecodeConfig, schedule: str, chunk_lengths=(4, 4)) -> list[dict]:
    """The context-growing caches a schedule keeps for a context of cfg.context
    tokens per sequence, and how often each is read while C_{<=L} tokens (one
    meta-context) are generated.  A flat Transformer keeps one token-level
    cache and reads it for every token.  Hierarchical generation keeps a
    global cache at every level l (T / C_{<=l} rows) and advances level l once
    per level-l chunk, i.e. C_{<=L} / C_{<=l} times per meta-context.
    Recursive generation keeps the top level only and reads it once.
    Returns [{level, rows, reads_per_meta, tokens_per_read}], lowest level first."""
    assert schedule in SCHEDULES
    total = int(np.prod(chunk_lengths))
    assert total == cfg.compress
    ctx = cfg.context + cfg.shared_context
    if schedule == "flat":
        return [{"level": 0, "rows": ctx, "reads_per_meta": total, "tokens_per_read": 1}]
    out, upto = [], 1
    for level, c in enumerate(chunk_lengths, start=1):
        upto *= c
        out.append({"level": level, "rows": ctx // upto, "reads_per_meta": total // upto,
                    "tokens_per_read": upto})
    return out if schedule == "hierarchical" else out[-1:]


def global_kv_bytes_per_token(cfg: DecodeConfig, schedule: str, chunk_lengths=(4, 4)) -> float:
    """K+V bytes of the global caches read per generated token and sequence at
    the context length of the workload: sum over levels of rows * bytes per row
    / tokens per read."""
    per_row = cfg.Hkv * cfg.dh * 2 * 2
    return sum(c["rows"] * per_row / c["tokens_per_read"] for c in global_caches(cfg, schedule, chunk_lengths))


def cumulative_global_rows(T: int, schedule: str, chunk_lengths=(4, 4)) -> int:
    """Cache rows read by the global attention while T tokens are generated from
    an empty context: level l advances once per C_{<=l} tokens and its step g
    attends g rows, sum_{g=1}^{M_l} g with M_l = T / C_{<=l} (the cumulative
    global KV reads of Section 2.3.2); level 0 is the flat Transformer."""
    assert schedule in SCHEDULES
    tri = lambda m: m * (m + 1) // 2
    if schedule == "flat":
        return tri(T)
    upto, per_level = 1, []
    for c in chunk_lengths:
        upto *= c
        per_level.append(tri(T // upto))
    return sum(per_level) if schedule == "hierarchical" else per_level[-1]


def chunk_kv_bytes(cfg: DecodeConfig, lens: np.ndarray) -> int:
    return int(lens.astype(np.int64).sum()) * cfg.Hkv * cfg.dh * 2 * 2


def shard_units(n_units: int, world_size: int, rank: int) -> tuple[int, int]:
    """Contiguous [lo, hi) slice of independent units (sequences or chunks)
    owned by a rank; remainders go to the lowest ranks."""
    base, rem = divmod(n_units, world_size)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)
