"""Seeded synthetic inputs for the GVote compression pass.

This module only manufactures tensors (hidden states, W_q, K, V, cu_seqlens) with the
shapes, length regimes and attention sparsity of the paper's workloads (Section 4.1:
Llama-3.x / Qwen2.5 models on short, 4K, 34K, 51K and >128K contexts).  It serves both the
CPU oracle and the CUDA path with byte-identical inputs and contains none of the method's
steps: no fit, no sampling, no scoring, no selection.

The one piece of geometry it needs is where to point the planted "heavy" keys.  Real
models store keys already rotated by RoPE, so a planted key is built the same way: the
mean hidden state is pushed through one query head's rows of W_q and the result is turned
by an ordinary rotate-half RoPE rotation at the midpoint of the future-position window.
A mistake here would only make the synthetic attention less sparse; neither the oracle
nor the kernels ever see this direction.

All arrays are NumPy.  bf16 tensors are carried as uint16 bit patterns (NumPy has no
bf16); `bf16_to_f32` widens them exactly.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Sequence

import numpy as np


# ----------------------------------------------------------------------------- bf16 helpers
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even), returned as uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    bits = x.view(np.uint32)
    lsb = (bits >> np.uint32(16)) & np.uint32(1)
    rounded = bits + np.uint32(0x7FFF) + lsb
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to float32 exactly."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32)


# ----------------------------------------------------------------------------- configs
@dataclass(frozen=True)
class GVoteConfig:
    """Shape and hyper-parameters of one workload (one entry of the benchmark list)."""

    name: str
    d_h: int                 # hidden size
    n_q_heads: int
    n_kv_heads: int
    d_k: int                 # head dim
    rope_theta: float
    S: int                   # synthetic queries per request
    p_nuc: float             # nucleus mass threshold
    seq_lens: Sequence[int]  # cached tokens per request (ragged batch)
    n_layers: int = 1
    n_f: int = 128           # future positions averaged by RoPE
    n_s: int = 4             # sink tokens skipped by the fit
    seed: int = 0
    # --- input-shaping knobs (not hyper-parameters of the method) ---
    h_mode: str = "standard"         # "standard": N(0,1);  "diag": N(mu, diag Sigma)
    n_outlier_channels: int = 4
    outlier_scale: float = 8.0
    heavy_frac: Sequence[float] = (0.01,)   # per request (or broadcast)
    heavy_count: Optional[int] = None       # overrides heavy_frac when set
    heavy_frac_layer_range: Optional[Sequence[float]] = None  # per-layer U[lo,hi]
    heavy_lead: float = 8.0          # target logit lead of a planted key for the mean query
    heavy_norm_cap: float = 1.0      # planted offset norm <= cap * sqrt(d_k)
    heavy_gain: float = 2.5          # planted rows also carry this multiple of the N(0,1) row
    local_window: int = 0            # last tokens with a weaker planted offset
    local_scale: float = 0.25
    key_scale: float = 1.0           # standard deviation of an ordinary key row's entries
    heavy_all_heads: bool = False    # planted keys line up with every query head of the group, not only its first

    @property
    def G(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def batch(self) -> int:
        return len(self.seq_lens)

    @property
    def total_tokens(self) -> int:
        return int(sum(self.seq_lens))

    def cu_seqlens(self) -> np.ndarray:
        cu = np.zeros(self.batch + 1, dtype=np.int32)
        cu[1:] = np.cumsum(np.asarray(self.seq_lens, dtype=np.int64))
        return cu


def _ragged_lengths(seed: int) -> List[int]:
    rng = np.random.default_rng(seed)
    short = rng.integers(256, 1024, size=8, endpoint=True)
    long_ = rng.integers(4096, 16384, size=8, endpoint=True)
    # interleave so neighbouring work items differ in size
    out: List[int] = []
    for a, b in zip(short, long_):
        out += [int(a), int(b)]
    return out


def make_config(name: str, **overrides) -> GVoteConfig:
    """The five benchmark workloads, by name: c0 … c4."""
    if name == "c0":
        cfg = GVoteConfig(name="c0", d_h=512, n_q_heads=8, n_kv_heads=2, d_k=64,
                          rope_theta=1.0e4, S=16, p_nuc=0.95, seq_lens=(512,), seed=0,
                          h_mode="standard", n_outlier_channels=3, heavy_count=16)
    elif name == "c1":
        cfg = GVoteConfig(name="c1", d_h=4096, n_q_heads=32, n_kv_heads=8, d_k=128,
                          rope_theta=5.0e5, S=32, p_nuc=0.95, seq_lens=(4096,), seed=1,
                          h_mode="diag", heavy_frac=(0.01,))
    elif name == "c2":
        cfg = GVoteConfig(name="c2", d_h=4096, n_q_heads=32, n_kv_heads=8, d_k=128,
                          rope_theta=5.0e5, S=32, p_nuc=0.95, seq_lens=(32768,), seed=2,
                          n_layers=32, h_mode="diag", heavy_frac_layer_range=(0.002, 0.05))
    elif name == "c3":
        lens = _ragged_lengths(3)
        fr = [0.10 if n <= 1024 else 0.005 for n in lens]
        cfg = GVoteConfig(name="c3", d_h=4096, n_q_heads=32, n_kv_heads=8, d_k=128,
                          rope_theta=5.0e5, S=32, p_nuc=0.95, seq_lens=tuple(lens), seed=3,
                          h_mode="diag", heavy_frac=tuple(fr))
    elif name == "c4":
        cfg = GVoteConfig(name="c4", d_h=3584, n_q_heads=28, n_kv_heads=4, d_k=128,
                          rope_theta=1.0e6, S=64, p_nuc=0.98, seq_lens=(131072,), seed=4,
                          n_layers=28, h_mode="diag", heavy_frac=(0.001,), local_window=512,
                          heavy_gain=4.0)
    else:
        raise ValueError(f"unknown config {name!r}")
    return replace(cfg, **overrides) if overrides else cfg


# ----------------------------------------------------------------------------- generators
@dataclass
class LayerInputs:
    """Inputs of one layer's compression pass (all requests of the batch packed)."""

    h: np.ndarray            # [total_tokens, d_h] float32, layer-norm output
    W_q: np.ndarray          # [n_q_heads*d_k, d_h] bf16 bits (one row per output feature)
    b_q: Optional[np.ndarray]  # [n_q_heads*d_k] float32 or None
    K: np.ndarray            # [n_kv_heads, total_tokens, d_k] bf16 bits
    V: np.ndarray            # [n_kv_heads, total_tokens, d_k] bf16 bits
    cu_seqlens: np.ndarray   # [batch+1] int32
    layer_id: int
    heavy_positions: Dict = field(default_factory=dict)  # (request, kv_head) -> int64 array


def _planted_direction(W_q_f32: np.ndarray, mean_h: np.ndarray, head: int, d_k: int,
                       theta: float, position: float) -> np.ndarray:
    """Unit vector a stored (already RoPE-rotated) key would need to point along to line
    up with the mean hidden state seen through query head `head`."""
    rows = W_q_f32[head * d_k:(head + 1) * d_k].astype(np.float64)
    m = rows @ mean_h.astype(np.float64)
    half = d_k // 2
    ang = position * theta ** (-2.0 * np.arange(half) / d_k)
    c, s = np.cos(ang), np.sin(ang)
    out = np.empty(d_k)
    out[:half] = m[:half] * c - m[half:] * s
    out[half:] = m[half:] * c + m[:half] * s
    nrm = np.linalg.norm(out)
    return out / nrm if nrm > 0 else out


def layer_rng(cfg: GVoteConfig, layer: int) -> np.random.Generator:
    return np.random.default_rng([cfg.seed, layer, 0x6A09E667])


def make_layer(cfg: GVoteConfig, layer: int = 0, with_bias: bool = False) -> LayerInputs:
    """Generate one layer's inputs.  Deterministic in (cfg, layer)."""
    rng = layer_rng(cfg, layer)
    d_h, d_k, Hq, Hkv, G = cfg.d_h, cfg.d_k, cfg.n_q_heads, cfg.n_kv_heads, cfg.G
    cu = cfg.cu_seqlens()
    T = cfg.total_tokens

    W = rng.standard_normal((Hq * d_k, d_h), dtype=np.float32) * np.float32(1.0 / np.sqrt(d_h))
    W_bits = f32_to_bf16_bits(W)
    W_f32 = bf16_to_f32(W_bits)
    b_q = (rng.standard_normal(Hq * d_k, dtype=np.float32) * np.float32(0.1)) if with_bias else None

    h = np.empty((T, d_h), dtype=np.float32)
    K = np.empty((Hkv, T, d_k), dtype=np.float32)
    heavy_positions: Dict = {}

    outlier_ch = rng.choice(d_k, size=cfg.n_outlier_channels, replace=False)
    if cfg.heavy_frac_layer_range is not None:
        lo, hi = cfg.heavy_frac_layer_range
        layer_frac = float(rng.uniform(lo, hi))
    else:
        layer_frac = None

    for r in range(cfg.batch):
        a, b = int(cu[r]), int(cu[r + 1])
        N = b - a
        z = rng.standard_normal((N, d_h), dtype=np.float32)
        if cfg.h_mode == "diag":
            mu = rng.standard_normal(d_h).astype(np.float32) * np.float32(0.1)
            var = np.exp(rng.uniform(np.log(0.1), np.log(10.0), size=d_h))
            z *= np.sqrt(var).astype(np.float32)
            z += mu
        elif cfg.h_mode == "mean":
            # hidden states that hardly move around a large mean: every query, current or synthetic,
            # then points almost the same way (the regime in which planted keys have a known fate)
            z *= np.float32(0.02)
            z += rng.standard_normal(d_h).astype(np.float32)
        h[a:b] = z
        mean_h = h[a + min(cfg.n_s, max(N - 1, 0)):b].mean(axis=0, dtype=np.float64)

        if layer_frac is not None:
            frac = layer_frac
        else:
            frac = cfg.heavy_frac[r] if r < len(cfg.heavy_frac) else cfg.heavy_frac[-1]
        n_heavy = cfg.heavy_count if cfg.heavy_count is not None else max(1, int(round(frac * N)))
        n_heavy = min(n_heavy, N)
        pos_star = N + 0.5 * (cfg.n_f - 1)

        for kh in range(Hkv):
            Kn = rng.standard_normal((N, d_k), dtype=np.float32) * np.float32(cfg.key_scale)
            mhat = _planted_direction(W_f32, mean_h, kh * G, d_k, cfg.rope_theta, pos_star)
            if cfg.heavy_all_heads:
                for g in range(kh * G + 1, (kh + 1) * G):
                    mhat = mhat + _planted_direction(W_f32, mean_h, g, d_k, cfg.rope_theta, pos_star)
            # norm of the mean query seen through this head (before rotation; rotation keeps it)
            m_norm = np.linalg.norm(W_f32[kh * G * d_k:(kh * G + 1) * d_k].astype(np.float64) @ mean_h)
            alpha = cfg.heavy_lead * np.sqrt(d_k) / max(m_norm, 1e-12)
            alpha = min(alpha, cfg.heavy_norm_cap * np.sqrt(d_k))
            pos = np.sort(rng.choice(N, size=n_heavy, replace=False))
            Kn[pos] = Kn[pos] * np.float32(cfg.heavy_gain) + (alpha * mhat).astype(np.float32)
            if cfg.local_window > 0:
                w0 = max(0, N - cfg.local_window)
                Kn[w0:] += (cfg.local_scale * alpha * mhat).astype(np.float32)
            Kn[:, outlier_ch] *= np.float32(cfg.outlier_scale)
            K[kh, a:b] = Kn
            heavy_positions[(r, kh)] = pos.astype(np.int64)

    V = rng.standard_normal((Hkv, T, d_k), dtype=np.float32)
    return LayerInputs(h=h, W_q=W_bits, b_q=b_q, K=f32_to_bf16_bits(K), V=f32_to_bf16_bits(V),
                       cu_seqlens=cu, layer_id=layer, heavy_positions=heavy_positions)


def make_planted(n_heavy: int, seed: int = 40, N: int = 600, S: int = 8, p_nuc: float = 0.9,
                 n_q_heads: int = 4, n_kv_heads: int = 2, d_k: int = 64, d_h: int = 64) -> GVoteConfig:
    """A workload whose answer is known by construction: hidden states with a dominant mean (all queries
    nearly parallel), small ordinary keys, and n_heavy planted keys per KV head lined up with every query
    head of the group, far enough ahead that they hold more than p of every query's attention between
    them.  The nucleus of every query then lies inside the planted set, and so does every vote."""
    return GVoteConfig(name=f"planted{n_heavy}", d_h=d_h, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, d_k=d_k,
                       rope_theta=1.0e4, S=S, p_nuc=p_nuc, seq_lens=(N,), n_f=8, n_s=2, seed=seed, h_mode="mean",
                       n_outlier_channels=0, heavy_count=n_heavy, heavy_lead=16.0, heavy_norm_cap=1.0e6,
                       heavy_gain=0.0, key_scale=0.25, heavy_all_heads=True)


def make_small(seed: int, d_h: int = 64, n_q_heads: int = 4, n_kv_heads: int = 2, d_k: int = 32,
               seq_lens: Sequence[int] = (40,), S: int = 4, p_nuc: float = 0.9,
               theta: float = 1.0e4, n_f: int = 8, n_s: int = 2, **kw) -> GVoteConfig:
    """A free-form small configuration for unit tests and edge cases."""
    return GVoteConfig(name=f"small{seed}", d_h=d_h, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads,
                       d_k=d_k, rope_theta=theta, S=S, p_nuc=p_nuc, seq_lens=tuple(seq_lens),
                       n_f=n_f, n_s=n_s, seed=seed, h_mode=kw.pop("h_mode", "diag"),
                       n_outlier_channels=kw.pop("n_outlier_channels", 2),
                       heavy_frac=kw.pop("heavy_frac", (0.05,)), **kw)
