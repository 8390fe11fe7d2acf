"""Helpers shared by the parity tests: run the oracle on a synthetic layer, run the CUDA
library on the same bytes, and compare masks with the tolerance band the tests state."""
from __future__ import annotations

import math
from typing import Dict, Optional

import numpy as np

from oracle import gvote_oracle as o


def oracle_kwargs(cfg, layer_id=0, seed=None):
    return dict(n_q_heads=cfg.n_q_heads, d_k=cfg.d_k, theta=cfg.rope_theta, S=cfg.S,
                p_nuc=float(np.float32(cfg.p_nuc)), n_f=cfg.n_f, n_s=cfg.n_s,
                seed=cfg.seed if seed is None else seed, layer_id=layer_id)


def k_band(a0: np.ndarray, p: float, band: float):
    """Range of |C0| allowed when the cumulative mass may be off by `band` at the boundary."""
    cs = np.cumsum(np.sort(a0)[::-1])
    lo = int(np.searchsorted(cs, p - band, side="left")) + 1      # first size with mass >= p - band
    hi = int(np.searchsorted(cs, p + band, side="left")) + 1      # first size with mass >= p + band
    return max(1, min(lo, a0.shape[0])), max(1, min(hi, a0.shape[0]))


def check_vote_against_oracle(Q: np.ndarray, K: np.ndarray, p: float, sel_mode: str, include_c0: bool,
                              gpu_mask: np.ndarray, gpu_b_step: np.ndarray, *, mass_band=1e-3,
                              logit_band=1e-3) -> Dict[str, float]:
    """Q [H_q, S+1, d_k], K [H_kv, N, d_k] fp64 (the oracle's operands); gpu_mask [H_kv, N] bool.

    Asserts: every |C0| lies in the mass band; every key the oracle rules in by more than the band
    is kept; every kept key is ruled in within the band.  Returns mismatch statistics."""
    H_q, S1, d_k = Q.shape
    H_kv, N, _ = K.shape
    G = H_q // H_kv
    must = np.zeros((H_kv, N), dtype=bool)
    may = np.zeros((H_kv, N), dtype=bool)
    for g in range(H_q):
        kh = g // G
        L = (Q[g] @ K[kh].T) / math.sqrt(d_k)
        A = o.softmax_rows(L)
        lo, hi = k_band(A[0], p, mass_band)
        kg = int(gpu_b_step[g])
        assert lo <= kg <= hi, f"head {g}: |C0| = {kg} outside [{lo}, {hi}]"
        rows = range(0 if include_c0 else 1, S1)
        for s in rows:
            if s == 0 or sel_mode == "topp":
                order = np.argsort(-A[s], kind="stable")
                before = np.concatenate([[0.0], np.cumsum(A[s][order])[:-1]])   # mass ahead of each key
                must[kh, order[before < p - mass_band]] = True
                may[kh, order[before < p + mass_band]] = True
            else:
                srt = np.sort(L[s])[::-1]
                Lk = srt[min(kg, N) - 1]
                eps = logit_band * max(1.0, abs(Lk))
                must[kh, L[s] > Lk + eps] = True
                may[kh, L[s] >= Lk - eps] = True
    missing = must & ~gpu_mask
    extra = gpu_mask & ~may
    assert not missing.any(), f"{int(missing.sum())} keys ruled in by the oracle are missing"
    assert not extra.any(), f"{int(extra.sum())} kept keys are outside the oracle's band"
    return {"band_keys": int((may & ~must).sum())}


def upload_layer(li, gv, torch, device="cuda"):
    """LayerInputs -> dict of device tensors."""
    d = dict(
        h=torch.from_numpy(li.h).to(device),
        W_q=gv.bf16_from_bits(li.W_q, device),
        b_q=None if li.b_q is None else torch.from_numpy(li.b_q).to(device),
        K=gv.bf16_from_bits(li.K, device),
        V=gv.bf16_from_bits(li.V, device),
        cu=torch.from_numpy(li.cu_seqlens).to(device),
    )
    return d


def to_group_major(Q: np.ndarray, G: int) -> np.ndarray:
    """Oracle query rows [H_q, S+1, d_k] (row 0 = current query) -> the library's layout
    [H_kv, G*S + G, d_k]: per KV head the S synthetic rows of each of its G heads, then the G
    current-query rows."""
    H_q, S1, d_k = Q.shape
    S, H_kv = S1 - 1, H_q // G
    out = np.empty((H_kv, G * S1, d_k), dtype=Q.dtype)
    for g in range(H_q):
        kh, gl = divmod(g, G)
        out[kh, gl * S:(gl + 1) * S] = Q[g, 1:]
        out[kh, G * S + gl] = Q[g, 0]
    return out


def from_group_major(Qg: np.ndarray, G: int) -> np.ndarray:
    H_kv, R, d_k = Qg.shape
    S1 = R // G
    S = S1 - 1
    out = np.empty((H_kv * G, S1, d_k), dtype=Qg.dtype)
    for g in range(H_kv * G):
        kh, gl = divmod(g, G)
        out[g, 1:] = Qg[kh, gl * S:(gl + 1) * S]
        out[g, 0] = Qg[kh, G * S + gl]
    return out
