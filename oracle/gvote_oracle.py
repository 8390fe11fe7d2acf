"""CPU oracle for the GVote compression pass — TEST INFRASTRUCTURE, not the product.

A plain, slow, fp64 NumPy restatement of Algorithm 1 ("GVote: Adaptive Monte-Carlo
KV-cache compression") and Steps 1-4 of Section 3.2, taken step by step in the paper's
order and notation.  Only the tests, the smoke check and the benchmark's CPU-baseline leg
may import it; the CUDA library never does, and the two share no code.  The only thing
both sides implement alike is the published integer definition of Philox4x32-10 and the
counter layout that keys it.

No blocking, fusion or reordering: a matmul, a sort and a cumulative sum are used as
library steps, everything else is written out.  Floating point is fp64 throughout.  The
places where the GPU data path rounds to bf16 (the projection's input rows and the rotated
queries) are mirrored as explicit rounding steps when `mirror_rounding=True`.

Readings of the paper where it is silent (each is a parameter or stated where used):
  * selection for synthetic queries: top-k with k = |C0| (Algorithm 1, TopK step; Section 3.1
    last paragraph) is the default `sel_mode="topk"`; `sel_mode="topp"` applies the
    Section 3.1 top-p rule to every synthetic row instead;
  * Q0 is the query of the last cached token; one A0 row and one k per query head;
  * variance is the unbiased estimator; the first n_s rows are skipped (Step 2);
  * future positions are N .. N+n_f-1; RoPE is rotate-half with w_j = theta^(-2j/d_k);
  * top-p keeps the shortest prefix, in (weight desc, index asc) order, whose running sum
    reaches p (the crossing element is kept); top-k ties go to the lower index;
  * applying the pass again to a pruned cache (`recompress_request`, beyond the paper): every
    query head votes over the rows its own KV head still holds; positions come from the
    number of tokens seen, not from the number of rows stored.

Parity status: every function below is pinned by tests/ against closed forms, brute
force, published known-answer vectors or textbook library routines, except the end-to-end
masks and budgets of `compress`, for which the paper prints no worked example: there the
header says it plainly — end-to-end parity unpinned by the paper; it rests on the pinned
parts plus the invariants of Section 3.3 (union contains every voter's set, |union| >= |C|).
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

# ----------------------------------------------------------------------------- bf16
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to fp64."""
    w = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return w.view(np.float32).astype(np.float64)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even to the bf16 grid, result kept in fp64.

    Written as arithmetic on the value (not on float32 bit patterns): the value is first
    rounded to fp32 (the GPU holds it in fp32 at that point), then to 8 significant bits.
    """
    x32 = np.asarray(x, dtype=np.float64).astype(np.float32).astype(np.float64)
    out = np.zeros_like(x32)
    nz = x32 != 0.0
    m, e = np.frexp(x32[nz])            # x = m * 2^e, 0.5 <= |m| < 1
    e = np.maximum(e, -125)             # bf16 subnormals share the exponent of 2^-126
    m = x32[nz] / np.ldexp(1.0, e)
    q = np.rint(m * 256.0) / 256.0      # 8 significant bits; np.rint is ties-to-even
    out[nz] = np.ldexp(q, e)
    return out


# ----------------------------------------------------------------------------- Philox
PHILOX_M0 = 0xD2511F53
PHILOX_M1 = 0xCD9E8D57
PHILOX_W0 = 0x9E3779B9
PHILOX_W1 = 0xBB67AE85


def philox4x32_10(counter: np.ndarray, key: Tuple[int, int]) -> np.ndarray:
    """Philox4x32 with 10 rounds (Salmon et al., "Parallel random numbers: as easy as
    1, 2, 3", SC'11).  `counter` is [..., 4] uint32; returns [..., 4] uint32."""
    c = np.asarray(counter, dtype=np.uint64) & np.uint64(0xFFFFFFFF)
    c0, c1, c2, c3 = c[..., 0], c[..., 1], c[..., 2], c[..., 3]
    k0, k1 = int(key[0]) & 0xFFFFFFFF, int(key[1]) & 0xFFFFFFFF
    mask = np.uint64(0xFFFFFFFF)
    for rnd in range(10):
        p0 = np.uint64(PHILOX_M0) * c0          # 64-bit products of 32-bit values
        p1 = np.uint64(PHILOX_M1) * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & mask
        hi1, lo1 = p1 >> np.uint64(32), p1 & mask
        c0, c1, c2, c3 = (hi1 ^ c1 ^ np.uint64(k0)), lo1, (hi0 ^ c3 ^ np.uint64(k1)), lo0
        k0 = (k0 + PHILOX_W0) & 0xFFFFFFFF
        k1 = (k1 + PHILOX_W1) & 0xFFFFFFFF
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def gvote_philox_raw(S: int, d_h: int, seed: int, layer_id: int, request_id: int) -> np.ndarray:
    """The u32 stream behind the S x d_h normal draws: counter = (c div 4, s, layer, request),
    key = (seed low word, seed high word); the four outputs serve channels 4b..4b+3.
    Returns [S, 4*ceil(d_h/4)] uint32."""
    nb = (d_h + 3) // 4
    ctr = np.zeros((S, nb, 4), dtype=np.uint32)
    ctr[..., 0] = np.arange(nb, dtype=np.uint32)[None, :]
    ctr[..., 1] = np.arange(S, dtype=np.uint32)[:, None]
    ctr[..., 2] = np.uint32(layer_id & 0xFFFFFFFF)
    ctr[..., 3] = np.uint32(request_id & 0xFFFFFFFF)
    out = philox4x32_10(ctr, (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF))
    return out.reshape(S, nb * 4)


def uniform_open01(x: np.ndarray) -> np.ndarray:
    """u = ((x >> 9) + 0.5) * 2^-23: the top 23 bits plus a half-step offset, so u lies strictly
    inside (0, 1) and needs 24 significant bits at most — exact in fp32 as well as fp64."""
    return ((np.asarray(x, dtype=np.uint32) >> np.uint32(9)).astype(np.float64) + 0.5) * 2.0 ** -23


def box_muller(raw: np.ndarray) -> np.ndarray:
    """Standard normals from u32 words, pairwise: words (4b, 4b+1) give channels 4b, 4b+1 as
    r*cos(2 pi u1), r*sin(2 pi u1) with r = sqrt(-2 ln u0); words (4b+2, 4b+3) likewise."""
    u = uniform_open01(raw)
    u0, u1 = u[..., 0::2], u[..., 1::2]
    r = np.sqrt(-2.0 * np.log(u0))
    z = np.empty_like(u)
    z[..., 0::2] = r * np.cos(2.0 * math.pi * u1)
    z[..., 1::2] = r * np.sin(2.0 * math.pi * u1)
    return z


# ----------------------------------------------------------------------------- Step 2: fit
def fit(h: np.ndarray, n_s: int) -> Tuple[np.ndarray, np.ndarray]:
    """Step 2 of Section 3.2 (the Gaussian fit of Algorithm 1): per-channel mean and (unbiased) variance of the
    hidden states along the sequence axis, ignoring the first n_s (sink) tokens."""
    x = np.asarray(h, dtype=np.float64)[n_s:]
    T = x.shape[0]
    if T < 2:
        raise ValueError("fit needs at least two rows after the sink tokens")
    mu = x.sum(axis=0) / T
    d = x - mu
    var = (d * d).sum(axis=0) / (T - 1)
    return mu, var


@dataclass
class FitState:
    """Running moments of the hidden states seen so far (per channel): count, mean and the sum of
    squared deviations from the mean."""
    n: int
    mean: np.ndarray
    m2: np.ndarray


def fit_state(rows: np.ndarray) -> FitState:
    """Moments of a block of hidden-state rows [T, d_h] (T may be 0)."""
    x = np.asarray(rows, dtype=np.float64)
    T = x.shape[0]
    if T == 0:
        z = np.zeros(x.shape[1])
        return FitState(0, z, z.copy())
    mean = x.sum(axis=0) / T
    d = x - mean
    return FitState(T, mean, (d * d).sum(axis=0))


def fit_merge(a: FitState, b: FitState) -> FitState:
    """Moments of the union of two disjoint blocks from their moments (the pairwise update of
    Chan, Golub and LeVeque): the Gaussian of Step 2 can be fitted while the prompt streams by,
    block by block, without keeping the hidden states."""
    if a.n == 0:
        return FitState(b.n, b.mean.copy(), b.m2.copy())
    if b.n == 0:
        return FitState(a.n, a.mean.copy(), a.m2.copy())
    n = a.n + b.n
    delta = b.mean - a.mean
    return FitState(n, a.mean + delta * (b.n / n), a.m2 + b.m2 + delta * delta * (a.n * b.n / n))


def fit_finish(s: FitState) -> Tuple[np.ndarray, np.ndarray]:
    """Step 2's (mu, unbiased variance) from running moments."""
    if s.n < 2:
        raise ValueError("fit needs at least two rows")
    return s.mean.copy(), s.m2 / (s.n - 1)


# ----------------------------------------------------------------------------- Step 3: sample
def sample(mu: np.ndarray, var: np.ndarray, S: int, seed: int, layer_id: int,
           request_id: int) -> Tuple[np.ndarray, np.ndarray]:
    """Step 3 of Section 3.2 (the sampling step of Algorithm 1): H~ in R^{S x d_h} drawn from N(mu, diag var).
    Returns (H~, raw u32 words)."""
    d_h = mu.shape[0]
    raw = gvote_philox_raw(S, d_h, seed, layer_id, request_id)
    z = box_muller(raw)[:, :d_h]
    return mu[None, :] + np.sqrt(var)[None, :] * z, raw


# ----------------------------------------------------------------------------- RoPE
def rope_frequencies(d_k: int, theta: float) -> np.ndarray:
    j = np.arange(d_k // 2, dtype=np.float64)
    return theta ** (-2.0 * j / d_k)


def average_cos_sin(N: int, n_f: int, d_k: int, theta: float) -> Tuple[np.ndarray, np.ndarray]:
    """AverageCosSin of Algorithm 1: mean of cos and of sin over the n_f future positions
    N, N+1, ..., N+n_f-1, per RoPE frequency.  Direct summation."""
    w = rope_frequencies(d_k, theta)
    cbar = np.zeros_like(w)
    sbar = np.zeros_like(w)
    for i in range(n_f):
        cbar += np.cos((N + i) * w)
        sbar += np.sin((N + i) * w)
    return cbar / n_f, sbar / n_f


def rope_apply(x: np.ndarray, c: np.ndarray, s: np.ndarray) -> np.ndarray:
    """Rotate-half RoPE with per-frequency (c, s): pairs (j, j + d_k/2)."""
    half = x.shape[-1] // 2
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


# ----------------------------------------------------------------------------- attention rows
def softmax_rows(L: np.ndarray) -> np.ndarray:
    """Eq. 1: softmax along the key axis."""
    m = L.max(axis=-1, keepdims=True)
    e = np.exp(L - m)
    return e / e.sum(axis=-1, keepdims=True)


def top_p_set(a: np.ndarray, p: float) -> np.ndarray:
    """TopP (the set C0 of Algorithm 1; Section 3.1): the minimal set of keys whose weights reach
    cumulative mass p.  Keys are taken by (weight desc, index asc); the key that crosses
    p is kept.  Returns the selected indices in that order."""
    order = np.argsort(-a, kind="stable")
    csum = np.cumsum(a[order])
    hit = np.nonzero(csum >= p)[0]
    n = int(hit[0]) + 1 if hit.size else a.shape[0]
    return order[:n]


def top_k_set(l: np.ndarray, k: int) -> np.ndarray:
    """TopK on logits (the TopK step of Algorithm 1); ties go to the lower index; k clamps to N."""
    k = max(0, min(int(k), l.shape[0]))
    return np.argsort(-l, kind="stable")[:k]


# ----------------------------------------------------------------------------- projection
def project_queries(X: np.ndarray, W_q: np.ndarray, b_q: Optional[np.ndarray], n_q_heads: int,
                    d_k: int) -> np.ndarray:
    """X [rows, d_h] times the stored weight W_q [n_q_heads*d_k, d_h] (one row per output
    feature, i.e. the paper's W_q transposed) -> [n_q_heads, rows, d_k]."""
    q = X @ W_q.T
    if b_q is not None:
        q = q + np.asarray(b_q, dtype=np.float64)[None, :]
    return q.reshape(X.shape[0], n_q_heads, d_k).transpose(1, 0, 2)


@dataclass
class RequestResult:
    mu: np.ndarray
    var: np.ndarray
    H_tilde: np.ndarray                # [S, d_h]
    Q: np.ndarray                      # [H_q, S+1, d_k] rotated (and rounded if mirrored); row 0 real
    b_step: np.ndarray                 # [H_q] int   k_g = |C0| of query head g
    mask: np.ndarray                   # [H_kv, N] bool  keep-set per KV head
    budget: np.ndarray                 # [H_kv] int
    row_sets: Optional[List[List[np.ndarray]]] = None   # [H_q][S+1] selected indices
    probs: Optional[np.ndarray] = None                  # [H_q, S+1, N] softmax rows


def queries_for_request(H_tilde: np.ndarray, h_last: np.ndarray, W_q: np.ndarray,
                        b_q: Optional[np.ndarray], N: int, *, n_q_heads: int, d_k: int,
                        theta: float, n_f: int, mirror_rounding: bool = True) -> np.ndarray:
    """Algorithm 1, the current query Q0 and the synthetic queries Q~ (AverageCosSin, RoPE): project [h_last; H~] through W_q; rotate row 0
    exactly at position N-1 and rows 1..S with the averaged cos/sin of positions N..N+n_f-1.
    Returns [H_q, S+1, d_k]."""
    X = np.concatenate([np.asarray(h_last, dtype=np.float64)[None, :], H_tilde], axis=0)
    if mirror_rounding:
        X = round_to_bf16(X)
    q = project_queries(X, W_q, b_q, n_q_heads, d_k)
    w = rope_frequencies(d_k, theta)
    c0, s0 = np.cos((N - 1) * w), np.sin((N - 1) * w)
    cbar, sbar = average_cos_sin(N, n_f, d_k, theta)
    out = np.empty_like(q)
    out[:, 0] = rope_apply(q[:, 0], c0, s0)
    out[:, 1:] = rope_apply(q[:, 1:], cbar, sbar)
    if mirror_rounding:
        out = round_to_bf16(out)
    return out


def vote(Q: np.ndarray, K: np.ndarray, *, p_nuc: float, sel_mode: str = "topk",
         include_c0: bool = False, keep_rows: bool = False, keep_probs: bool = False):
    """Algorithm 1 for one request, from the queries on: the current-query steps (A0, C0, B_step) and the
    vote (logits, TopK, union).

    Q [H_q, S+1, d_k] (row 0 of each head is the real query), K [H_kv, N, d_k].
    Returns (mask [H_kv, N] bool, budget [H_kv], b_step [H_q], row_sets, probs)."""
    H_q, R1, d_k = Q.shape
    H_kv, N, _ = K.shape
    G = H_q // H_kv
    mask = np.zeros((H_kv, N), dtype=bool)
    b_step = np.zeros(H_q, dtype=np.int64)
    row_sets: Optional[List[List[np.ndarray]]] = [] if keep_rows else None
    probs = np.zeros((H_q, R1, N)) if keep_probs else None
    for g in range(H_q):
        kh = g // G
        L = (Q[g] @ K[kh].T) / math.sqrt(d_k)            # the logits (synthetic rows and A0's row)
        A = softmax_rows(L)
        if keep_probs:
            probs[g] = A
        C0 = top_p_set(A[0], p_nuc)                      # C0 = TopP(A0, p)
        k = int(C0.shape[0])                             # B_step = |C0|
        b_step[g] = k
        sets = [C0]
        for s in range(1, R1):
            if sel_mode == "topk":
                Cs = top_k_set(L[s], k)                  # TopK step
            elif sel_mode == "topp":
                Cs = top_p_set(A[s], p_nuc)              # Section 3.1 rule per synthetic query
            else:
                raise ValueError(sel_mode)
            sets.append(Cs)
            mask[kh, Cs] = True                          # union
        if include_c0:
            mask[kh, C0] = True
        if keep_rows:
            row_sets.append(sets)
    budget = mask.sum(axis=1).astype(np.int64)
    return mask, budget, b_step, row_sets, probs


def attention_overlap(Q: np.ndarray, K: np.ndarray, mask: np.ndarray) -> np.ndarray:
    """Section 3.3's yardstick, applied to the pass's own output: the share of the current query's
    attention (softmax weights of Eq. 1) that falls on the keys the pass keeps, per query head.
    Q [H_q, S+1, d_k] (row 0 of each head is the current query), K [H_kv, N, d_k], mask [H_kv, N]."""
    H_q, _, d_k = Q.shape
    G = H_q // K.shape[0]
    out = np.zeros(H_q)
    for g in range(H_q):
        kh = g // G
        a0 = softmax_rows((Q[g, :1] @ K[kh].T) / math.sqrt(d_k))[0]
        out[g] = a0[mask[kh]].sum()
    return out


def compact(K: np.ndarray, V: np.ndarray, mask: np.ndarray):
    """Algorithm 1, the pruning step: keep the rows of the keep-set, in ascending index order.
    K, V [H_kv, N, d_k] (any dtype; moved, not computed on); returns lists per head."""
    Kc, Vc = [], []
    for kh in range(K.shape[0]):
        idx = np.nonzero(mask[kh])[0]
        Kc.append(K[kh][idx])
        Vc.append(V[kh][idx])
    return Kc, Vc


def pack_varlen(K: np.ndarray, V: np.ndarray, cu_seqlens: np.ndarray, masks: Sequence[np.ndarray]):
    """Section 3.4 of the paper hands the per-head, non-uniform caches to a variable-length
    attention kernel: every (request, KV head) pair becomes one "sequence" of its kept rows.

    K, V [H_kv, T, d_k] (any dtype; moved, not computed on), requests packed along T by
    cu_seqlens; masks[r] [H_kv, N_r] bool.  Returns (K_packed, V_packed, cu_seqlens_k):
    K_packed [total_kept, d_k] holds sequence s = r * H_kv + h at rows
    cu_seqlens_k[s] .. cu_seqlens_k[s+1]-1, kept rows in ascending index order."""
    H_kv, d_k = K.shape[0], K.shape[2]
    parts_k, parts_v, lens = [], [], []
    for r in range(len(cu_seqlens) - 1):
        a, b = int(cu_seqlens[r]), int(cu_seqlens[r + 1])
        for kh in range(H_kv):
            idx = np.nonzero(masks[r][kh])[0]
            parts_k.append(K[kh, a:b][idx])
            parts_v.append(V[kh, a:b][idx])
            lens.append(idx.shape[0])
    cu_k = np.zeros(len(lens) + 1, dtype=np.int64)
    cu_k[1:] = np.cumsum(lens)
    empty = np.zeros((0, d_k), dtype=K.dtype)
    return (np.concatenate(parts_k + [empty], axis=0), np.concatenate(parts_v + [empty.astype(V.dtype)], axis=0), cu_k)


def compress_request(h: np.ndarray, W_q: np.ndarray, b_q: Optional[np.ndarray], K: np.ndarray,
                     *, n_q_heads: int, d_k: int, theta: float, S: int, p_nuc: float, n_f: int,
                     n_s: int, seed: int, layer_id: int, request_id: int,
                     sel_mode: str = "topk", include_c0: bool = False,
                     mirror_rounding: bool = True, h_last: Optional[np.ndarray] = None,
                     keep_rows: bool = False, keep_probs: bool = False) -> RequestResult:
    """Algorithm 1 for one request and one layer, up to the union (pruning is `compact`).

    h [N, d_h] fp64 hidden states; W_q, K already widened to fp64 (exact bf16 values)."""
    N = K.shape[1]
    mu, var = fit(h, n_s)                                               # fit
    H_tilde, _ = sample(mu, var, S, seed, layer_id, request_id)         # sample
    hl = h[-1] if h_last is None else h_last
    Q = queries_for_request(H_tilde, hl, W_q, b_q, N, n_q_heads=n_q_heads, d_k=d_k,
                            theta=theta, n_f=n_f, mirror_rounding=mirror_rounding)  # Q0, Q~
    mask, budget, b_step, rows, probs = vote(Q, K, p_nuc=p_nuc, sel_mode=sel_mode,
                                             include_c0=include_c0, keep_rows=keep_rows,
                                             keep_probs=keep_probs)     # A0, C0, vote
    return RequestResult(mu=mu, var=var, H_tilde=H_tilde, Q=Q, b_step=b_step, mask=mask,
                         budget=budget, row_sets=rows, probs=probs)


@dataclass
class RecompressResult:
    b_step: np.ndarray                 # [H_q] int   k_g = |C0| of query head g over its KV head's keys
    masks: List[np.ndarray]            # per KV head: [len_kh] bool over that head's cache slots
    budget: np.ndarray                 # [H_kv] int
    token_pos: Optional[List[np.ndarray]]   # per KV head: original positions of the slots that stay
    Q: np.ndarray                      # [H_q, S+1, d_k]


def recompress_request(mu: np.ndarray, var: np.ndarray, h_last: np.ndarray, W_q: np.ndarray,
                       b_q: Optional[np.ndarray], K_heads: Sequence[np.ndarray], seq_len: int, *,
                       n_q_heads: int, d_k: int, theta: float, S: int, p_nuc: float, n_f: int,
                       seed: int, layer_id: int, request_id: int, sel_mode: str = "topk",
                       include_c0: bool = False, mirror_rounding: bool = True,
                       token_pos: Optional[Sequence[np.ndarray]] = None) -> RecompressResult:
    """Algorithm 1 applied again to a cache that an earlier pass has already pruned and that has
    grown since (the extension Section 3.4 leaves open: there the pass runs once, after prefill).

    KV head kh now holds K_heads[kh] [len_kh, d_k]: the rows that survived plus the rows appended
    since, each still rotated at the position it was written at, so head lengths differ and a
    slot number no longer is a position.  What Algorithm 1 calls N splits in two: the keys a
    query head sees are the len_kh rows of its own KV head (the current-query steps and the vote run
    per head on those), while the positions of the current query and of AverageCosSin come from seq_len, the number of tokens the
    request has seen: the current query sits at seq_len - 1 and the synthetic queries average
    positions seq_len .. seq_len + n_f - 1.  mu and var are the caller's running fit.
    token_pos[kh] [len_kh] (optional) maps slots to original positions; the result carries the
    map of the slots that stay."""
    H_kv = len(K_heads)
    G = n_q_heads // H_kv
    H_tilde, _ = sample(mu, var, S, seed, layer_id, request_id)                      # sample
    Q = queries_for_request(H_tilde, h_last, W_q, b_q, seq_len, n_q_heads=n_q_heads, d_k=d_k,
                            theta=theta, n_f=n_f, mirror_rounding=mirror_rounding)   # Q0, Q~
    masks: List[np.ndarray] = []
    b_step = np.zeros(n_q_heads, dtype=np.int64)
    budget = np.zeros(H_kv, dtype=np.int64)
    for kh in range(H_kv):
        Kh = np.asarray(K_heads[kh], dtype=np.float64)
        if Kh.shape[0] == 0:
            masks.append(np.zeros(0, dtype=bool))
            continue
        m, b, ks, _, _ = vote(Q[kh * G:(kh + 1) * G], Kh[None], p_nuc=p_nuc, sel_mode=sel_mode,
                              include_c0=include_c0)                                  # A0, C0, vote
        masks.append(m[0])
        budget[kh] = b[0]
        b_step[kh * G:(kh + 1) * G] = ks
    kept_pos = None
    if token_pos is not None:
        kept_pos = [np.asarray(token_pos[kh])[masks[kh]] for kh in range(H_kv)]      # pruning, on the map
    return RecompressResult(b_step=b_step, masks=masks, budget=budget, token_pos=kept_pos, Q=Q)


def compress_layer(h: np.ndarray, W_q_bits: np.ndarray, b_q: Optional[np.ndarray],
                   K_bits: np.ndarray, V_bits: np.ndarray, cu_seqlens: np.ndarray, *,
                   n_q_heads: int, d_k: int, theta: float, S: int, p_nuc: float, n_f: int,
                   n_s: int, seed: int, layer_id: int, sel_mode: str = "topk",
                   include_c0: bool = False, mirror_rounding: bool = True,
                   keep_rows: bool = False, keep_probs: bool = False):
    """The whole pass for a ragged batch of requests packed along the token axis.

    h [T, d_h] fp32; W_q_bits [H_q*d_k, d_h], K_bits/V_bits [H_kv, T, d_k] bf16 bit patterns.
    Returns (results per request, compacted K bits per request per head, same for V)."""
    W = bf16_bits_to_f64(W_q_bits)
    results, Kc_all, Vc_all = [], [], []
    for r in range(len(cu_seqlens) - 1):
        a, b = int(cu_seqlens[r]), int(cu_seqlens[r + 1])
        Kr = bf16_bits_to_f64(K_bits[:, a:b])
        res = compress_request(np.asarray(h[a:b], dtype=np.float64), W, b_q, Kr,
                               n_q_heads=n_q_heads, d_k=d_k, theta=theta, S=S, p_nuc=p_nuc,
                               n_f=n_f, n_s=n_s, seed=seed, layer_id=layer_id, request_id=r,
                               sel_mode=sel_mode, include_c0=include_c0,
                               mirror_rounding=mirror_rounding, keep_rows=keep_rows,
                               keep_probs=keep_probs)
        Kc, Vc = compact(K_bits[:, a:b], V_bits[:, a:b], res.mask)      # pruning
        results.append(res)
        Kc_all.append(Kc)
        Vc_all.append(Vc)
    return results, Kc_all, Vc_all


def pack_mask_bits(mask_row: np.ndarray) -> np.ndarray:
    """Bit n%32 of word n/32 (little-endian within the word), zero padding."""
    N = mask_row.shape[0]
    nw = (N + 31) // 32
    padded = np.zeros(nw * 32, dtype=np.uint8)
    padded[:N] = mask_row.astype(np.uint8)
    return np.packbits(padded.reshape(nw, 32), axis=1, bitorder="little").view(np.uint32).reshape(nw)
