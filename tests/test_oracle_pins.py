"""Pins for the CPU oracle: every step is checked against something other than itself —
published known-answer vectors, closed forms, brute force on tiny inputs, textbook or
library routines, and the invariants the paper states (Section 3.1-3.3, Algorithm 1)."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import gvote_oracle as o

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- Philox / normals
def test_philox_known_answers():
    n = 0
    for line in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        out = o.philox4x32_10(np.array(w[:4], dtype=np.uint32), (w[4], w[5]))
        assert [int(x) for x in out] == w[6:]
        n += 1
    assert n == 3


def test_philox_counter_layout():
    S, d_h, seed, layer, req = 3, 10, 0x123456789ABCDEF, 7, 5
    raw = o.gvote_philox_raw(S, d_h, seed, layer, req)
    assert raw.shape == (S, 12)
    for s in range(S):
        for c in range(12):
            ctr = np.array([c // 4, s, layer, req], dtype=np.uint32)
            ref = o.philox4x32_10(ctr, (seed & 0xFFFFFFFF, seed >> 32))
            assert int(raw[s, c]) == int(ref[c % 4])


def test_philox_streams_nested_in_S():
    a = o.gvote_philox_raw(4, 16, 9, 1, 0)
    b = o.gvote_philox_raw(9, 16, 9, 1, 0)
    assert np.array_equal(a, b[:4])
    assert not np.array_equal(o.gvote_philox_raw(4, 16, 9, 2, 0), a)   # layer word matters
    assert not np.array_equal(o.gvote_philox_raw(4, 16, 9, 1, 1), a)   # request word matters


def test_uniform_is_open_interval_and_exact():
    x = np.array([0, 1, 511, 512, 0xFFFFFFFF], dtype=np.uint32)
    u = o.uniform_open01(x)
    assert u[0] == 2.0 ** -24 and u[2] == 2.0 ** -24 and u[3] == 1.5 * 2.0 ** -23
    assert u[-1] == 1.0 - 2.0 ** -24
    assert np.all(u.astype(np.float32).astype(np.float64) == u)       # exact in fp32


def test_box_muller_moments_and_ks():
    from scipy import stats
    raw = o.gvote_philox_raw(256, 4096, 42, 0, 0)
    z = o.box_muller(raw).ravel()
    n = z.size
    assert abs(z.mean()) < 4.0 / math.sqrt(n)
    assert abs(z.var() - 1.0) < 4.0 * math.sqrt(2.0 / n)
    assert abs(stats.skew(z)) < 4.0 * math.sqrt(6.0 / n)
    assert stats.kstest(z[:200000], "norm").pvalue > 1e-3
    # the cos and sin branches are uncorrelated
    assert abs(np.corrcoef(z[0::2], z[1::2])[0, 1]) < 4.0 / math.sqrt(n / 2)


def test_box_muller_single_value_by_hand():
    raw = np.array([[0x80000000, 0x40000000, 0x00000000, 0xC0000000]], dtype=np.uint32)
    z = o.box_muller(raw)[0]
    u0, u1 = (2 ** 22 + 0.5) / 2 ** 23, (2 ** 21 + 0.5) / 2 ** 23
    assert z[0] == pytest.approx(math.sqrt(-2 * math.log(u0)) * math.cos(2 * math.pi * u1), rel=1e-14)
    assert z[1] == pytest.approx(math.sqrt(-2 * math.log(u0)) * math.sin(2 * math.pi * u1), rel=1e-14)
    u2, u3 = 0.5 / 2 ** 23, (3 * 2 ** 21 + 0.5) / 2 ** 23
    assert z[3] == pytest.approx(math.sqrt(-2 * math.log(u2)) * math.sin(2 * math.pi * u3), rel=1e-12)


def test_sample_converges_to_fitted_gaussian():
    rng = np.random.default_rng(0)
    d_h = 32
    mu = rng.normal(size=d_h)
    var = rng.uniform(0.1, 10.0, size=d_h)
    S = 40000
    H, _ = o.sample(mu, var, S, seed=3, layer_id=0, request_id=0)
    se = np.sqrt(var / S)
    assert np.all(np.abs(H.mean(axis=0) - mu) < 5 * se)
    assert np.all(np.abs(H.var(axis=0) / var - 1.0) < 5 * math.sqrt(2.0 / S))
    C = np.corrcoef(H.T)
    off = C - np.diag(np.diag(C))
    assert np.abs(off).max() < 5.5 / math.sqrt(S)                      # diagonal covariance


# ----------------------------------------------------------------------------- fit
def test_fit_alternating_closed_form():
    T, n_s = 104, 4
    a = np.array([0.5, -2.0, 3.0])
    b = np.array([1.0, 0.25, 7.0])
    t = np.arange(T)[:, None]
    h = a + b * (-1.0) ** t
    h[:n_s] = 1e6                                # sink rows must be ignored
    mu, var = o.fit(h, n_s)
    n = T - n_s
    assert np.allclose(mu, a, atol=1e-12)
    assert np.allclose(var, b * b * n / (n - 1), rtol=1e-12)


def test_fit_ramp_closed_form_and_library():
    T = 50
    h = np.arange(T, dtype=np.float64)[:, None] * np.array([1.0, 2.0]) + np.array([3.0, -1.0])
    mu, var = o.fit(h, 0)
    assert np.allclose(mu, [(T - 1) / 2 + 3.0, (T - 1) - 1.0])
    assert np.allclose(var, [T * (T + 1) / 12.0, 4 * T * (T + 1) / 12.0])
    rng = np.random.default_rng(1)
    h = rng.normal(size=(200, 7)) * 3 + 1
    mu, var = o.fit(h, 4)
    assert np.allclose(mu, np.mean(h[4:], axis=0)) and np.allclose(var, np.var(h[4:], axis=0, ddof=1))
    with pytest.raises(ValueError):
        o.fit(h[:5], 4)


# ----------------------------------------------------------------------------- RoPE
def test_average_cos_sin_closed_form():
    for (N, n_f, d_k, theta) in [(512, 128, 64, 1e4), (4096, 128, 128, 5e5), (131072, 37, 128, 1e6)]:
        cbar, sbar = o.average_cos_sin(N, n_f, d_k, theta)
        w = theta ** (-2.0 * np.arange(d_k // 2) / d_k)
        # sum_{i<n} cos(a + i w) = sin(n w/2)/sin(w/2) * cos(a + (n-1) w/2)
        ratio = np.sin(n_f * w / 2) / np.sin(w / 2) / n_f
        assert np.allclose(cbar, ratio * np.cos(N * w + (n_f - 1) * w / 2), atol=1e-12)
        assert np.allclose(sbar, ratio * np.sin(N * w + (n_f - 1) * w / 2), atol=1e-12)
        assert np.all(cbar ** 2 + sbar ** 2 <= 1.0 + 1e-12)            # a shrunk rotation


def test_average_cos_sin_one_position_is_plain_rope():
    cbar, sbar = o.average_cos_sin(77, 1, 32, 1e4)
    w = 1e4 ** (-2.0 * np.arange(16) / 32)
    assert np.allclose(cbar, np.cos(77 * w)) and np.allclose(sbar, np.sin(77 * w))


def test_rope_is_complex_rotation_of_half_pairs():
    rng = np.random.default_rng(2)
    d_k, pos, theta = 16, 13, 1e4
    x = rng.normal(size=(3, d_k))
    w = o.rope_frequencies(d_k, theta)
    y = o.rope_apply(x, np.cos(pos * w), np.sin(pos * w))
    z = (x[:, :8] + 1j * x[:, 8:]) * np.exp(1j * pos * w)
    assert np.allclose(y[:, :8], z.real) and np.allclose(y[:, 8:], z.imag)
    assert np.allclose(np.linalg.norm(y, axis=1), np.linalg.norm(x, axis=1))
    assert w[0] == 1.0 and w[-1] == pytest.approx(theta ** (-14.0 / 16))


def test_rope_scores_depend_on_relative_position():
    rng = np.random.default_rng(3)
    d_k, theta = 32, 1e4
    q, k = rng.normal(size=d_k), rng.normal(size=d_k)
    w = o.rope_frequencies(d_k, theta)
    def rot(v, p):
        return o.rope_apply(v, np.cos(p * w), np.sin(p * w))
    assert np.dot(rot(q, 40), rot(k, 33)) == pytest.approx(np.dot(rot(q, 107), rot(k, 100)), rel=1e-10)


def test_averaged_rope_equals_average_of_rotated_queries():
    """Linearity: rotating once with the mean cos/sin equals the mean of the n_f rotations."""
    rng = np.random.default_rng(4)
    d_k, theta, N, n_f = 16, 1e4, 21, 5
    x = rng.normal(size=d_k)
    w = o.rope_frequencies(d_k, theta)
    cbar, sbar = o.average_cos_sin(N, n_f, d_k, theta)
    acc = sum(o.rope_apply(x, np.cos((N + i) * w), np.sin((N + i) * w)) for i in range(n_f)) / n_f
    assert np.allclose(o.rope_apply(x, cbar, sbar), acc)


# ----------------------------------------------------------------------------- projection, softmax
def test_projection_layout_by_loops():
    rng = np.random.default_rng(5)
    rows, d_h, H, d_k = 3, 6, 2, 4
    X, W, b = rng.normal(size=(rows, d_h)), rng.normal(size=(H * d_k, d_h)), rng.normal(size=H * d_k)
    q = o.project_queries(X, W, b, H, d_k)
    for g in range(H):
        for r in range(rows):
            for j in range(d_k):
                ref = sum(X[r, c] * W[g * d_k + j, c] for c in range(d_h)) + b[g * d_k + j]
                assert q[g, r, j] == pytest.approx(ref, rel=1e-12)


def test_softmax_matches_library_and_sums_to_one():
    from scipy.special import softmax
    rng = np.random.default_rng(6)
    L = rng.normal(size=(5, 33)) * 10
    A = o.softmax_rows(L)
    assert np.allclose(A, softmax(L, axis=-1), rtol=1e-12)
    assert np.allclose(A.sum(axis=1), 1.0)
    assert np.allclose(o.softmax_rows(L + 1000.0), A)                  # shift invariance


def test_queries_row0_exact_rope_rows_averaged():
    rng = np.random.default_rng(7)
    d_h, H, d_k, S, N, n_f, theta = 12, 2, 8, 3, 30, 4, 1e4
    Ht, hl = rng.normal(size=(S, d_h)), rng.normal(size=d_h)
    W = rng.normal(size=(H * d_k, d_h))
    Q = o.queries_for_request(Ht, hl, W, None, N, n_q_heads=H, d_k=d_k, theta=theta, n_f=n_f,
                              mirror_rounding=False)
    w = o.rope_frequencies(d_k, theta)
    for g in range(H):
        q0 = W[g * d_k:(g + 1) * d_k] @ hl
        z = (q0[:4] + 1j * q0[4:]) * np.exp(1j * (N - 1) * w)
        assert np.allclose(Q[g, 0], np.concatenate([z.real, z.imag]))
        for s in range(S):
            qs = W[g * d_k:(g + 1) * d_k] @ Ht[s]
            z = (qs[:4] + 1j * qs[4:]) * np.mean([np.exp(1j * (N + i) * w) for i in range(n_f)], axis=0)
            assert np.allclose(Q[g, 1 + s], np.concatenate([z.real, z.imag]))


def test_round_to_bf16_matches_torch():
    import torch
    rng = np.random.default_rng(8)
    x = np.concatenate([rng.normal(size=5000) * 10.0 ** rng.integers(-6, 6, size=5000),
                        [0.0, 1.0, -1.0, 1.00390625, 1.01171875, 3.0e-39, 65280.0]])
    ref = torch.tensor(x, dtype=torch.float64).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(o.round_to_bf16(x), ref)


def _torch_bf16(x):
    """bf16 rounding by a routine other than the oracle's (torch's conversion), result in fp64."""
    import torch
    return torch.tensor(np.asarray(x), dtype=torch.float64).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()


def test_mirrored_roundings_sit_before_the_product_and_after_the_rotation():
    """Where `mirror_rounding=True` rounds: the projection's input rows X = [h_last; H~] before the
    product, the rotated queries after RoPE, and nowhere else.  Each claim is checked against a
    statement that a rounding put elsewhere fails."""
    rng = np.random.default_rng(21)
    d_h, H, d_k, S, N, n_f, theta = 40, 3, 8, 5, 77, 6, 1e4
    Ht, hl = rng.normal(size=(S, d_h)) * 3, rng.normal(size=d_h)
    W = _torch_bf16(rng.normal(size=(H * d_k, d_h)) / math.sqrt(d_h))
    b = rng.normal(size=H * d_k) * 0.1
    kw = dict(n_q_heads=H, d_k=d_k, theta=theta, n_f=n_f)
    Qm = o.queries_for_request(Ht, hl, W, b, N, mirror_rounding=True, **kw)
    # (a) the last step is a rounding: every entry lies on the bf16 grid
    assert np.array_equal(Qm, _torch_bf16(Qm))
    # (b) exactly one rounding lies between the product of the rounded rows and the result: the error
    # against the unrounded rotation of those rows is at most half a bf16 step of the result's binade
    Xr = _torch_bf16(np.concatenate([hl[None], Ht]))
    Qx = o.queries_for_request(Xr[1:], Xr[0], W, b, N, mirror_rounding=False, **kw)
    half_step = 2.0 ** (np.floor(np.log2(np.abs(Qx))) - 8)
    assert np.all(np.abs(Qm - Qx) <= half_step)
    assert np.array_equal(Qm, _torch_bf16(Qx))
    # a second rounding between the product and the rotation (the planted mistake) breaks (b) somewhere
    w = o.rope_frequencies(d_k, theta)
    q_pre = _torch_bf16(o.project_queries(Xr, W, b, H, d_k))
    c0, s0 = np.cos((N - 1) * w), np.sin((N - 1) * w)
    cb, sb = o.average_cos_sin(N, n_f, d_k, theta)
    wrong = np.empty_like(q_pre)
    wrong[:, 0] = o.rope_apply(q_pre[:, 0], c0, s0)
    wrong[:, 1:] = o.rope_apply(q_pre[:, 1:], cb, sb)
    assert np.any(np.abs(_torch_bf16(wrong) - Qx) > half_step)
    # (c) against the unrounded pass the two roundings together stay within what two roundings allow:
    # the input rounding moves a row by at most 2^-9 relative per entry, i.e. the product by at most
    # 2^-9 * sum |x_c W_fc|, the rotation mixes two features with |cos|, |sin| <= 1, and the final
    # rounding adds half a step of the result
    Qi = o.queries_for_request(Ht, hl, W, b, N, mirror_rounding=False, **kw)
    X = np.concatenate([hl[None], Ht])
    prod = (np.abs(X) @ np.abs(W).T).reshape(S + 1, H, d_k).transpose(1, 0, 2) * 2.0 ** -9
    mix = prod + np.concatenate([prod[..., d_k // 2:], prod[..., :d_k // 2]], axis=-1)
    assert np.all(np.abs(Qm - Qi) <= mix + 2.0 ** -8 * np.abs(Qi) + 1e-12)
    assert np.any(Qm != _torch_bf16(Qi))                       # and the input rounding is not a no-op


def test_input_rows_are_rounded_before_the_product_not_after():
    """A hand case where the place of the first rounding changes the bits.  One head, no rotation
    (N = 1 puts the current query at position 0, where RoPE is the identity), a weight row that adds
    two channels: x = (1 + 2^-8, 2^-8).  Rounded first, 1 + 2^-8 is a tie that goes to the even
    neighbour 1, the sum is 1 + 2^-8 and the final rounding gives 1 again.  Summed first, the result
    is 1 + 2^-7, which bf16 holds exactly."""
    d_k = 2
    W = np.zeros((d_k, 2))
    W[0] = [1.0, 1.0]
    hl = np.array([1.0 + 2.0 ** -8, 2.0 ** -8])
    Ht = np.zeros((1, 2))
    Q = o.queries_for_request(Ht, hl, W, None, 1, n_q_heads=1, d_k=d_k, theta=1e4, n_f=1, mirror_rounding=True)
    assert Q[0, 0, 0] == 1.0
    Qi = o.queries_for_request(Ht, hl, W, None, 1, n_q_heads=1, d_k=d_k, theta=1e4, n_f=1, mirror_rounding=False)
    assert Qi[0, 0, 0] == 1.0 + 2.0 ** -7 and _torch_bf16(Qi)[0, 0, 0] == 1.0 + 2.0 ** -7


def test_bf16_bits_widen_exactly():
    import torch
    bits = np.arange(0, 65536, 7, dtype=np.uint16)
    bits = bits[(bits & 0x7F80) != 0x7F80]                             # skip inf/nan
    ref = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(o.bf16_bits_to_f64(bits), ref)


# ----------------------------------------------------------------------------- top-p / top-k
def _brute_min_subset_size(a, p):
    """Smallest subset size whose mass reaches p, over all 2^N subsets."""
    N = a.shape[0]
    bits = ((np.arange(1 << N)[:, None] >> np.arange(N)[None, :]) & 1).astype(np.float64)
    mass = bits @ a
    size = bits.sum(axis=1)
    ok = mass >= p
    return int(size[ok].min()) if ok.any() else N


@pytest.mark.parametrize("N", [1, 2, 5, 9, 12, 16])
def test_top_p_is_minimal_by_brute_force(N):
    rng = np.random.default_rng(100 + N)
    for trial in range(6 if N < 16 else 2):
        a = o.softmax_rows(rng.normal(size=(1, N)) * rng.uniform(0.5, 4.0))[0]
        for p in (0.3, 0.5, 0.9, 0.95):
            C = o.top_p_set(a, p)
            assert a[C].sum() >= p or len(C) == N
            assert len(C) == _brute_min_subset_size(a, p)
            if len(C) > 1:                                             # dropping the weakest loses p
                assert a[C[:-1]].sum() < p
            assert len(set(C.tolist())) == len(C)


def test_top_p_special_cases():
    a = np.array([0.01, 0.96, 0.01, 0.02])
    assert o.top_p_set(a, 0.95).tolist() == [1]                        # one dominant key -> size 1
    u = np.full(8, 0.125)                                              # exact binary weights
    assert o.top_p_set(u, 0.5).tolist() == [0, 1, 2, 3]                # ties -> lower index, ceil(pN)
    assert o.top_p_set(u, 0.5625).tolist() == [0, 1, 2, 3, 4]
    assert len(o.top_p_set(u, 1.0)) == 8
    assert o.top_p_set(np.array([0.25, 0.5, 0.25]), 0.75).tolist() == [1, 0]   # crossing key kept
    assert len(o.top_p_set(np.array([1.0]), 0.95)) == 1


@pytest.mark.parametrize("N", [1, 3, 8, 12])
def test_top_k_by_brute_force(N):
    rng = np.random.default_rng(200 + N)
    l = rng.normal(size=N)
    for k in range(0, N + 2):
        C = o.top_k_set(l, k)
        kk = min(k, N)
        assert len(C) == kk
        best = max((sum(l[list(c)]) for c in itertools.combinations(range(N), kk)), default=0.0)
        assert l[C].sum() == pytest.approx(best)
    assert o.top_k_set(l, 1).tolist() == [int(np.argmax(l))]
    assert sorted(o.top_k_set(l, N).tolist()) == list(range(N))


def test_top_k_ties_lower_index_first():
    l = np.array([1.0, 3.0, 3.0, 0.0, 3.0])
    assert o.top_k_set(l, 2).tolist() == [1, 2]
    assert o.top_k_set(np.zeros(6), 3).tolist() == [0, 1, 2]


# ----------------------------------------------------------------------------- vote / union
def _small_problem(seed, H_q=4, H_kv=2, d_k=8, S=5, N=14):
    rng = np.random.default_rng(seed)
    Q = rng.normal(size=(H_q, S + 1, d_k)) * 2.0
    K = rng.normal(size=(H_kv, N, d_k))
    return Q, K


@pytest.mark.parametrize("mode", ["topk", "topp"])
def test_vote_union_contains_every_voter_and_counts(mode):
    Q, K = _small_problem(11)
    mask, budget, b_step, rows, probs = o.vote(Q, K, p_nuc=0.8, sel_mode=mode, keep_rows=True,
                                               keep_probs=True)
    H_q, H_kv, G = Q.shape[0], K.shape[0], Q.shape[0] // K.shape[0]
    N = K.shape[1]
    for g in range(H_q):
        kh = g // G
        assert b_step[g] == len(rows[g][0])
        for s in range(1, Q.shape[1]):
            assert mask[kh, rows[g][s]].all()                          # union contains C^(s)
            assert budget[kh] >= len(rows[g][s])                       # |union| >= |C^(s)| (Sec. 3.3)
            if mode == "topk":
                assert len(rows[g][s]) == min(b_step[g], N)
            else:
                assert probs[g, s, rows[g][s]].sum() >= 0.8 - 1e-12    # kept mass >= p
    for kh in range(H_kv):
        union = set()
        for g in range(kh * G, (kh + 1) * G):
            for s in range(1, Q.shape[1]):
                union |= set(rows[g][s].tolist())
        assert set(np.nonzero(mask[kh])[0].tolist()) == union          # nothing but the votes
        assert budget[kh] == len(union)
        if mode == "topk":
            ks = b_step[kh * G:(kh + 1) * G]
            assert ks.max() <= budget[kh] <= min(N, (Q.shape[1] - 1) * ks.sum())


def test_vote_by_brute_force_tiny():
    """The current-query steps (A0, C0, B_step) and the vote (logits, TopK, union) of Algorithm 1 re-derived
    with exhaustive subset search on N=10."""
    Q, K = _small_problem(12, H_q=2, H_kv=1, d_k=4, S=3, N=10)
    p = 0.7
    mask, budget, b_step, _, _ = o.vote(Q, K, p_nuc=p)
    N = K.shape[1]
    expect = np.zeros(N, dtype=bool)
    for g in range(2):
        L = np.array([[sum(Q[g, r, j] * K[0, n, j] for j in range(4)) / 2.0 for n in range(N)]
                      for r in range(Q.shape[1])])
        e = np.exp(L[0] - L[0].max())
        a0 = e / e.sum()
        k = _brute_min_subset_size(a0, p)
        assert b_step[g] == k
        for s in range(1, Q.shape[1]):
            best = max(itertools.combinations(range(N), k), key=lambda c: sum(L[s, list(c)]))
            expect[list(best)] = True
    assert np.array_equal(mask[0], expect) and budget[0] == expect.sum()


def test_vote_include_c0_flag():
    Q, K = _small_problem(13)
    m0, _, _, rows, _ = o.vote(Q, K, p_nuc=0.9, keep_rows=True)
    m1, b1, _, _, _ = o.vote(Q, K, p_nuc=0.9, include_c0=True)
    G = Q.shape[0] // K.shape[0]
    for kh in range(K.shape[0]):
        want = m0[kh].copy()
        for g in range(kh * G, (kh + 1) * G):
            want[rows[g][0]] = True
        assert np.array_equal(m1[kh], want)


def test_vote_S1_single_head_is_single_query_selection():
    Q, K = _small_problem(14, H_q=1, H_kv=1, S=1, N=16)
    mask, budget, b_step, _, probs = o.vote(Q, K, p_nuc=0.9, keep_probs=True)
    assert budget[0] == b_step[0]
    L = Q[0, 1] @ K[0].T
    assert set(np.nonzero(mask[0])[0].tolist()) == set(np.argsort(-L, kind="stable")[:b_step[0]].tolist())
    m2, b2, _, _, pr = o.vote(Q, K, p_nuc=0.9, sel_mode="topp", keep_probs=True)
    assert set(np.nonzero(m2[0])[0].tolist()) == set(o.top_p_set(pr[0, 1], 0.9).tolist())


def test_vote_dominant_key():
    """One key far ahead of all others: |C0| = 1, so every top-k voter picks one key and the
    budget is at most S*G; in top-p mode a voter whose own mass sits on one key picks it alone."""
    rng = np.random.default_rng(15)
    d_k, N, S = 8, 20, 4
    K = rng.normal(size=(1, N, d_k)) * 0.05
    K[0, 7] = 0.0
    K[0, 7, 0] = 50.0
    Q = np.abs(rng.normal(size=(2, S + 1, d_k))) + 1.0                 # positive along key 7
    mask, budget, b_step, _, _ = o.vote(Q, K, p_nuc=0.95)
    assert b_step.tolist() == [1, 1] and budget[0] == 1 and mask[0, 7]
    mask, budget, _, _, _ = o.vote(Q, K, p_nuc=0.95, sel_mode="topp")
    assert budget[0] == 1 and mask[0, 7]


def test_budget_monotone_in_S_and_p():
    from paper_2509_03136_b200 import synth
    cfg = synth.make_small(21, seq_lens=(96,), S=8, p_nuc=0.9)
    li = synth.make_layer(cfg, 0)
    kw = dict(n_q_heads=cfg.n_q_heads, d_k=cfg.d_k, theta=cfg.rope_theta, n_f=cfg.n_f, n_s=cfg.n_s,
              seed=5, layer_id=0)
    def run(S, p, mode):
        res, _, _ = o.compress_layer(li.h, li.W_q, None, li.K, li.V, li.cu_seqlens, S=S, p_nuc=p,
                                     sel_mode=mode, **kw)
        return res[0]
    for mode in ("topk", "topp"):
        small, big = run(3, 0.9, mode), run(8, 0.9, mode)
        assert np.all(big.mask | ~small.mask)                          # nested samples -> nested masks
        lo, hi = run(8, 0.6, mode), run(8, 0.95, mode)
        assert np.all(hi.b_step >= lo.b_step)
        assert np.all(hi.budget >= lo.budget)


# ----------------------------------------------------------------------------- compaction, packing
def test_compact_cases():
    rng = np.random.default_rng(16)
    K = rng.integers(0, 65535, size=(2, 9, 4)).astype(np.uint16)
    V = rng.integers(0, 65535, size=(2, 9, 4)).astype(np.uint16)
    mask = np.zeros((2, 9), dtype=bool)
    mask[0, [1, 4, 8]] = True
    Kc, Vc = o.compact(K, V, mask)
    assert np.array_equal(Kc[0], np.stack([K[0, 1], K[0, 4], K[0, 8]]))
    assert np.array_equal(Vc[0], np.stack([V[0, 1], V[0, 4], V[0, 8]]))
    assert Kc[1].shape == (0, 4)                                       # empty keep-set
    Kc, _ = o.compact(K, V, np.ones((2, 9), dtype=bool))
    assert np.array_equal(Kc[1], K[1])                                 # identity when all kept


def test_pack_mask_bits_layout():
    m = np.zeros(70, dtype=bool)
    m[[0, 31, 32, 69]] = True
    w = o.pack_mask_bits(m)
    assert w.dtype == np.uint32 and w.tolist() == [(1 << 31) | 1, 1, 1 << 5]


# ----------------------------------------------------------------------------- whole pass
def test_compress_layer_ragged_requests_are_independent():
    from paper_2509_03136_b200 import synth
    cfg = synth.make_small(22, seq_lens=(33, 64, 17), S=4)
    li = synth.make_layer(cfg, 0)
    kw = dict(n_q_heads=cfg.n_q_heads, d_k=cfg.d_k, theta=cfg.rope_theta, S=cfg.S, p_nuc=cfg.p_nuc,
              n_f=cfg.n_f, n_s=cfg.n_s, seed=1, layer_id=3)
    res, Kc, Vc = o.compress_layer(li.h, li.W_q, None, li.K, li.V, li.cu_seqlens, **kw)
    cu = li.cu_seqlens
    for r in range(3):
        a, b = int(cu[r]), int(cu[r + 1])
        W = o.bf16_bits_to_f64(li.W_q)
        alone = o.compress_request(li.h[a:b].astype(np.float64), W, None,
                                   o.bf16_bits_to_f64(li.K[:, a:b]), request_id=r,
                                   **{k: v for k, v in kw.items()})
        assert np.array_equal(alone.mask, res[r].mask)
        for kh in range(cfg.n_kv_heads):
            assert Kc[r][kh].shape[0] == res[r].budget[kh]
            assert np.array_equal(Kc[r][kh], li.K[kh, a:b][res[r].mask[kh]])
            assert np.array_equal(Vc[r][kh], li.V[kh, a:b][res[r].mask[kh]])


# ----------------------------------------------------------------------------- varlen packing
def test_pack_varlen_hand_example():
    # two requests (3 and 2 tokens), two heads, d_k = 1: rows are labelled head * 100 + token
    K = np.array([[[0], [1], [2], [3], [4]], [[100], [101], [102], [103], [104]]], dtype=np.int32)
    V = K + 1000
    cu = np.array([0, 3, 5])
    masks = [np.array([[1, 0, 1], [0, 0, 0]], bool), np.array([[0, 1], [1, 1]], bool)]
    Kp, Vp, cu_k = o.pack_varlen(K, V, cu, masks)
    assert Kp[:, 0].tolist() == [0, 2, 4, 103, 104]          # (r0,h0) (r0,h1: none) (r1,h0) (r1,h1)
    assert Vp[:, 0].tolist() == [1000, 1002, 1004, 1103, 1104]
    assert cu_k.tolist() == [0, 2, 2, 3, 5]


def test_pack_varlen_slices_are_the_compacted_heads_and_identity():
    rng = np.random.default_rng(21)
    H, d = 3, 4
    lens = [7, 1, 12]
    cu = np.concatenate([[0], np.cumsum(lens)])
    K = rng.integers(0, 1000, size=(H, cu[-1], d))
    V = rng.integers(0, 1000, size=(H, cu[-1], d))
    masks = [rng.random((H, n)) < 0.5 for n in lens]
    Kp, Vp, cu_k = o.pack_varlen(K, V, cu, masks)
    assert cu_k[-1] == sum(int(m.sum()) for m in masks) == Kp.shape[0] == Vp.shape[0]
    for r, n in enumerate(lens):
        Kc, Vc = o.compact(K[:, cu[r]:cu[r + 1]], V[:, cu[r]:cu[r + 1]], masks[r])
        for h in range(H):
            s = r * H + h
            assert np.array_equal(Kp[cu_k[s]:cu_k[s + 1]], Kc[h]) and np.array_equal(Vp[cu_k[s]:cu_k[s + 1]], Vc[h])
    # keeping everything just re-orders the cache request-major, head-minor
    full = [np.ones((H, n), bool) for n in lens]
    Kf, _, cu_f = o.pack_varlen(K, V, cu, full)
    assert np.array_equal(Kf, np.concatenate([K[h, cu[r]:cu[r + 1]] for r in range(3) for h in range(H)]))
    assert np.array_equal(np.diff(cu_f), np.repeat(lens, H))
    # keeping nothing gives empty buffers
    Ke, Ve, cu_e = o.pack_varlen(K, V, cu, [np.zeros((H, n), bool) for n in lens])
    assert Ke.shape == (0, d) and cu_e.tolist() == [0] * (3 * H + 1)


# ----------------------------------------------------------------------------- streaming fit
def test_fit_merge_equals_fit_of_the_concatenation():
    rng = np.random.default_rng(41)
    h = rng.normal(size=(97, 6)) * rng.uniform(0.1, 5, size=6) + rng.normal(size=6) * 20
    n_s = 4
    cuts = [n_s, 10, 11, 50, 97]                                  # uneven blocks, one of a single row
    st = o.fit_state(h[0:0])
    for a, b in zip(cuts[:-1], cuts[1:]):
        st = o.fit_merge(st, o.fit_state(h[a:b]))
    mu, var = o.fit_finish(st)
    assert st.n == 97 - n_s
    assert np.allclose(mu, h[n_s:].mean(axis=0), rtol=1e-13) and np.allclose(var, h[n_s:].var(axis=0, ddof=1), rtol=1e-12)
    mu2, var2 = o.fit(h, n_s)                                     # the one-shot fit of Step 2
    assert np.allclose(mu, mu2, rtol=1e-13) and np.allclose(var, var2, rtol=1e-12)


def test_fit_merge_is_symmetric_and_has_an_identity():
    rng = np.random.default_rng(42)
    A, B = rng.normal(size=(5, 3)), rng.normal(size=(9, 3)) + 3
    ab, ba = o.fit_merge(o.fit_state(A), o.fit_state(B)), o.fit_merge(o.fit_state(B), o.fit_state(A))
    assert ab.n == ba.n == 14 and np.allclose(ab.mean, ba.mean, rtol=1e-14) and np.allclose(ab.m2, ba.m2, rtol=1e-13)
    e = o.fit_state(A[0:0])
    same = o.fit_merge(e, o.fit_state(A))
    assert same.n == 5 and np.array_equal(same.mean, o.fit_state(A).mean) and np.array_equal(same.m2, o.fit_state(A).m2)
    # two blocks of one row each: variance of two points is (x - y)^2 / 2
    two = o.fit_merge(o.fit_state(A[:1]), o.fit_state(A[1:2]))
    assert np.allclose(o.fit_finish(two)[1], (A[0] - A[1]) ** 2 / 2, rtol=1e-13)
    with pytest.raises(ValueError):
        o.fit_finish(o.fit_state(A[:1]))


# ----------------------------------------------------------------------------- attention overlap
def test_attention_overlap_special_cases():
    rng = np.random.default_rng(51)
    H_q, H_kv, S1, d_k, N = 4, 2, 3, 8, 50
    Q = rng.normal(size=(H_q, S1, d_k)) * 2
    K = rng.normal(size=(H_kv, N, d_k))
    ones, none = np.ones((H_kv, N), bool), np.zeros((H_kv, N), bool)
    assert np.allclose(o.attention_overlap(Q, K, ones), 1.0, rtol=1e-14) and np.all(o.attention_overlap(Q, K, none) == 0)
    m = rng.random((H_kv, N)) < 0.4
    assert np.allclose(o.attention_overlap(Q, K, m) + o.attention_overlap(Q, K, ~m), 1.0, rtol=1e-13)   # additivity
    # keeping exactly the top-p set of the current query keeps at least p of its attention, and
    # dropping that set's last key falls below p (minimality)
    for g in range(H_q):
        kh = g // 2
        a0 = o.softmax_rows((Q[g, :1] @ K[kh].T) / math.sqrt(d_k))[0]
        C0 = o.top_p_set(a0, 0.9)
        mk = none.copy(); mk[kh, C0] = True
        assert o.attention_overlap(Q, K, mk)[g] >= 0.9
        mk[kh, C0[-1]] = False
        assert o.attention_overlap(Q, K, mk)[g] < 0.9
    # by hand: two keys with logits 0 and ln 3 -> weights 1/4 and 3/4
    Q1 = np.zeros((1, 1, 4)); Q1[0, 0, 0] = 2.0
    K1 = np.zeros((1, 2, 4)); K1[0, 1, 0] = math.log(3.0)         # logit = 2 * ln3 / sqrt(4) = ln 3
    assert o.attention_overlap(Q1, K1, np.array([[False, True]]))[0] == pytest.approx(0.75, rel=1e-14)


# ----------------------------------------------------------------------------- the pass applied again
def _recompress_problem(seed, H_q=4, H_kv=2, d_k=16, d_h=24, N0=30):
    rng = np.random.default_rng(seed)
    W = rng.normal(size=(H_q * d_k, d_h)) / math.sqrt(d_h)
    mu, var = rng.normal(size=d_h), rng.uniform(0.5, 2.0, size=d_h)
    h_last = rng.normal(size=d_h)
    k0 = rng.normal(size=(H_kv, N0, d_k))                  # keys before rotation, one per position
    return W, mu, var, h_last, k0


def _keys_at(k0_head, pos, d_k, theta, shift=0):
    """Rows `pos` of the unrotated keys, rotated at positions pos + shift."""
    w = o.rope_frequencies(d_k, theta)
    at = (np.asarray(pos, dtype=np.float64) + shift)[:, None]
    return o.rope_apply(k0_head[np.asarray(pos, dtype=int)], np.cos(at * w), np.sin(at * w))


def test_recompress_of_an_unpruned_cache_is_the_pass_itself():
    rng = np.random.default_rng(40)
    H_q, H_kv, d_k, d_h, N, S, n_s = 4, 2, 8, 12, 26, 5, 2
    h = rng.normal(size=(N, d_h))
    W = rng.normal(size=(H_q * d_k, d_h)) / math.sqrt(d_h)
    K = rng.normal(size=(H_kv, N, d_k))
    kw = dict(n_q_heads=H_q, d_k=d_k, theta=1e4, S=S, p_nuc=0.8, n_f=4, seed=9, layer_id=3, request_id=1)
    first = o.compress_request(h, W, None, K, n_s=n_s, **kw)
    mu, var = o.fit(h, n_s)
    again = o.recompress_request(mu, var, h[-1], W, None, [K[0], K[1]], N, **kw)
    for kh in range(H_kv):
        assert np.array_equal(again.masks[kh], first.mask[kh])
    assert np.array_equal(again.budget, first.budget) and np.array_equal(again.b_step, first.b_step)


def test_recompress_positions_come_from_tokens_seen_not_rows_stored():
    """RoPE scores depend on relative position only, so moving every stored key and the count of
    tokens seen by the same offset changes nothing; a query placed by the number of rows stored
    would not move with them."""
    d_k, theta, N0 = 16, 1e4, 30
    W, mu, var, h_last, k0 = _recompress_problem(41, d_k=d_k, N0=N0)
    rng = np.random.default_rng(42)
    pos = [np.sort(rng.choice(N0, size=n, replace=False)) for n in (17, 9)]
    kw = dict(n_q_heads=4, d_k=d_k, theta=theta, S=3, p_nuc=0.5, n_f=4, seed=5, layer_id=0, request_id=0,
              mirror_rounding=False)
    base = o.recompress_request(mu, var, h_last, W, None, [_keys_at(k0[kh], pos[kh], d_k, theta) for kh in range(2)],
                                N0, **kw)
    for shift in (1, 57):
        moved = o.recompress_request(mu, var, h_last, W, None,
                                     [_keys_at(k0[kh], pos[kh], d_k, theta, shift) for kh in range(2)],
                                     N0 + shift, **kw)
        for kh in range(2):
            assert np.array_equal(moved.masks[kh], base.masks[kh])
        assert np.array_equal(moved.b_step, base.b_step)
    # the control: keys moved, count of tokens seen left alone -> different logits, different queries
    stale = o.recompress_request(mu, var, h_last, W, None,
                                 [_keys_at(k0[kh], pos[kh], d_k, theta, 57) for kh in range(2)], N0, **kw)
    assert np.array_equal(stale.Q, base.Q)
    assert (not np.array_equal(stale.b_step, base.b_step)
            or any(not np.array_equal(stale.masks[kh], base.masks[kh]) for kh in range(2)))


def test_recompress_by_brute_force_each_head_over_its_own_rows():
    d_k, theta = 4, 1e4
    W, mu, var, h_last, k0 = _recompress_problem(43, H_q=2, H_kv=2, d_k=d_k, d_h=6, N0=12)
    pos = [np.array([0, 2, 3, 5, 8, 9, 11]), np.array([1, 4, 6, 10])]
    K_heads = [_keys_at(k0[kh], pos[kh], d_k, theta) for kh in range(2)]
    p = 0.7
    res = o.recompress_request(mu, var, h_last, W, None, K_heads, 12, n_q_heads=2, d_k=d_k, theta=theta, S=3,
                               p_nuc=p, n_f=2, seed=1, layer_id=0, request_id=0, token_pos=pos)
    for kh in range(2):
        n = K_heads[kh].shape[0]
        assert res.masks[kh].shape == (n,)
        L = np.array([[sum(res.Q[kh, r, j] * K_heads[kh][i, j] for j in range(d_k)) / 2.0 for i in range(n)]
                      for r in range(4)])
        e = np.exp(L[0] - L[0].max())
        k = _brute_min_subset_size(e / e.sum(), p)
        assert res.b_step[kh] == k
        expect = np.zeros(n, dtype=bool)
        for s in range(1, 4):
            best = max(itertools.combinations(range(n), k), key=lambda c: sum(L[s, list(c)]))
            expect[list(best)] = True
        assert np.array_equal(res.masks[kh], expect) and res.budget[kh] == expect.sum()
        assert res.token_pos[kh].tolist() == [int(pos[kh][i]) for i in range(n) if expect[i]]


def test_recompress_after_a_first_pass_shrinks_and_keeps_the_map_consistent():
    rng = np.random.default_rng(44)
    H_q, H_kv, d_k, d_h, N, n_s = 4, 2, 8, 12, 40, 2
    h = rng.normal(size=(N, d_h))
    W = rng.normal(size=(H_q * d_k, d_h)) / math.sqrt(d_h)
    K = rng.normal(size=(H_kv, N, d_k)) * 1.5
    kw = dict(n_q_heads=H_q, d_k=d_k, theta=1e4, S=4, p_nuc=0.6, n_f=4, layer_id=0, request_id=0, include_c0=True)
    first = o.compress_request(h, W, None, K, n_s=n_s, seed=3, **kw)
    pos1 = [np.nonzero(first.mask[kh])[0] for kh in range(H_kv)]
    mu, var = o.fit(h, n_s)
    again = o.recompress_request(mu, var, h[-1], W, None, [K[kh][pos1[kh]] for kh in range(H_kv)], N, seed=4,
                                 token_pos=pos1, **kw)
    for kh in range(H_kv):
        assert again.budget[kh] <= first.budget[kh] and again.masks[kh].shape[0] == first.budget[kh]
        assert set(again.token_pos[kh].tolist()) <= set(pos1[kh].tolist())
        assert np.all(np.diff(again.token_pos[kh]) > 0)
    # the first pass kept the current query's own nucleus (include_c0), and the weights of a subset that
    # holds it only grow when renormalised: the nucleus cannot get larger
    assert np.all(again.b_step <= first.b_step)


def test_recompress_head_with_no_rows():
    W, mu, var, h_last, k0 = _recompress_problem(45, d_k=8, d_h=10, N0=9)
    K_heads = [_keys_at(k0[0], np.arange(9), 8, 1e4), np.zeros((0, 8))]
    res = o.recompress_request(mu, var, h_last, W, None, K_heads, 9, n_q_heads=4, d_k=8, theta=1e4, S=3, p_nuc=0.9,
                               n_f=2, seed=1, layer_id=0, request_id=0, token_pos=[np.arange(9), np.zeros(0, dtype=int)])
    assert res.budget[1] == 0 and res.masks[1].shape == (0,) and res.token_pos[1].shape == (0,)
    assert res.b_step[2] == 0 and res.b_step[3] == 0 and res.budget[0] >= res.b_step[:2].max() > 0


# ----------------------------------------------------------------------------- planted structure, end to end
def _planted_run(n_heavy, p_nuc):
    from paper_2509_03136_b200 import synth
    cfg = synth.make_planted(n_heavy, p_nuc=p_nuc)
    li = synth.make_layer(cfg, 0)
    res, _, _ = o.compress_layer(li.h, li.W_q, li.b_q, li.K, li.V, li.cu_seqlens, n_q_heads=cfg.n_q_heads, d_k=cfg.d_k,
                                 theta=cfg.rope_theta, S=cfg.S, p_nuc=float(np.float32(cfg.p_nuc)), n_f=cfg.n_f,
                                 n_s=cfg.n_s, seed=cfg.seed, layer_id=0)
    return cfg, li, res[0]


@pytest.mark.parametrize("n_heavy", [4, 12, 40])
def test_planted_keys_are_exactly_what_the_pass_keeps(n_heavy):
    """End to end on inputs whose answer is known by construction (Section 3.3: the union keeps what the
    queries need).  All queries nearly parallel, n_heavy planted keys per KV head that hold more than
    99.7 % of every query's attention between them in near-equal shares: with p = 0.99 the nucleus of
    the current query is the whole planted set, every synthetic query's top-k is that set, and the keep
    mask is exactly the planted positions - no more, no less."""
    cfg, li, r = _planted_run(n_heavy, 0.99)
    assert r.b_step.tolist() == [n_heavy] * cfg.n_q_heads
    for kh in range(cfg.n_kv_heads):
        assert np.array_equal(np.nonzero(r.mask[kh])[0], li.heavy_positions[(0, kh)])
        assert r.budget[kh] == n_heavy


def test_budget_tracks_the_planted_count():
    """Same construction at p = 0.9: near-equal planted weights make the nucleus ceil(0.9 n) of the n planted
    keys (up to the small spread of their weights), nothing outside the planted set is ever kept, and the
    budget grows with the planted count: the budget is set by the data, not by a quota."""
    budgets = []
    for n_heavy in (4, 12, 40, 120):
        cfg, li, r = _planted_run(n_heavy, 0.9)
        for kh in range(cfg.n_kv_heads):
            kept = np.nonzero(r.mask[kh])[0]
            assert np.isin(kept, li.heavy_positions[(0, kh)]).all()
            assert math.ceil(0.9 * n_heavy) <= r.budget[kh] <= n_heavy
            assert r.budget[kh] >= r.b_step[kh * cfg.G:(kh + 1) * cfg.G].max()       # |union| >= |C| (Section 3.3)
        budgets.append(int(r.budget.min()))
    assert budgets == sorted(budgets) and len(set(budgets)) == 4


def test_planted_positions_of_the_small_workloads_are_kept():
    """The heavy positions planted in the two small benchmark workloads are all in the keep mask."""
    from paper_2509_03136_b200 import synth
    for name in ("c0", "c1"):
        cfg = synth.make_config(name)
        li = synth.make_layer(cfg, 0)
        res, _, _ = o.compress_layer(li.h, li.W_q, li.b_q, li.K, li.V, li.cu_seqlens, n_q_heads=cfg.n_q_heads,
                                     d_k=cfg.d_k, theta=cfg.rope_theta, S=cfg.S, p_nuc=float(np.float32(cfg.p_nuc)),
                                     n_f=cfg.n_f, n_s=cfg.n_s, seed=cfg.seed, layer_id=0)
        for kh in range(cfg.n_kv_heads):
            assert res[0].mask[kh][li.heavy_positions[(0, kh)]].all()
