"""Parity of the CUDA library against the CPU oracle, stage by stage and end to end, through the
C ABI.  Tolerances (stated where used): Philox words and compaction bit-exact; fit 1e-5 relative;
normal draws 1e-5 absolute on z; rotated queries within one bf16 step; softmax rows 2e-2 relative
where the weight is >= 1e-6; masks identical outside the 1e-3 band around each selection
threshold; budgets within 0.5 % of N."""
import math
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import gvote_oracle as o
from paper_2509_03136_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gv():
    from paper_2509_03136_b200 import build as gbuild
    gbuild.build()
    from paper_2509_03136_b200 import gvote
    gvote.load()
    return gvote


def _geom(cfg):
    return (cfg.batch, cfg.total_tokens, max(cfg.seq_lens))


def _small_cfgs():
    return [
        synth.make_small(1, seq_lens=(40,), S=4),
        synth.make_small(2, seq_lens=(33, 64, 17), S=5, d_h=72, d_k=16),
        synth.make_small(3, seq_lens=(129, 31, 257), S=7, d_h=256, n_q_heads=6, n_kv_heads=2, d_k=64, n_f=16),
        synth.make_small(4, seq_lens=(1000,), S=9, d_h=128, n_q_heads=2, n_kv_heads=2, d_k=128, p_nuc=0.99),
    ]


# ----------------------------------------------------------------------------- sample
@pytest.mark.parametrize("d_h,S,batch", [(512, 16, 1), (72, 3, 4), (4096, 32, 2)])
def test_sample_philox_bit_exact_and_normals(gv, d_h, S, batch):
    seed, layer = 0x0123456789ABCDEF, 11
    p = gv.make_params(d_h=d_h, n_q_heads=8, n_kv_heads=2, d_k=64, rope_theta=1e4, S=S, p_nuc=0.95, n_f=8, n_s=0,
                       seed=seed, layer_id=layer)
    rng = np.random.default_rng(5)
    mu = rng.normal(size=(batch, d_h)).astype(np.float32)
    var = rng.uniform(0.1, 10, size=(batch, d_h)).astype(np.float32)
    H = torch.empty(batch, S, d_h, device="cuda")
    raw = torch.empty(batch, S, d_h, dtype=torch.int32, device="cuda")
    gv.gvote_sample(p, torch.from_numpy(mu).cuda(), torch.from_numpy(var).cuda(), batch, H, raw)
    H, raw = H.cpu().numpy(), raw.cpu().numpy().view(np.uint32)
    for r in range(batch):
        Ho, rawo = o.sample(mu[r].astype(np.float64), var[r].astype(np.float64), S, seed, layer, r)
        assert np.array_equal(raw[r], rawo[:, :d_h])                                   # bit-exact
        sig = np.sqrt(var[r].astype(np.float64))
        z_gpu = (H[r] - mu[r]) / sig
        z_or = (Ho - mu[r]) / sig
        assert np.abs(z_gpu - z_or).max() < 1e-5 + 2e-6 * np.abs(mu[r] / sig).max()    # 1e-5 abs on z


# ----------------------------------------------------------------------------- fit
@pytest.mark.parametrize("name,lens,d_h,n_s", [("a", (40,), 64, 2), ("b", (33, 64, 17), 72, 4),
                                               ("c", (5000, 700), 1024, 4), ("d", (6,), 8, 4)])
def test_fit_matches_oracle(gv, name, lens, d_h, n_s):
    rng = np.random.default_rng(7)
    T = sum(lens)
    h = (rng.normal(size=(T, d_h)) * rng.uniform(0.3, 3, size=d_h) + rng.normal(size=d_h) * 5).astype(np.float32)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    p = gv.make_params(d_h=d_h, n_q_heads=2, n_kv_heads=1, d_k=16, rope_theta=1e4, S=2, p_nuc=0.9, n_f=4, n_s=n_s,
                       seed=0)
    geom = (len(lens), T, max(lens))
    ws = gv.alloc_workspace(p, *geom)
    mu = torch.empty(len(lens), d_h, device="cuda")
    var = torch.empty_like(mu)
    gv.gvote_fit(p, torch.from_numpy(h).cuda(), torch.from_numpy(cu).cuda(), geom, mu, var, ws)
    for r in range(len(lens)):
        m, v = o.fit(h[cu[r]:cu[r + 1]], n_s)
        assert np.allclose(var[r].cpu().numpy(), v, rtol=1e-5, atol=0)
        assert np.abs(mu[r].cpu().numpy() - m).max() <= 1e-5 * np.sqrt(v).max() + 1e-6 * np.abs(m).max()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_fit_strided_rows_ragged_strips_and_long_chunks(gv, dtype):
    """Hidden states that are a column window of a wider buffer (row stride > d_h), d_h that leaves a
    partial 256-channel strip, one long request (many whole stages per chunk plus a ragged last one)
    next to short ones; the mean sits far from zero relative to the spread."""
    rng = np.random.default_rng(9)
    lens, d_h, ld, n_s = (9001, 70, 333), 328, 344, 4
    T = sum(lens)
    wide = (rng.normal(size=(T, ld)) * rng.uniform(0.05, 2, size=ld) + rng.normal(size=ld) * 40).astype(np.float32)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    bf = dtype == "bf16"
    buf = torch.from_numpy(wide).cuda()
    if bf:
        buf = buf.bfloat16()
    h = buf[:, 8:8 + d_h]                                  # 16-byte aligned window, stride ld
    href = h.double().cpu().numpy()
    p = gv.make_params(d_h=d_h, n_q_heads=2, n_kv_heads=1, d_k=16, rope_theta=1e4, S=2, p_nuc=0.9, n_f=4, n_s=n_s,
                       seed=0, h_dtype=gv.DTYPE_BF16 if bf else gv.DTYPE_F32)
    geom = (len(lens), T, max(lens))
    ws = gv.alloc_workspace(p, *geom)
    mu = torch.empty(len(lens), d_h, device="cuda"); var = torch.empty_like(mu)
    gv.gvote_fit(p, h, torch.from_numpy(cu).cuda(), geom, mu, var, ws)
    assert gv.gvote_poll_status(ws) == 0
    for r in range(len(lens)):
        m, v = o.fit(href[cu[r]:cu[r + 1]], n_s)
        assert np.allclose(var[r].cpu().numpy(), v, rtol=1e-5, atol=0)
        assert np.abs(mu[r].cpu().numpy() - m).max() <= 1e-5 * np.sqrt(v).max() + 1e-6 * np.abs(m).max()


def test_fit_bf16_hidden_states(gv):
    rng = np.random.default_rng(8)
    h = torch.from_numpy(rng.normal(size=(300, 128)).astype(np.float32)).bfloat16()
    cu = np.array([0, 300], dtype=np.int32)
    p = gv.make_params(d_h=128, n_q_heads=2, n_kv_heads=1, d_k=16, rope_theta=1e4, S=2, p_nuc=0.9, n_f=4, n_s=4,
                       seed=0, h_dtype=gv.DTYPE_BF16)
    geom = (1, 300, 300)
    ws = gv.alloc_workspace(p, *geom)
    mu = torch.empty(1, 128, device="cuda"); var = torch.empty_like(mu)
    gv.gvote_fit(p, h.cuda(), torch.from_numpy(cu).cuda(), geom, mu, var, ws)
    m, v = o.fit(h.double().numpy(), 4)
    assert np.allclose(var[0].cpu().numpy(), v, rtol=1e-5) and np.allclose(mu[0].cpu().numpy(), m, atol=1e-5)


# ----------------------------------------------------------------------------- project
@pytest.mark.parametrize("idx", range(4))
@pytest.mark.parametrize("bias", [False, True])
def test_project_matches_oracle(gv, idx, bias):
    cfg = _small_cfgs()[idx]
    li = synth.make_layer(cfg, 0, with_bias=bias)
    p = gv.params_from_config(cfg)
    rng = np.random.default_rng(9)
    Ht = rng.normal(size=(cfg.batch, cfg.S, cfg.d_h)).astype(np.float32) * 2
    hl = rng.normal(size=(cfg.batch, cfg.d_h)).astype(np.float32)
    d = pu.upload_layer(li, gv, torch)
    ws = gv.alloc_workspace(p, *_geom(cfg))
    Q = torch.empty(cfg.batch, cfg.n_kv_heads, cfg.G * (cfg.S + 1), cfg.d_k, dtype=torch.bfloat16, device="cuda")
    gv.gvote_project(p, torch.from_numpy(Ht).cuda(), torch.from_numpy(hl).cuda(), d["W_q"], d["b_q"], d["cu"],
                     cfg.batch, Q, ws)
    Qg = Q.float().cpu().numpy().astype(np.float64)
    W = o.bf16_bits_to_f64(li.W_q)
    for r in range(cfg.batch):
        Qo = o.queries_for_request(Ht[r].astype(np.float64), hl[r].astype(np.float64), W, li.b_q, cfg.seq_lens[r],
                                   n_q_heads=cfg.n_q_heads, d_k=cfg.d_k, theta=cfg.rope_theta, n_f=cfg.n_f)
        diff = np.abs(pu.from_group_major(Qg[r], cfg.G) - Qo)
        assert np.all(diff <= 2.0 ** -7 * np.abs(Qo) + 1e-6)            # at most one bf16 step
        assert (diff == 0).mean() > 0.98


# ----------------------------------------------------------------------------- vote (given the oracle's queries)
def _run_vote(gv, cfg, li, Q_or, sel_mode, include_c0, want_probs):
    p = gv.params_from_config(cfg, sel_mode=gv.SEL_TOPP if sel_mode == "topp" else gv.SEL_TOPK_C0,
                              include_c0=include_c0)
    geom = _geom(cfg)
    ws = gv.alloc_workspace(p, *geom, softmax_dump=want_probs)
    K = gv.bf16_from_bits(li.K)
    cu = torch.from_numpy(li.cu_seqlens).cuda()
    Qgm = np.ascontiguousarray(np.stack([pu.to_group_major(q, cfg.G) for q in Q_or]))
    Qd = torch.from_numpy(Qgm).to(torch.bfloat16).contiguous().cuda()   # values are on the bf16 grid already
    mask = torch.full((cfg.n_kv_heads, gv.mask_row_words(cfg.total_tokens, cfg.batch)), -1, dtype=torch.int32,
                      device="cuda")
    budget = torch.empty(cfg.batch, cfg.n_kv_heads, dtype=torch.int32, device="cuda")
    b_step = torch.empty(cfg.batch, cfg.n_q_heads, dtype=torch.int32, device="cuda")
    probs = None
    if want_probs:
        probs = torch.empty(cfg.n_q_heads * (cfg.S + 1) * cfg.total_tokens, device="cuda")
    gv.gvote_vote(p, Qd, K, cu, geom, mask, budget, b_step, ws, probs)
    assert gv.gvote_poll_status(ws) == 0
    _run_vote.exact_heads = gv.gvote_exact_heads(ws)
    return mask.cpu().numpy(), budget.cpu().numpy(), b_step.cpu().numpy(), None if probs is None else probs.cpu().numpy()


def _oracle_queries(cfg, li, seed=None):
    W = o.bf16_bits_to_f64(li.W_q)
    out = []
    for r in range(cfg.batch):
        a, b = int(li.cu_seqlens[r]), int(li.cu_seqlens[r + 1])
        h = li.h[a:b].astype(np.float64)
        mu, var = o.fit(h, cfg.n_s)
        Ht, _ = o.sample(mu, var, cfg.S, cfg.seed if seed is None else seed, 0, r)
        out.append(o.queries_for_request(Ht, h[-1], W, li.b_q, b - a, n_q_heads=cfg.n_q_heads, d_k=cfg.d_k,
                                         theta=cfg.rope_theta, n_f=cfg.n_f))
    return out


def _check_vote(gv, cfg, li, sel_mode, include_c0=False, want_probs=True):
    Q_or = _oracle_queries(cfg, li)
    mask, budget, b_step, probs = _run_vote(gv, cfg, li, Q_or, sel_mode, include_c0, want_probs)
    pf = float(np.float32(cfg.p_nuc))
    poff = 0
    for r in range(cfg.batch):
        a, b = int(li.cu_seqlens[r]), int(li.cu_seqlens[r + 1])
        N = b - a
        Kr = o.bf16_bits_to_f64(li.K[:, a:b])
        gm = np.stack([gv.unpack_mask(mask[h], gv.mask_word_offset(a, r), N) for h in range(cfg.n_kv_heads)])
        pu.check_vote_against_oracle(Q_or[r], Kr, pf, sel_mode, include_c0, gm, b_step[r])
        om, ob, obs, _, op = o.vote(Q_or[r], Kr, p_nuc=pf, sel_mode=sel_mode, include_c0=include_c0,
                                    keep_probs=want_probs)
        assert np.array_equal(budget[r], gm.sum(axis=1))                     # budget = popcount
        assert np.all(np.abs(budget[r] - ob) <= max(1, 0.005 * N))           # within 0.5 % of N
        assert (gm != om).sum() <= max(2, 0.005 * N * cfg.n_kv_heads)
        if want_probs:
            pg = probs[poff:poff + cfg.n_q_heads * (cfg.S + 1) * N].reshape(cfg.n_q_heads, cfg.S + 1, N)
            big = op >= 1e-6
            assert np.abs(pg[big] / op[big] - 1.0).max() < 2e-2              # stated score tolerance
            poff += cfg.n_q_heads * (cfg.S + 1) * N
        # padding bits of the request's last word stay zero
        if N % 32:
            last = mask[:, gv.mask_word_offset(a, r) + N // 32].view(np.uint32)
            assert np.all(last >> np.uint32(N % 32) == 0)


# "topk" asks for the softmax rows too, which takes the route that keeps fp32 logits of every row;
# "topk-fused" is the default route (no S x N logits anywhere), as the whole pass runs it
@pytest.mark.parametrize("idx", range(4))
@pytest.mark.parametrize("mode", ["topk", "topk-fused", "topp"])
def test_vote_small(gv, idx, mode):
    cfg = _small_cfgs()[idx]
    _check_vote(gv, cfg, synth.make_layer(cfg, 0), mode.split("-")[0], want_probs=not mode.endswith("fused"))


@pytest.mark.parametrize("probs", [True, False])
def test_vote_include_c0(gv, probs):
    cfg = _small_cfgs()[2]
    _check_vote(gv, cfg, synth.make_layer(cfg, 0), "topk", include_c0=True, want_probs=probs)


@pytest.mark.parametrize("name,mode", [("c0", "topk"), ("c0", "topk-fused"), ("c0", "topp"), ("c1", "topk"),
                                       ("c1", "topk-fused"), ("c1", "topp"), ("c3", "topk-fused")])
def test_vote_configs(gv, name, mode):
    cfg = synth.make_config(name)
    _check_vote(gv, cfg, synth.make_layer(cfg, 0), mode.split("-")[0], want_probs=not mode.endswith("fused"))


def test_vote_many_row_chunks_strict_band(gv):
    """G = 7 query heads per KV head and S = 64 synthetic queries: 448 synthetic rows per KV head, i.e.
    four 128-row chunks in the score contraction, on rows long enough for the sampled bracket (ragged
    last tile).  Oracle's queries, default 1e-3 bands."""
    cfg = synth.make_small(21, seq_lens=(9001,), S=64, d_h=128, n_q_heads=7, n_kv_heads=1, d_k=128, p_nuc=0.98,
                           heavy_frac=(0.01,))
    _check_vote(gv, cfg, synth.make_layer(cfg, 0), "topk", want_probs=False)


@pytest.mark.parametrize("lens", [(3000,), (9001, 700)])
def test_vote_more_row_chunks_than_one_cta_holds(gv, lens):
    """S = 330 synthetic queries for each of 2 heads per KV head: 660 rows, six 128-row chunks, more than the
    four a CTA of the second pass holds (two chunk groups there, three in the first pass), the last chunk
    partly empty.  Oracle's queries, default 1e-3 bands."""
    cfg = synth.make_small(26, seq_lens=lens, S=330, d_h=64, n_q_heads=4, n_kv_heads=2, d_k=128, p_nuc=0.9,
                           heavy_frac=(0.01,))
    _check_vote(gv, cfg, synth.make_layer(cfg, 0), "topk", want_probs=False)
    assert _run_vote.exact_heads == 0


@pytest.mark.parametrize("lens", [(4097,), (4224, 8191, 127), (4096, 2, 3, 129), (12345,)])
def test_vote_lengths_around_the_sampling_switch(gv, lens):
    """Rows of exactly 32 key tiles are still sampled completely, 33 tiles are the first sampled in part
    (stride 1: every full tile, the ragged one left out); ragged batches mix both kinds, two-key and three-key
    requests included.  G = 3 heads of S = 50 synthetic queries give 150 rows per KV head: a second row chunk
    that is mostly empty.  Oracle's queries, default 1e-3 bands."""
    cfg = synth.make_small(25, seq_lens=lens, S=50, d_h=64, n_q_heads=6, n_kv_heads=2, d_k=64, p_nuc=0.93,
                           heavy_frac=(0.02,), n_s=0)
    _check_vote(gv, cfg, synth.make_layer(cfg, 0), "topk", want_probs=False)
    assert _run_vote.exact_heads == 0


@pytest.mark.parametrize("N", [33000, 50001])
def test_vote_topp_long_rows_strict_band(gv, N):
    """Per-sample top-p on rows of more than 32K keys (N = 50001 no longer fits the shared-memory
    staging of a row).  Oracle's queries, default 1e-3 bands."""
    cfg = synth.make_small(22, seq_lens=(N,), S=3, d_h=64, n_q_heads=2, n_kv_heads=1, d_k=64, p_nuc=0.95,
                           heavy_frac=(0.002,))
    _check_vote(gv, cfg, synth.make_layer(cfg, 0), "topp", want_probs=False)


def test_budget_grows_with_S_and_with_p(gv):
    """Section 3.5 / Section 4.4: more synthetic queries or a larger nucleus can only add keys.  The samples
    are counter based, so the first S' draws of an S-run are the S'-run: keep masks are nested in S (bit for
    bit); budgets do not shrink as p grows; and every setting's budget agrees with the oracle's."""
    import bench
    cfg = synth.make_small(23, seq_lens=(700, 333), S=8, d_h=128, n_q_heads=4, n_kv_heads=2, d_k=64, p_nuc=0.9,
                           heavy_frac=(0.03,))
    li = synth.make_layer(cfg, 0)
    d = pu.upload_layer(li, gv, torch)
    p0 = gv.params_from_config(cfg)
    geom = _geom(cfg)
    ws = gv.alloc_workspace(p0, *geom)
    mu = torch.empty(cfg.batch, cfg.d_h, device="cuda"); var = torch.empty_like(mu)
    gv.gvote_fit(p0, d["h"], d["cu"], geom, mu, var, ws)
    cu = li.cu_seqlens
    h_last = torch.from_numpy(np.stack([li.h[int(cu[r + 1]) - 1] for r in range(cfg.batch)])).cuda()
    W = o.bf16_bits_to_f64(li.W_q)

    def oracle_budget(S, pn):
        out = []
        for r in range(cfg.batch):
            a, b = int(cu[r]), int(cu[r + 1])
            kw = pu.oracle_kwargs(cfg)
            kw.update(S=S, p_nuc=float(np.float32(pn)))
            out.append(o.compress_request(li.h[a:b].astype(np.float64), W, li.b_q, o.bf16_bits_to_f64(li.K[:, a:b]),
                                          request_id=r, **kw).budget)
        return np.stack(out)

    prev = None
    for S in (1, 2, 4, 8, 16):
        mask, budget, ov, _ = bench.select_once(gv, torch, cfg, li, d, S, 0.9, mu, var, h_last, reps=1)
        if prev is not None:
            assert np.all((prev & ~mask) == 0)                                  # nested in S
        prev = mask
        assert np.all(np.abs(budget - oracle_budget(S, 0.9)) <= 4)
        assert np.all((ov >= 0) & (ov <= 1 + 1e-5))
    last = None
    for pn in (0.5, 0.8, 0.9, 0.97):
        _, budget, ov, _ = bench.select_once(gv, torch, cfg, li, d, 8, pn, mu, var, h_last, reps=1)
        if last is not None:
            assert np.all(budget >= last)                                       # monotone in p
        last = budget
        assert np.all(np.abs(budget - oracle_budget(8, pn)) <= 4)


@pytest.mark.parametrize("d_k,G", [(256, 2), (192, 1), (64, 17)])
def test_vote_shapes_outside_the_fused_route(gv, d_k, G):
    """Head dimensions above 128 and more than 16 query heads per KV head are served by the kernels that keep
    fp32 rows (the workspace is sized for them): same answers, same bands."""
    cfg = synth.make_small(24, seq_lens=(300, 1100), S=5, d_h=64, n_q_heads=2 * G, n_kv_heads=2, d_k=d_k, p_nuc=0.9)
    _check_vote(gv, cfg, synth.make_layer(cfg, 0), "topk", want_probs=False)
    _check_compress(gv, cfg, synth.make_layer(cfg, 0))


def test_vote_degenerate_all_keys_equal(gv):
    """Every logit ties: top-p keeps ceil(p N) keys and top-k keeps exactly k, lowest indices first."""
    cfg = synth.make_small(5, seq_lens=(100,), S=3, d_h=64, n_q_heads=2, n_kv_heads=1, d_k=32, p_nuc=0.5)
    li = synth.make_layer(cfg, 0)
    li.K[:] = li.K[:, :1, :]                                                 # one key repeated
    Q_or = _oracle_queries(cfg, li)
    mask, budget, b_step, _ = _run_vote(gv, cfg, li, Q_or, "topk", False, False)
    assert b_step.tolist() == [[50, 50]] and budget.tolist() == [[50]]
    gm = gv.unpack_mask(mask[0], 0, 100)
    assert gm[:50].all() and not gm[50:].any()


def test_vote_single_dominant_key(gv):
    cfg = synth.make_small(6, seq_lens=(77,), S=4, d_h=64, n_q_heads=2, n_kv_heads=1, d_k=32, p_nuc=0.95)
    li = synth.make_layer(cfg, 0)
    Q_or = _oracle_queries(cfg, li)
    Kf = np.zeros((1, 77, 32), dtype=np.float32)
    # key 13 lines up with every row of every head by construction: sum of the sign patterns
    qsum = np.sign(np.concatenate([Q_or[0][g] for g in range(2)]).sum(axis=0))
    Kf[0, 13] = 40.0 * qsum
    li.K = synth.f32_to_bf16_bits(Kf)
    Kr = o.bf16_bits_to_f64(li.K)
    om, ob, obs, _, _ = o.vote(Q_or[0], Kr, p_nuc=float(np.float32(0.95)))
    mask, budget, b_step, _ = _run_vote(gv, cfg, li, Q_or, "topk", False, False)
    assert b_step[0].tolist() == obs.tolist()
    assert np.array_equal(gv.unpack_mask(mask[0], 0, 77), om[0])


@pytest.mark.parametrize("shift_sampled,shift_sign", [(0.0, 0.0), (-6.0, 0.0), (+6.0, 0.0), (0.0, 1.0)])
def test_vote_long_rows_with_misleading_sample(gv, shift_sampled, shift_sign):
    """Rows long enough for the sampled bracket of the fused top-k.  The kernels sample whole 128-key tiles
    (one from every stretch of `stride` tiles, at a hashed offset); shifting the logits of exactly those
    tiles makes the sample's bracket miss the true threshold, so the exact route has to take over.
    shift_sign = 1 centres the logits on zero with tiny magnitudes (half-precision codes are densest
    there)."""
    N, d_k, S = 16384, 64, 6
    cfg = synth.make_small(11, seq_lens=(N,), S=S, d_h=64, n_q_heads=2, n_kv_heads=1, d_k=d_k, p_nuc=0.9)
    li = synth.make_layer(cfg, 0)
    rng = np.random.default_rng(3)
    e = rng.normal(size=d_k)
    e /= np.linalg.norm(e)
    v = rng.normal(size=N) * (1e-3 if shift_sign else 1.0)
    sampled = np.zeros(N, dtype=bool)
    n_tiles = N // 128
    want = min(max(n_tiles >> 3, 32), 128)               # the sampling plan of the kernels (vote_geom.cuh)
    stride = n_tiles // want
    for j in range(want):
        t = j * stride + (((j * 2654435761) & 0xFFFFFFFF) >> 15) % stride
        sampled[t * 128:(t + 1) * 128] = True
    v[sampled] += shift_sampled
    Kf = (v[:, None] * e[None, :] * math.sqrt(d_k)).astype(np.float32)[None]          # logit of key n = v_n q.e
    li.K = synth.f32_to_bf16_bits(Kf)
    q = o.round_to_bf16(np.stack([e * (1.0 + 0.05 * r) for r in range(S + 1)]))     # rows differ a little
    Q_or = [np.stack([q, q[::-1].copy()])]
    mask, budget, b_step, _ = _run_vote(gv, cfg, li, Q_or, "topk", False, False)
    # a shifted sample makes the bracket miss: the head must have gone the exact way (and only then)
    assert _run_vote.exact_heads == (1 if shift_sampled else 0), _run_vote.exact_heads
    Kr = o.bf16_bits_to_f64(li.K)
    gm = np.stack([gv.unpack_mask(mask[0], 0, N)])
    pu.check_vote_against_oracle(Q_or[0], Kr, float(np.float32(cfg.p_nuc)), "topk", False, gm, b_step[0])
    om, ob, _, _, _ = o.vote(Q_or[0], Kr, p_nuc=float(np.float32(cfg.p_nuc)))
    assert abs(int(budget[0, 0]) - int(ob[0])) <= 0.005 * N


def test_vote_exact_route_for_some_heads_of_a_batch(gv):
    """Three requests, two KV heads each, 512 synthetic rows (four row chunks) per head.  The samples of the
    first and the last request are shifted so that their brackets miss: four (request, KV head) pairs are
    selected again by the exact route while the request in the middle keeps its sampled result."""
    N, d_k, S, Hq, Hkv = 8192, 64, 64, 16, 2
    cfg = synth.make_small(12, seq_lens=(N, N, N), S=S, d_h=64, n_q_heads=Hq, n_kv_heads=Hkv, d_k=d_k, p_nuc=0.9)
    li = synth.make_layer(cfg, 0)
    rng = np.random.default_rng(5)
    e = rng.normal(size=d_k)
    e /= np.linalg.norm(e)
    n_tiles = N // 128
    want = min(max(n_tiles >> 3, 32), 128)               # the sampling plan of the kernels (vote_geom.cuh)
    stride = n_tiles // want
    sampled = np.zeros(N, dtype=bool)
    for j in range(want):
        t = j * stride + (((j * 2654435761) & 0xFFFFFFFF) >> 15) % stride
        sampled[t * 128:(t + 1) * 128] = True
    Kf = np.empty((Hkv, 3 * N, d_k), dtype=np.float32)
    for r in range(3):
        v = rng.normal(size=N)
        if r != 1:
            v[sampled] -= 6.0
        Kf[:, r * N:(r + 1) * N] = (v[:, None] * e[None, :] * math.sqrt(d_k)).astype(np.float32)[None]
    li.K = synth.f32_to_bf16_bits(Kf)
    q = o.round_to_bf16(np.stack([e * (1.0 + 0.01 * i) for i in range(S + 1)]))
    Q_or = [np.stack([q if g % 2 == 0 else q[::-1].copy() for g in range(Hq)]) for _ in range(3)]
    mask, budget, b_step, _ = _run_vote(gv, cfg, li, Q_or, "topk", False, False)
    assert _run_vote.exact_heads == 4, _run_vote.exact_heads
    for r in range(3):
        Kr = o.bf16_bits_to_f64(li.K[:, r * N:(r + 1) * N])
        gm = np.stack([gv.unpack_mask(mask[h], gv.mask_word_offset(r * N, r), N) for h in range(Hkv)])
        pu.check_vote_against_oracle(Q_or[r], Kr, float(np.float32(cfg.p_nuc)), "topk", False, gm, b_step[r])
        om, ob, _, _, _ = o.vote(Q_or[r], Kr, p_nuc=float(np.float32(cfg.p_nuc)))
        assert np.all(np.abs(budget[r] - ob) <= 0.005 * N)


# ----------------------------------------------------------------------------- compact
@pytest.mark.parametrize("lens,Hkv,d_k,density", [((40,), 2, 32, 0.5), ((129, 31, 257), 2, 64, 0.2),
                                                  ((5000, 300), 3, 128, 0.7), ((4096,), 8, 128, 0.05),
                                                  ((1000,), 1, 8, 1.0), ((1000,), 1, 16, 0.0),
                                                  ((131072,), 4, 128, 0.01), ((131072,), 4, 128, 0.3),
                                                  ((131072,), 8, 128, 0.9), ((131072,), 4, 128, 0.7)])
def test_compact_bit_exact(gv, lens, Hkv, d_k, density):
    rng = np.random.default_rng(12)
    T, B = sum(lens), len(lens)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    K = rng.integers(0, 65536, size=(Hkv, T, d_k)).astype(np.uint16)
    V = rng.integers(0, 65536, size=(Hkv, T, d_k)).astype(np.uint16)
    keep = rng.random((Hkv, T)) < density
    if density == 0.7:
        keep[0, :T // 3 + 135] = True                                         # long fully-kept prefix
        if Hkv > 1:
            keep[1, :] = True                                                 # a head that keeps every key
    words = np.zeros((Hkv, gv.mask_row_words(T, B)), dtype=np.uint32)
    for r in range(B):
        for h in range(Hkv):
            w = o.pack_mask_bits(keep[h, cu[r]:cu[r + 1]])
            off = gv.mask_word_offset(int(cu[r]), r)
            words[h, off:off + len(w)] = w
    p = gv.make_params(d_h=64, n_q_heads=Hkv, n_kv_heads=Hkv, d_k=d_k, rope_theta=1e4, S=2, p_nuc=0.9, n_f=4, n_s=0,
                       seed=0)
    geom = (B, T, max(lens))
    ws = gv.alloc_workspace(p, *geom)
    Kd, Vd = gv.bf16_from_bits(K), gv.bf16_from_bits(V)
    budget = torch.empty(B, Hkv, dtype=torch.int32, device="cuda")
    md = torch.from_numpy(words.view(np.int32)).cuda()
    for rep in range(2):                                                      # second run: same flags reused
        Kd.copy_(gv.bf16_from_bits(K)); Vd.copy_(gv.bf16_from_bits(V))
        gv.gvote_compact(p, Kd, Vd, md, torch.from_numpy(cu).cuda(), geom, budget, ws)
        assert gv.gvote_poll_status(ws) == 0
        Kg, Vg, bg = gv.bits_from_bf16(Kd), gv.bits_from_bf16(Vd), budget.cpu().numpy()
        for r in range(B):
            a, b = int(cu[r]), int(cu[r + 1])
            Kc, Vc = o.compact(K[:, a:b], V[:, a:b], keep[:, a:b])
            for h in range(Hkv):
                n = Kc[h].shape[0]
                assert bg[r, h] == n
                assert np.array_equal(Kg[h, a:a + n], Kc[h]) and np.array_equal(Vg[h, a:a + n], Vc[h])


def test_compact_strided_heads(gv):
    """K and V as views of a [T, Hkv, d_k] cache (token-major), not dense per head."""
    rng = np.random.default_rng(13)
    T, Hkv, d_k = 700, 2, 64
    base = rng.integers(0, 65536, size=(2, T, Hkv, d_k)).astype(np.uint16)
    keep = rng.random((Hkv, T)) < 0.3
    words = np.stack([o.pack_mask_bits(keep[h]) for h in range(Hkv)])
    words = np.concatenate([words, np.zeros((Hkv, gv.mask_row_words(T, 1) - words.shape[1]), np.uint32)], axis=1)
    p = gv.make_params(d_h=64, n_q_heads=Hkv, n_kv_heads=Hkv, d_k=d_k, rope_theta=1e4, S=2, p_nuc=0.9, n_f=4, n_s=0,
                       seed=0)
    geom = (1, T, T)
    ws = gv.alloc_workspace(p, *geom)
    KV = gv.bf16_from_bits(base)
    Kd, Vd = KV[0].permute(1, 0, 2), KV[1].permute(1, 0, 2)                   # [Hkv, T, d_k] strided
    budget = torch.empty(1, Hkv, dtype=torch.int32, device="cuda")
    gv.gvote_compact(p, Kd, Vd, torch.from_numpy(words.view(np.int32)).cuda(),
                     torch.tensor([0, T], dtype=torch.int32, device="cuda"), geom, budget, ws)
    out = gv.bits_from_bf16(KV)
    for h in range(Hkv):
        n = int(keep[h].sum())
        assert np.array_equal(out[0, :n, h], base[0, keep[h], h]) and np.array_equal(out[1, :n, h], base[1, keep[h], h])


# ----------------------------------------------------------------------------- attention overlap
@pytest.mark.parametrize("idx", range(4))
def test_overlap_matches_oracle(gv, idx):
    """gvote_overlap on the mask gvote_vote produced, against the oracle on the same mask: fp32 logits
    of bf16 operands against fp64, 1e-4 absolute on a number in [0, 1]."""
    cfg = _small_cfgs()[idx]
    li = synth.make_layer(cfg, 0)
    Q_or = _oracle_queries(cfg, li)
    mask, budget, b_step, _ = _run_vote(gv, cfg, li, Q_or, "topk", False, False)
    p = gv.params_from_config(cfg)
    geom = _geom(cfg)
    ws = gv.alloc_workspace(p, *geom)
    Qgm = np.ascontiguousarray(np.stack([pu.to_group_major(q, cfg.G) for q in Q_or]))
    Qd = torch.from_numpy(Qgm).to(torch.bfloat16).contiguous().cuda()
    ov = torch.empty(cfg.batch, cfg.n_q_heads, device="cuda")
    gv.gvote_overlap(p, Qd, gv.bf16_from_bits(li.K), torch.from_numpy(mask).cuda(), torch.from_numpy(li.cu_seqlens).cuda(),
                     geom, ov, ws)
    ov = ov.cpu().numpy()
    for r in range(cfg.batch):
        a, b = int(li.cu_seqlens[r]), int(li.cu_seqlens[r + 1])
        gm = np.stack([gv.unpack_mask(mask[h], gv.mask_word_offset(a, r), b - a) for h in range(cfg.n_kv_heads)])
        ref = o.attention_overlap(Q_or[r], o.bf16_bits_to_f64(li.K[:, a:b]), gm)
        assert np.abs(ov[r] - ref).max() < 1e-4, (ov[r], ref)


# ----------------------------------------------------------------------------- varlen packing
@pytest.mark.parametrize("lens,Hkv,d_k,density", [((40,), 2, 32, 0.5), ((129, 31, 257), 2, 64, 0.2),
                                                  ((5000, 300), 3, 128, 0.7), ((4096,), 8, 128, 0.05),
                                                  ((1000,), 1, 8, 1.0), ((1000, 77), 2, 16, 0.0),
                                                  ((131072,), 4, 128, 0.01), ((131072,), 4, 128, 0.9)])
def test_pack_varlen_bit_exact(gv, lens, Hkv, d_k, density):
    """gvote_pack against the oracle's packing, bit for bit, with K and V left untouched."""
    rng = np.random.default_rng(31)
    T, B = sum(lens), len(lens)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    K = rng.integers(0, 65536, size=(Hkv, T, d_k)).astype(np.uint16)
    V = rng.integers(0, 65536, size=(Hkv, T, d_k)).astype(np.uint16)
    keep = rng.random((Hkv, T)) < density
    words = np.zeros((Hkv, gv.mask_row_words(T, B)), dtype=np.uint32)
    for r in range(B):
        for h in range(Hkv):
            w = o.pack_mask_bits(keep[h, cu[r]:cu[r + 1]])
            off = gv.mask_word_offset(int(cu[r]), r)
            words[h, off:off + len(w)] = w
    Ko, Vo, cu_k = o.pack_varlen(K, V, cu, [keep[:, cu[r]:cu[r + 1]] for r in range(B)])
    p = gv.make_params(d_h=64, n_q_heads=Hkv, n_kv_heads=Hkv, d_k=d_k, rope_theta=1e4, S=2, p_nuc=0.9, n_f=4, n_s=0,
                       seed=0)
    geom = (B, T, max(lens))
    ws = gv.alloc_workspace(p, *geom)
    Kd, Vd = gv.bf16_from_bits(K), gv.bf16_from_bits(V)
    rows = max(int(cu_k[-1]), 1)
    Kp = torch.zeros(rows, d_k, dtype=torch.bfloat16, device="cuda"); Vp = torch.zeros_like(Kp)
    cuk = torch.full((B * Hkv + 1,), -1, dtype=torch.int32, device="cuda")
    budget = torch.empty(B, Hkv, dtype=torch.int32, device="cuda")
    md = torch.from_numpy(words.view(np.int32)).cuda()
    for rep in range(2):
        gv.gvote_pack(p, Kd, Vd, md, torch.from_numpy(cu).cuda(), geom, Kp, Vp, cuk, budget, ws)
        assert gv.gvote_poll_status(ws) == 0
        assert np.array_equal(cuk.cpu().numpy(), cu_k)
        assert np.array_equal(budget.cpu().numpy().ravel(), np.diff(cu_k))
        n = int(cu_k[-1])
        assert np.array_equal(gv.bits_from_bf16(Kp)[:n], Ko) and np.array_equal(gv.bits_from_bf16(Vp)[:n], Vo)
        assert np.array_equal(gv.bits_from_bf16(Kd), K) and np.array_equal(gv.bits_from_bf16(Vd), V)


def test_pack_varlen_reports_buffers_that_are_too_small(gv):
    rng = np.random.default_rng(32)
    T, Hkv, d_k = 600, 2, 32
    K = rng.integers(0, 65536, size=(Hkv, T, d_k)).astype(np.uint16)
    keep = np.ones((Hkv, T), dtype=bool)
    words = np.stack([np.concatenate([o.pack_mask_bits(keep[h]), np.zeros(1, np.uint32)]) for h in range(Hkv)])
    words = words[:, :gv.mask_row_words(T, 1)]
    p = gv.make_params(d_h=64, n_q_heads=Hkv, n_kv_heads=Hkv, d_k=d_k, rope_theta=1e4, S=2, p_nuc=0.9, n_f=4, n_s=0,
                       seed=0)
    geom = (1, T, T)
    ws = gv.alloc_workspace(p, *geom)
    Kd = gv.bf16_from_bits(K)
    Kp = torch.zeros(700, d_k, dtype=torch.bfloat16, device="cuda"); Vp = torch.zeros_like(Kp)   # 1200 rows are kept
    cuk = torch.empty(Hkv + 1, dtype=torch.int32, device="cuda")
    budget = torch.empty(1, Hkv, dtype=torch.int32, device="cuda")
    gv.gvote_pack(p, Kd, Kd, torch.from_numpy(np.ascontiguousarray(words).view(np.int32)).cuda(),
                  torch.tensor([0, T], dtype=torch.int32, device="cuda"), geom, Kp, Vp, cuk, budget, ws)
    assert gv.gvote_poll_status(ws) == -3
    assert cuk.cpu().numpy().tolist() == [0, 600, 1200]
    assert np.array_equal(gv.bits_from_bf16(Kp)[:600], K[0])          # what fits is written
    assert gv.gvote_poll_status(ws) == -3                               # the status stays until it is cleared
    gv.gvote_clear_status(ws)
    assert gv.gvote_poll_status(ws) == 0


# ----------------------------------------------------------------------------- whole pass
def _queries_left_in(gv, p, ws, geom):
    """The rotated queries a whole-pass call left in its workspace, [batch, H_kv, G (S+1), d_k] as fp64."""
    return gv.workspace_queries(p, ws, *geom).float().cpu().numpy().astype(np.float64)


def _check_mask_against_own_queries(gv, cfg, Qg_r, Qo, K64, p_nuc, sel_mode, gm, b_step_r):
    """Whole pass, second half: the mask against the oracle's vote on the queries the GPU itself used, inside
    the 1e-3 bands.  Those queries against the oracle's: the GPU fits in fp32 and draws with fp32
    Box-Muller, so an entry of X can land on the neighbouring bf16 value and move every product of its row
    by |w| ulp(x): bounded here by one bf16 step of the entry plus 2^-6 of the row's largest entry (a wrong
    sign, index or rotation is off by the query's own magnitude), and nine entries in ten must be equal."""
    G = cfg.n_q_heads // cfg.n_kv_heads
    Qr = pu.from_group_major(Qg_r, G)
    scale = np.abs(Qo).max(axis=-1, keepdims=True)
    assert np.all(np.abs(Qr - Qo) <= 2.0 ** -7 * np.abs(Qo) + 2.0 ** -6 * scale), np.abs(Qr - Qo).max()
    assert (Qr == Qo).mean() > 0.9
    pu.check_vote_against_oracle(Qr, K64, p_nuc, sel_mode, False, gm, b_step_r)          # 1e-3 bands


def _run_compress(gv, cfg, li, sel_mode="topk", layer_id=0):
    p = gv.params_from_config(cfg, layer_id=layer_id, sel_mode=gv.SEL_TOPP if sel_mode == "topp" else gv.SEL_TOPK_C0)
    geom = _geom(cfg)
    ws = gv.alloc_workspace(p, *geom)
    d = pu.upload_layer(li, gv, torch)
    mask = torch.empty(cfg.n_kv_heads, gv.mask_row_words(cfg.total_tokens, cfg.batch), dtype=torch.int32, device="cuda")
    budget = torch.empty(cfg.batch, cfg.n_kv_heads, dtype=torch.int32, device="cuda")
    b_step = torch.empty(cfg.batch, cfg.n_q_heads, dtype=torch.int32, device="cuda")
    gv.gvote_compress(p, d["h"], d["W_q"], d["b_q"], d["K"], d["V"], d["cu"], geom, mask, budget, b_step, ws)
    assert gv.gvote_poll_status(ws) == 0
    return (mask.cpu().numpy(), budget.cpu().numpy(), b_step.cpu().numpy(), gv.bits_from_bf16(d["K"]),
            gv.bits_from_bf16(d["V"]), _queries_left_in(gv, p, ws, geom))


def _check_compress(gv, cfg, li, sel_mode="topk", layer_id=0, runner=None):
    """End to end.  The GPU draws its own samples (fp32 fit and Box-Muller), so a few query values
    land on the neighbouring bf16 step: masks are compared with the oracle's own run inside the score
    tolerance (2e-2) band, budgets to 0.5 % of N, and - the strict check - with the oracle's vote on the
    queries the GPU left in its workspace inside the 1e-3 bands.  Compaction is checked bit-exactly
    against the GPU's own mask."""
    mask, budget, b_step, Kg, Vg, Qg = (runner or _run_compress)(gv, cfg, li, sel_mode, layer_id)
    kw = pu.oracle_kwargs(cfg, layer_id)
    res, _, _ = o.compress_layer(li.h, li.W_q, li.b_q, li.K, li.V, li.cu_seqlens, sel_mode=sel_mode, **kw)
    pf = kw["p_nuc"]
    for r in range(cfg.batch):
        a, b = int(li.cu_seqlens[r]), int(li.cu_seqlens[r + 1])
        N = b - a
        gm = np.stack([gv.unpack_mask(mask[h], gv.mask_word_offset(a, r), N) for h in range(cfg.n_kv_heads)])
        Kr = o.bf16_bits_to_f64(li.K[:, a:b])
        pu.check_vote_against_oracle(res[r].Q, Kr, pf, sel_mode, False, gm, b_step[r], mass_band=2e-2, logit_band=2e-2)
        _check_mask_against_own_queries(gv, cfg, Qg[r], res[r].Q, Kr, pf, sel_mode, gm, b_step[r])
        assert np.all(np.abs(budget[r] - res[r].budget) <= max(2, 0.005 * N)), (budget[r], res[r].budget)
        Kc, Vc = o.compact(li.K[:, a:b], li.V[:, a:b], gm)
        for h in range(cfg.n_kv_heads):
            n = int(gm[h].sum())
            assert budget[r, h] == n
            assert np.array_equal(Kg[h, a:a + n], Kc[h]) and np.array_equal(Vg[h, a:a + n], Vc[h])


@pytest.mark.parametrize("idx", range(4))
def test_compress_small(gv, idx):
    cfg = _small_cfgs()[idx]
    _check_compress(gv, cfg, synth.make_layer(cfg, 0, with_bias=(idx % 2 == 1)))


@pytest.mark.parametrize("name,mode", [("c0", "topk"), ("c0", "topp"), ("c1", "topk"), ("c1", "topp"), ("c3", "topk"),
                                       ("c3", "topp")])
def test_compress_configs(gv, name, mode):
    cfg = synth.make_config(name)
    _check_compress(gv, cfg, synth.make_layer(cfg, 0), mode)


@pytest.mark.parametrize("n_heavy,p_nuc", [(4, 0.99), (12, 0.99), (40, 0.99), (40, 0.9), (120, 0.9)])
def test_compress_planted_answer(gv, n_heavy, p_nuc):
    """Inputs whose answer is known by construction (see synth.make_planted): at p = 0.99 the keep mask is
    exactly the planted positions; at p = 0.9 nothing outside them is kept.  And the oracle agrees."""
    cfg = synth.make_planted(n_heavy, p_nuc=p_nuc)
    li = synth.make_layer(cfg, 0)
    mask, budget, b_step, Kg, Vg, _ = _run_compress(gv, cfg, li)
    for kh in range(cfg.n_kv_heads):
        kept = np.nonzero(gv.unpack_mask(mask[kh], 0, cfg.total_tokens))[0]
        planted = li.heavy_positions[(0, kh)]
        assert np.isin(kept, planted).all()
        if p_nuc == 0.99:
            assert np.array_equal(kept, planted) and budget[0, kh] == n_heavy
    _check_compress(gv, cfg, li)


def _run_compress_bf16_h(gv, cfg, li, sel_mode="topk", layer_id=0):
    p = gv.params_from_config(cfg, layer_id=layer_id, h_dtype=gv.DTYPE_BF16)
    geom = _geom(cfg)
    ws = gv.alloc_workspace(p, *geom)
    d = pu.upload_layer(li, gv, torch)
    mask = torch.empty(cfg.n_kv_heads, gv.mask_row_words(cfg.total_tokens, cfg.batch), dtype=torch.int32, device="cuda")
    budget = torch.empty(cfg.batch, cfg.n_kv_heads, dtype=torch.int32, device="cuda")
    b_step = torch.empty(cfg.batch, cfg.n_q_heads, dtype=torch.int32, device="cuda")
    gv.gvote_compress(p, d["h"].bfloat16(), d["W_q"], d["b_q"], d["K"], d["V"], d["cu"], geom, mask, budget, b_step, ws)
    assert gv.gvote_poll_status(ws) == 0
    return (mask.cpu().numpy(), budget.cpu().numpy(), b_step.cpu().numpy(), gv.bits_from_bf16(d["K"]),
            gv.bits_from_bf16(d["V"]), _queries_left_in(gv, p, ws, geom))


@pytest.mark.parametrize("name", ["small2", "c1", "c3"])
def test_compress_bf16_hidden_states(gv, name):
    """The whole pass with the hidden states in bf16 (half the bytes of the fit): the oracle gets the same
    bf16 values widened to fp64."""
    cfg = _small_cfgs()[2] if name == "small2" else synth.make_config(name)
    li = synth.make_layer(cfg, 0)
    li.h = torch.from_numpy(li.h).bfloat16().float().numpy()      # the values bf16 can hold
    _check_compress(gv, cfg, li, runner=_run_compress_bf16_h)


# ----------------------------------------------------------------------------- streaming fit
def _stream_fit(gv, p, cfg, li, n_blocks, rng):
    """Feed every request's rows after the sinks in n_blocks uneven blocks; returns (mu, var) tensors."""
    cu = li.cu_seqlens
    B = cfg.batch
    state = torch.zeros(B, 3, cfg.d_h, dtype=torch.float64, device="cuda")
    cuts = []
    for r in range(B):
        a, b = int(cu[r]) + cfg.n_s, int(cu[r + 1])
        inner = np.sort(rng.integers(a, b + 1, size=n_blocks - 1))
        cuts.append(np.concatenate([[a], inner, [b]]))
    for k in range(n_blocks):
        rows = [li.h[cuts[r][k]:cuts[r][k + 1]] for r in range(B)]
        lens = [x.shape[0] for x in rows]
        if sum(lens) == 0:
            continue
        block = torch.from_numpy(np.concatenate(rows)).cuda()
        cub = torch.from_numpy(np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)).cuda()
        geom = (B, sum(lens), max(lens))
        ws = gv.alloc_workspace(p, *geom)
        gv.gvote_fit_update(p, block, cub, geom, state, ws)
    mu = torch.empty(B, cfg.d_h, device="cuda"); var = torch.empty_like(mu)
    gv.gvote_fit_finish(p, state, B, mu, var)
    return mu, var


@pytest.mark.parametrize("idx,n_blocks", [(0, 1), (1, 3), (2, 4), (3, 7)])
def test_streaming_fit_matches_one_shot_fit(gv, idx, n_blocks):
    """Moments accumulated block by block (Chan merge, fp64 state) against the oracle's one-shot fit:
    1e-5 relative on the variance, 1e-5 of the largest standard deviation on the mean."""
    cfg = _small_cfgs()[idx]
    li = synth.make_layer(cfg, 0)
    p = gv.params_from_config(cfg)
    mu, var = _stream_fit(gv, p, cfg, li, n_blocks, np.random.default_rng(50 + idx))
    for r in range(cfg.batch):
        m, v = o.fit(li.h[li.cu_seqlens[r]:li.cu_seqlens[r + 1]], cfg.n_s)
        assert np.allclose(var[r].cpu().numpy(), v, rtol=1e-5, atol=0)
        assert np.abs(mu[r].cpu().numpy() - m).max() <= 1e-5 * np.sqrt(v).max() + 1e-6 * np.abs(m).max()


def _run_compress_moments(gv, cfg, li, sel_mode="topk", layer_id=0):
    p = gv.params_from_config(cfg, layer_id=layer_id, sel_mode=gv.SEL_TOPP if sel_mode == "topp" else gv.SEL_TOPK_C0)
    geom = _geom(cfg)
    ws = gv.alloc_workspace(p, *geom)
    d = pu.upload_layer(li, gv, torch)
    mu, var = _stream_fit(gv, p, cfg, li, 3, np.random.default_rng(60))
    h_last = torch.from_numpy(np.stack([li.h[int(li.cu_seqlens[r + 1]) - 1] for r in range(cfg.batch)])).cuda()
    mask = torch.empty(cfg.n_kv_heads, gv.mask_row_words(cfg.total_tokens, cfg.batch), dtype=torch.int32, device="cuda")
    budget = torch.empty(cfg.batch, cfg.n_kv_heads, dtype=torch.int32, device="cuda")
    b_step = torch.empty(cfg.batch, cfg.n_q_heads, dtype=torch.int32, device="cuda")
    gv.gvote_compress_moments(p, mu, var, h_last, d["W_q"], d["b_q"], d["K"], d["V"], d["cu"], geom, mask, budget,
                              b_step, ws)
    assert gv.gvote_poll_status(ws) == 0
    return (mask.cpu().numpy(), budget.cpu().numpy(), b_step.cpu().numpy(), gv.bits_from_bf16(d["K"]),
            gv.bits_from_bf16(d["V"]), _queries_left_in(gv, p, ws, geom))


@pytest.mark.parametrize("name", ["small2", "c0", "c1", "c3"])
def test_compress_from_streamed_moments(gv, name):
    """The pass with the Gaussian fitted upstream, block by block, against the oracle's whole pass."""
    cfg = _small_cfgs()[2] if name == "small2" else synth.make_config(name)
    _check_compress(gv, cfg, synth.make_layer(cfg, 0, with_bias=(name == "small2")), runner=_run_compress_moments)


# ----------------------------------------------------------------------------- the pass applied again
def _pruned_cache(cfg, li, rng, n_new, empty_head=None):
    """A cache as an earlier pass and some decoding would leave it: per (request, KV head) a random
    subset of the older tokens, in order, then the n_new latest tokens; the rest of each slab holds
    rows that must be ignored (large values, so that a leak shows).  Returns slabs and the map."""
    Hkv, T = cfg.n_kv_heads, cfg.total_tokens
    K = np.full_like(li.K, 0x4700)            # bf16 32768.0 in every unused row
    V = np.full_like(li.V, 0x4700)
    kv_len = np.zeros((cfg.batch, Hkv), dtype=np.int32)
    token_pos = np.full((Hkv, T), -1, dtype=np.int32)
    kept = []
    for r in range(cfg.batch):
        a, b = int(li.cu_seqlens[r]), int(li.cu_seqlens[r + 1])
        N = b - a
        old = max(N - n_new, 0)
        per_head = []
        for h in range(Hkv):
            if empty_head == (r, h):
                idx = np.zeros(0, dtype=np.int64)
            else:
                frac = rng.uniform(0.3, 0.9)
                idx = np.sort(rng.choice(old, size=max(1, int(frac * old)), replace=False)) if old > 0 else np.zeros(0, dtype=np.int64)
                idx = np.concatenate([idx, np.arange(old, N)]).astype(np.int64)
            n = idx.shape[0]
            K[h, a:a + n] = li.K[h, a + idx]
            V[h, a:a + n] = li.V[h, a + idx]
            kv_len[r, h] = n
            token_pos[h, a:a + n] = idx
            per_head.append(idx)
        kept.append(per_head)
    return K, V, kv_len, token_pos, kept


def _check_recompress(gv, cfg, li, sel_mode="topk", n_new=5, empty_head=None, seed=70):
    rng = np.random.default_rng(seed)
    Ks, Vs, kv_len, token_pos, kept = _pruned_cache(cfg, li, rng, n_new, empty_head)
    p = gv.params_from_config(cfg, sel_mode=gv.SEL_TOPP if sel_mode == "topp" else gv.SEL_TOPK_C0)
    geom = _geom(cfg)
    ws = gv.alloc_workspace(p, *geom)
    d = pu.upload_layer(li, gv, torch)
    dK, dV = gv.bf16_from_bits(Ks), gv.bf16_from_bits(Vs)
    mu = torch.empty(cfg.batch, cfg.d_h, device="cuda"); var = torch.empty_like(mu)
    gv.gvote_fit(p, d["h"], d["cu"], geom, mu, var, ws)
    cu = li.cu_seqlens
    h_last = torch.from_numpy(np.stack([li.h[int(cu[r + 1]) - 1] for r in range(cfg.batch)])).cuda()
    # tokens seen: more than the slab holds (the slabs of a pruned cache are shorter than its history)
    seen = (np.diff(cu) + 37 * (np.arange(cfg.batch) + 1)).astype(np.int32)
    seq_len = torch.from_numpy(seen).cuda()
    d_len = torch.from_numpy(kv_len).cuda()
    d_pos = torch.from_numpy(token_pos).cuda()
    mask = torch.empty(cfg.n_kv_heads, gv.mask_row_words(cfg.total_tokens, cfg.batch), dtype=torch.int32, device="cuda")
    budget = torch.empty(cfg.batch, cfg.n_kv_heads, dtype=torch.int32, device="cuda")
    b_step = torch.empty(cfg.batch, cfg.n_q_heads, dtype=torch.int32, device="cuda")
    gv.gvote_recompress(p, mu, var, h_last, d["W_q"], d["b_q"], dK, dV, d["cu"], d_len, seq_len, d_pos, geom, mask,
                        budget, b_step, ws)
    assert gv.gvote_poll_status(ws) == 0
    mask, budget, b_step = mask.cpu().numpy(), budget.cpu().numpy(), b_step.cpu().numpy()
    Kg, Vg, pos_g = gv.bits_from_bf16(dK), gv.bits_from_bf16(dV), d_pos.cpu().numpy()
    Qg = _queries_left_in(gv, p, ws, geom)

    W = o.bf16_bits_to_f64(li.W_q)
    kw = pu.oracle_kwargs(cfg)
    n_s = kw.pop("n_s")
    G = cfg.n_q_heads // cfg.n_kv_heads
    for r in range(cfg.batch):
        a, b = int(cu[r]), int(cu[r + 1])
        N = b - a
        m64, v64 = o.fit(li.h[a:b].astype(np.float64), n_s)
        heads = [o.bf16_bits_to_f64(Ks[h, a:a + kv_len[r, h]]) for h in range(cfg.n_kv_heads)]
        res = o.recompress_request(m64, v64, li.h[b - 1].astype(np.float64), W, li.b_q, heads, int(seen[r]), request_id=r,
                                   sel_mode=sel_mode, token_pos=kept[r], **kw)
        for h in range(cfg.n_kv_heads):
            n = int(kv_len[r, h])
            row = gv.unpack_mask(mask[h], gv.mask_word_offset(a, r), N)
            assert not row[n:].any(), "a slot beyond the head's rows was kept"
            gm = row[:n]
            if n == 0:
                assert budget[r, h] == 0 and not b_step[r, h * G:(h + 1) * G].any()
                continue
            pu.check_vote_against_oracle(res.Q[h * G:(h + 1) * G], heads[h][None], kw["p_nuc"], sel_mode, False,
                                         gm[None], b_step[r, h * G:(h + 1) * G], mass_band=2e-2, logit_band=2e-2)
            # and, inside the 1e-3 bands, against the oracle's vote on the queries the GPU used (per head: a
            # head's rows are its own kv_len)
            one_head = replace(cfg, n_q_heads=G, n_kv_heads=1)
            _check_mask_against_own_queries(gv, one_head, Qg[r, h:h + 1], res.Q[h * G:(h + 1) * G], heads[h][None],
                                            kw["p_nuc"], sel_mode, gm[None], b_step[r, h * G:(h + 1) * G])
            assert abs(int(budget[r, h]) - int(res.budget[h])) <= max(2, 0.005 * n)
            keep = np.nonzero(gm)[0]
            assert budget[r, h] == keep.shape[0]
            # rows and map entries move together, bit for bit
            assert np.array_equal(Kg[h, a:a + keep.shape[0]], Ks[h, a + keep])
            assert np.array_equal(Vg[h, a:a + keep.shape[0]], Vs[h, a + keep])
            assert np.array_equal(pos_g[h, a:a + keep.shape[0]], kept[r][h][keep])


@pytest.mark.parametrize("idx,mode", [(1, "topk"), (2, "topk"), (2, "topp"), (3, "topk")])
def test_recompress_small(gv, idx, mode):
    """The pass on a pruned, grown cache (heads of different lengths, positions from the tokens seen)
    against the oracle's per-head restatement; same bands as the whole-pass checks.  Case 1 has
    d_k = 16 and so runs the kernels that stand in where the tensor-core ones do not apply."""
    cfg = _small_cfgs()[idx]
    _check_recompress(gv, cfg, synth.make_layer(cfg, 0, with_bias=(idx == 3)), mode)


@pytest.mark.parametrize("name,mode", [("c0", "topk"), ("c0", "topp"), ("c1", "topk"), ("c3", "topk")])
def test_recompress_configs(gv, name, mode):
    cfg = synth.make_config(name)
    _check_recompress(gv, cfg, synth.make_layer(cfg, 0), mode, n_new=17)


def test_recompress_head_without_rows(gv):
    cfg = _small_cfgs()[2]
    _check_recompress(gv, cfg, synth.make_layer(cfg, 0), empty_head=(1, 0), n_new=3)


def test_entry_points_refuse_bad_arguments_before_any_launch(gv):
    """Host-side validation: a missing or misaligned pointer, a workspace that is too small, a shape the
    kernels do not take: an error code comes back and nothing has been enqueued."""
    cfg = _small_cfgs()[2]
    li = synth.make_layer(cfg, 0)
    p = gv.params_from_config(cfg)
    geom = _geom(cfg)
    ws = gv.alloc_workspace(p, *geom)
    d = pu.upload_layer(li, gv, torch)
    mu = torch.zeros(cfg.batch, cfg.d_h, device="cuda"); var = torch.ones_like(mu)
    h_last = torch.zeros(cfg.batch, cfg.d_h, device="cuda")
    mask = torch.empty(cfg.n_kv_heads, gv.mask_row_words(cfg.total_tokens, cfg.batch), dtype=torch.int32, device="cuda")
    budget = torch.empty(cfg.batch, cfg.n_kv_heads, dtype=torch.int32, device="cuda")
    b_step = torch.empty(cfg.batch, cfg.n_q_heads, dtype=torch.int32, device="cuda")
    kv_len = torch.zeros(cfg.batch, cfg.n_kv_heads, dtype=torch.int32, device="cuda")
    seen = torch.ones(cfg.batch, dtype=torch.int32, device="cuda")
    launches = gv.load().gvote_launch_count()

    def status_of(fn):
        with pytest.raises(gv.GVoteError) as e:
            fn()
        return e.value.status

    # a pointer the re-application needs is missing
    assert status_of(lambda: gv.gvote_recompress(p, mu, var, h_last, d["W_q"], d["b_q"], d["K"], d["V"], d["cu"], None,
                                                 seen, None, geom, mask, budget, b_step, ws)) == -1
    # a workspace one byte short
    assert status_of(lambda: gv.gvote_compress(p, d["h"], d["W_q"], d["b_q"], d["K"], d["V"], d["cu"], geom, mask,
                                               budget, b_step, ws[:-1])) == -3
    # a misaligned output
    odd = torch.empty(cfg.batch * cfg.n_kv_heads + 1, dtype=torch.int32, device="cuda")[1:].view(cfg.batch, cfg.n_kv_heads)
    assert status_of(lambda: gv.gvote_recompress(p, mu, var, h_last, d["W_q"], d["b_q"], d["K"], d["V"], d["cu"], kv_len,
                                                 seen, None, geom, mask, odd, b_step, ws)) == -2
    # the longest request must leave two rows for the fit after the sinks
    short = (cfg.batch, cfg.total_tokens, cfg.n_s + 1)
    assert status_of(lambda: gv.gvote_fit(p, d["h"], d["cu"], short, mu, var, ws)) == -1
    assert gv.load().gvote_launch_count() == launches


def test_recompress_of_a_full_cache_is_the_plain_pass(gv):
    """kv_len = N for every head and seq_len = N: the same bits as gvote_compress_moments."""
    cfg = synth.make_config("c1")
    li = synth.make_layer(cfg, 0)
    p = gv.params_from_config(cfg)
    geom = _geom(cfg)
    ws = gv.alloc_workspace(p, *geom)
    outs = []
    for again in (False, True):
        d = pu.upload_layer(li, gv, torch)
        mu = torch.empty(cfg.batch, cfg.d_h, device="cuda"); var = torch.empty_like(mu)
        gv.gvote_fit(p, d["h"], d["cu"], geom, mu, var, ws)
        cu = li.cu_seqlens
        h_last = torch.from_numpy(np.stack([li.h[int(cu[r + 1]) - 1] for r in range(cfg.batch)])).cuda()
        mask = torch.empty(cfg.n_kv_heads, gv.mask_row_words(cfg.total_tokens, cfg.batch), dtype=torch.int32, device="cuda")
        budget = torch.empty(cfg.batch, cfg.n_kv_heads, dtype=torch.int32, device="cuda")
        b_step = torch.empty(cfg.batch, cfg.n_q_heads, dtype=torch.int32, device="cuda")
        if again:
            lens = torch.from_numpy(np.diff(cu).astype(np.int32)).cuda()
            kv_len = lens[:, None].expand(cfg.batch, cfg.n_kv_heads).contiguous()
            gv.gvote_recompress(p, mu, var, h_last, d["W_q"], d["b_q"], d["K"], d["V"], d["cu"], kv_len, lens, None,
                                geom, mask, budget, b_step, ws)
        else:
            gv.gvote_compress_moments(p, mu, var, h_last, d["W_q"], d["b_q"], d["K"], d["V"], d["cu"], geom, mask,
                                      budget, b_step, ws)
        outs.append((mask.cpu().numpy(), budget.cpu().numpy(), b_step.cpu().numpy(), gv.bits_from_bf16(d["K"])))
    for x, y in zip(*outs):
        assert np.array_equal(x, y)


def test_compress_with_an_empty_request(gv):
    """A request without cached tokens in the middle of a batch: nothing is read or written for it
    (budget 0, |C0| 0) and its neighbours are unaffected."""
    cfg = synth.make_small(8, seq_lens=(40, 0, 33), S=4, d_h=64, n_q_heads=4, n_kv_heads=2, d_k=64)
    full = synth.make_small(8, seq_lens=(40, 33), S=4, d_h=64, n_q_heads=4, n_kv_heads=2, d_k=64)
    li = synth.make_layer(full, 0)
    li.cu_seqlens = np.array([0, 40, 40, 73], dtype=np.int32)
    mask, budget, b_step, Kg, Vg, Qg = _run_compress(gv, cfg, li)
    assert budget[1].tolist() == [0, 0] and b_step[1].tolist() == [0] * 4
    W = o.bf16_bits_to_f64(li.W_q)
    kw = pu.oracle_kwargs(cfg)
    for r, (a, b) in ((0, (0, 40)), (2, (40, 73))):
        res = o.compress_request(li.h[a:b].astype(np.float64), W, li.b_q, o.bf16_bits_to_f64(li.K[:, a:b]),
                                 request_id=r, **kw)
        gm = np.stack([gv.unpack_mask(mask[h], gv.mask_word_offset(a, r), b - a) for h in range(cfg.n_kv_heads)])
        pu.check_vote_against_oracle(res.Q, o.bf16_bits_to_f64(li.K[:, a:b]), kw["p_nuc"], "topk", False, gm, b_step[r],
                                     mass_band=2e-2, logit_band=2e-2)
        _check_mask_against_own_queries(gv, cfg, Qg[r], res.Q, o.bf16_bits_to_f64(li.K[:, a:b]), kw["p_nuc"], "topk", gm,
                                        b_step[r])
        assert np.all(np.abs(budget[r] - res.budget) <= 2)
        Kc, Vc = o.compact(li.K[:, a:b], li.V[:, a:b], gm)
        for h in range(cfg.n_kv_heads):
            n = int(gm[h].sum())
            assert np.array_equal(Kg[h, a:a + n], Kc[h]) and np.array_equal(Vg[h, a:a + n], Vc[h])


def test_compress_is_deterministic(gv):
    cfg = synth.make_config("c1")
    li = synth.make_layer(cfg, 0)
    a = _run_compress(gv, cfg, li)
    b = _run_compress(gv, cfg, li)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)


def _layers_to_check(default):
    """GVOTE_PARITY_LAYERS=a,b,... or "all" widens the full-size checks beyond the default layer (each
    layer costs the oracle some tens of seconds of CPU)."""
    import os
    want = os.environ.get("GVOTE_PARITY_LAYERS", "")
    if not want:
        return [default]
    return None if want == "all" else [int(x) for x in want.split(",")]


def test_compress_full_size_c2_layer(gv):
    """A layer of the 32K workload, in the launch configuration the benchmark times."""
    cfg = synth.make_config("c2")
    layers = _layers_to_check(3)
    for layer in (range(cfg.n_layers) if layers is None else layers):
        _check_compress(gv, cfg, synth.make_layer(cfg, layer), layer_id=layer)


def test_compress_full_size_c4_layer(gv):
    """One layer of the 128K-context Qwen2.5-7B-shaped workload (N = 131072, G = 7, S = 64, p = 0.98):
    two row chunks per KV head in the score contraction, 2 MB of mask bits, 1.9 GB of hidden states."""
    cfg = synth.make_config("c4")
    layers = _layers_to_check(1)
    for layer in (range(cfg.n_layers) if layers is None else layers):
        _check_compress(gv, cfg, synth.make_layer(cfg, layer), layer_id=layer)


def _check_stages_strict(gv, cfg, li, layer_id):
    """The stages one by one on a full-size layer, every stage fed what the stage before it produced on
    the GPU and checked against the oracle's step on those same inputs, so that each is held to its own
    stated tolerance at full size: fit 1e-5; normal draws 1e-5 on z; rotated queries within one bf16
    step plus the rounding of an fp32 accumulation; the vote inside the 1e-3 bands."""
    p = gv.params_from_config(cfg, layer_id=layer_id)
    geom = _geom(cfg)
    B, S, G = cfg.batch, cfg.S, cfg.G
    ws = gv.alloc_workspace(p, *geom)
    d = pu.upload_layer(li, gv, torch)
    mu = torch.empty(B, cfg.d_h, device="cuda"); var = torch.empty_like(mu)
    gv.gvote_fit(p, d["h"], d["cu"], geom, mu, var, ws)
    Ht = torch.empty(B, S, cfg.d_h, device="cuda")
    gv.gvote_sample(p, mu, var, B, Ht)
    cu = li.cu_seqlens
    h_last = torch.from_numpy(np.stack([li.h[int(cu[r + 1]) - 1] for r in range(B)])).cuda()
    Q = torch.empty(B, cfg.n_kv_heads, G * (S + 1), cfg.d_k, dtype=torch.bfloat16, device="cuda")
    gv.gvote_project(p, Ht, h_last, d["W_q"], d["b_q"], d["cu"], B, Q, ws)
    mask = torch.full((cfg.n_kv_heads, gv.mask_row_words(cfg.total_tokens, B)), -1, dtype=torch.int32, device="cuda")
    budget = torch.empty(B, cfg.n_kv_heads, dtype=torch.int32, device="cuda")
    b_step = torch.empty(B, cfg.n_q_heads, dtype=torch.int32, device="cuda")
    gv.gvote_vote(p, Q, d["K"], d["cu"], geom, mask, budget, b_step, ws)
    assert gv.gvote_poll_status(ws) == 0
    mu_g, var_g = mu.cpu().numpy().astype(np.float64), var.cpu().numpy().astype(np.float64)
    Ht_g = Ht.cpu().numpy().astype(np.float64)
    Qg = Q.float().cpu().numpy().astype(np.float64)
    mask, budget, b_step = mask.cpu().numpy(), budget.cpu().numpy(), b_step.cpu().numpy()
    W = o.bf16_bits_to_f64(li.W_q)
    kw = pu.oracle_kwargs(cfg, layer_id)
    for r in range(B):
        a, b = int(cu[r]), int(cu[r + 1])
        N = b - a
        h64 = li.h[a:b].astype(np.float64)
        # fit
        m64, v64 = o.fit(h64, cfg.n_s)
        assert np.allclose(var_g[r], v64, rtol=1e-5, atol=0)
        assert np.abs(mu_g[r] - m64).max() <= 1e-5 * np.sqrt(v64).max() + 1e-6 * np.abs(m64).max()
        # sample, from the GPU's moments
        Ho, _ = o.sample(mu_g[r], var_g[r], S, cfg.seed, layer_id, r)
        sig = np.sqrt(var_g[r])
        assert np.abs((Ht_g[r] - Ho) / sig).max() < 1e-5 + 2e-6 * np.abs(mu_g[r] / sig).max()
        # projection and RoPE, from the GPU's samples
        Qo = o.queries_for_request(Ht_g[r], h64[-1], W, li.b_q, N, n_q_heads=cfg.n_q_heads, d_k=cfg.d_k,
                                   theta=cfg.rope_theta, n_f=cfg.n_f)
        X = o.round_to_bf16(np.concatenate([h64[-1:], Ht_g[r]]))
        mag = (np.abs(X) @ np.abs(W).T).reshape(S + 1, cfg.n_q_heads, cfg.d_k).transpose(1, 0, 2)
        mag = mag + np.concatenate([mag[..., cfg.d_k // 2:], mag[..., :cfg.d_k // 2]], axis=-1)
        Qr = pu.from_group_major(Qg[r], G)
        diff = np.abs(Qr - Qo)
        assert np.all(diff <= 2.0 ** -7 * np.abs(Qo) + 2.0 ** -21 * mag)  # one bf16 step + fp32 accumulation
        assert (diff == 0).mean() > 0.98
        # the vote, from the GPU's queries
        Kr = o.bf16_bits_to_f64(li.K[:, a:b])
        gm = np.stack([gv.unpack_mask(mask[h], gv.mask_word_offset(a, r), N) for h in range(cfg.n_kv_heads)])
        pu.check_vote_against_oracle(Qr, Kr, kw["p_nuc"], "topk", False, gm, b_step[r])      # 1e-3 bands
        om, ob, _, _, _ = o.vote(Qr, Kr, p_nuc=kw["p_nuc"])
        assert np.array_equal(budget[r], gm.sum(axis=1))
        assert np.all(np.abs(budget[r] - ob) <= max(1, 0.005 * N))
        assert (gm != om).sum() <= max(2, 0.005 * N * cfg.n_kv_heads)


@pytest.mark.parametrize("name,layer", [("c2", 3), ("c4", 1), ("c3", 0)])
def test_stages_full_size_strict_band(gv, name, layer):
    """Full-size layers of the 32K, the 128K (G = 7, four row chunks) and the ragged workloads, stage by
    stage, the vote inside the 1e-3 bands."""
    cfg = synth.make_config(name)
    _check_stages_strict(gv, cfg, synth.make_layer(cfg, layer), layer)


def test_recompress_full_size_c2_layer(gv):
    """The pass applied again at the 32K workload's shapes: heads of 10K to 30K rows each, 256 of them new."""
    cfg = synth.make_config("c2")
    _check_recompress(gv, cfg, synth.make_layer(cfg, 3), n_new=256, seed=71)


def test_compress_host_variant_matches_device_variant(gv):
    cfg = synth.make_config("c0")
    li = synth.make_layer(cfg, 0)
    mask_d, budget_d, b_step_d, Kd, Vd, _ = _run_compress(gv, cfg, li)
    p = gv.params_from_config(cfg)
    h = torch.from_numpy(li.h).pin_memory()
    W = gv.bf16_from_bits(li.W_q, "cpu", pin=True)
    K = gv.bf16_from_bits(li.K, "cpu", pin=True).clone()
    V = gv.bf16_from_bits(li.V, "cpu", pin=True).clone()
    mask = torch.empty(cfg.n_kv_heads, gv.mask_row_words(cfg.total_tokens, 1), dtype=torch.int32)
    budget = torch.empty(1, cfg.n_kv_heads, dtype=torch.int32)
    b_step = torch.empty(1, cfg.n_q_heads, dtype=torch.int32)
    for _ in range(2):
        K.copy_(gv.bf16_from_bits(li.K, "cpu")); V.copy_(gv.bf16_from_bits(li.V, "cpu"))
        gv.gvote_compress_host(p, h, W, None, K, V, torch.from_numpy(li.cu_seqlens), mask, budget, b_step)
        assert np.array_equal(mask.numpy(), mask_d) and np.array_equal(budget.numpy(), budget_d)
        assert np.array_equal(gv.bits_from_bf16(K), Kd) and np.array_equal(gv.bits_from_bf16(V), Vd)
    gv.gvote_host_arena_release()


@pytest.mark.parametrize("name", ["small2", "c1", "c3"])
def test_workspace_queries_are_the_staged_projection(gv, name):
    """gvote_workspace_queries: the rotated queries the whole pass leaves in its workspace are those of the
    staged calls (fit -> sample -> project) on the same inputs: the same draws, the same roundings.  The fused
    middle of the pass merges the fit's partial sums in one step instead of two, so a mean may differ in its
    last bit and a query entry by one bf16 step: nearly all entries are equal, none is further than a step."""
    cfg = _small_cfgs()[2] if name == "small2" else synth.make_config(name)
    li = synth.make_layer(cfg, 0)
    p = gv.params_from_config(cfg)
    geom = _geom(cfg)
    B, S, G = cfg.batch, cfg.S, cfg.n_q_heads // cfg.n_kv_heads
    d = pu.upload_layer(li, gv, torch)
    ws = gv.alloc_workspace(p, *geom)
    mask = torch.empty(cfg.n_kv_heads, gv.mask_row_words(cfg.total_tokens, B), dtype=torch.int32, device="cuda")
    budget = torch.empty(B, cfg.n_kv_heads, dtype=torch.int32, device="cuda")
    b_step = torch.empty(B, cfg.n_q_heads, dtype=torch.int32, device="cuda")
    K, V = d["K"].clone(), d["V"].clone()
    gv.gvote_compress(p, d["h"], d["W_q"], d["b_q"], K, V, d["cu"], geom, mask, budget, b_step, ws)
    Q_pass = gv.workspace_queries(p, ws, *geom).float().cpu().numpy()
    ws2 = gv.alloc_workspace(p, *geom)
    mu = torch.empty(B, cfg.d_h, device="cuda"); var = torch.empty_like(mu)
    gv.gvote_fit(p, d["h"], d["cu"], geom, mu, var, ws2)
    Ht = torch.empty(B, S, cfg.d_h, device="cuda")
    gv.gvote_sample(p, mu, var, B, Ht)
    cu = li.cu_seqlens
    h_last = torch.from_numpy(np.stack([li.h[int(cu[r + 1]) - 1] for r in range(B)])).cuda()
    Q = torch.empty(B, cfg.n_kv_heads, G * (S + 1), cfg.d_k, dtype=torch.bfloat16, device="cuda")
    gv.gvote_project(p, Ht, h_last, d["W_q"], d["b_q"], d["cu"], B, Q, ws2)
    assert gv.gvote_poll_status(ws) == 0 and gv.gvote_poll_status(ws2) == 0
    Q_staged = Q.float().cpu().numpy()
    assert Q_pass.shape == Q_staged.shape
    assert (Q_pass == Q_staged).mean() > 0.99
    assert np.all(np.abs(Q_pass - Q_staged) <= 2.0 ** -7 * np.abs(Q_staged) + 1e-30)
    # the current-query rows do not depend on the fit at all: bit for bit
    cur = slice(G * S, G * (S + 1))
    assert np.array_equal(Q_pass[:, :, cur], Q_staged[:, :, cur])


def test_compress_takes_the_exact_route_when_the_sample_misleads(gv):
    """The whole pass with keys built against the queries it will use (they do not depend on K: a first run
    leaves them in the workspace): the logits of exactly the sampled tiles are shifted, so the brackets miss,
    the head is selected again by the exact route, the pruning step's mask scan must not merge the discarded
    tentative mask, and the result is still the oracle's vote on those queries, compacted bit for bit."""
    N, d_k, S = 16384, 64, 6
    cfg = synth.make_small(13, seq_lens=(N,), S=S, d_h=64, n_q_heads=2, n_kv_heads=1, d_k=d_k, p_nuc=0.9)
    li = synth.make_layer(cfg, 0)
    p = gv.params_from_config(cfg)
    geom = _geom(cfg)
    d = pu.upload_layer(li, gv, torch)
    mask = torch.empty(1, gv.mask_row_words(N, 1), dtype=torch.int32, device="cuda")
    budget = torch.empty(1, 1, dtype=torch.int32, device="cuda")
    b_step = torch.empty(1, 2, dtype=torch.int32, device="cuda")
    ws = gv.alloc_workspace(p, *geom)
    gv.gvote_compress(p, d["h"], d["W_q"], d["b_q"], d["K"].clone(), d["V"].clone(), d["cu"], geom, mask, budget, b_step, ws)
    Qg = _queries_left_in(gv, p, ws, geom)                 # [1, 1, G (S+1), d_k]
    e = Qg[0, 0].mean(axis=0)
    e /= np.linalg.norm(e)
    rng = np.random.default_rng(7)
    v = rng.normal(size=N)
    n_tiles = N // 128
    want = min(max(n_tiles >> 3, 32), 128)               # the sampling plan of the kernels (vote_geom.cuh)
    stride = n_tiles // want
    for j in range(want):
        t = j * stride + (((j * 2654435761) & 0xFFFFFFFF) >> 15) % stride
        v[t * 128:(t + 1) * 128] -= 6.0
    Kbits = synth.f32_to_bf16_bits((v[:, None] * e[None, :] * math.sqrt(d_k)).astype(np.float32)[None])
    Kd, Vd = gv.bf16_from_bits(Kbits), d["V"].clone()
    ws2 = gv.alloc_workspace(p, *geom)
    gv.gvote_compress(p, d["h"], d["W_q"], d["b_q"], Kd, Vd, d["cu"], geom, mask, budget, b_step, ws2)
    assert gv.gvote_poll_status(ws2) == 0
    assert gv.gvote_exact_heads(ws2) == 1
    assert np.array_equal(_queries_left_in(gv, p, ws2, geom), Qg)
    G = cfg.n_q_heads // cfg.n_kv_heads
    Qr = pu.from_group_major(Qg[0], G)
    Kr = o.bf16_bits_to_f64(Kbits)
    gm = np.stack([gv.unpack_mask(mask.cpu().numpy()[0], 0, N)])
    pu.check_vote_against_oracle(Qr, Kr, float(np.float32(cfg.p_nuc)), "topk", False, gm, b_step.cpu().numpy()[0])
    n = int(gm[0].sum())
    assert int(budget[0, 0]) == n
    Kc, Vc = o.compact(Kbits, li.V, gm)
    assert np.array_equal(gv.bits_from_bf16(Kd)[0, :n], Kc[0]) and np.array_equal(gv.bits_from_bf16(Vd)[0, :n], Vc[0])


@pytest.mark.parametrize("name", ["small2", "c1"])
def test_compress_with_the_current_query_set_in_the_union(gv, name):
    """include_c0 inside the whole pass: the current query's own top-p set is written into the keep mask by
    the top-p kernel, the synthetic rows' union reaches it through the tentative mask and the pruning step's
    scan: both must survive."""
    cfg = _small_cfgs()[2] if name == "small2" else synth.make_config(name)
    li = synth.make_layer(cfg, 0)
    p = gv.params_from_config(cfg, include_c0=True)
    geom = _geom(cfg)
    ws = gv.alloc_workspace(p, *geom)
    d = pu.upload_layer(li, gv, torch)
    mask = torch.empty(cfg.n_kv_heads, gv.mask_row_words(cfg.total_tokens, cfg.batch), dtype=torch.int32, device="cuda")
    budget = torch.empty(cfg.batch, cfg.n_kv_heads, dtype=torch.int32, device="cuda")
    b_step = torch.empty(cfg.batch, cfg.n_q_heads, dtype=torch.int32, device="cuda")
    gv.gvote_compress(p, d["h"], d["W_q"], d["b_q"], d["K"], d["V"], d["cu"], geom, mask, budget, b_step, ws)
    assert gv.gvote_poll_status(ws) == 0
    Qg = _queries_left_in(gv, p, ws, geom)
    mask, budget, b_step = mask.cpu().numpy(), budget.cpu().numpy(), b_step.cpu().numpy()
    Kg, Vg = gv.bits_from_bf16(d["K"]), gv.bits_from_bf16(d["V"])
    G = cfg.n_q_heads // cfg.n_kv_heads
    pf = float(np.float32(cfg.p_nuc))
    for r in range(cfg.batch):
        a, b = int(li.cu_seqlens[r]), int(li.cu_seqlens[r + 1])
        N = b - a
        gm = np.stack([gv.unpack_mask(mask[h], gv.mask_word_offset(a, r), N) for h in range(cfg.n_kv_heads)])
        Kr = o.bf16_bits_to_f64(li.K[:, a:b])
        Qr = pu.from_group_major(Qg[r], G)
        pu.check_vote_against_oracle(Qr, Kr, pf, "topk", True, gm, b_step[r])          # 1e-3 bands, C0 in the union
        om, ob, _, _, _ = o.vote(Qr, Kr, p_nuc=pf, include_c0=True)
        assert np.all(np.abs(budget[r] - ob) <= max(2, 0.005 * N))
        without, _, _, _, _ = o.vote(Qr, Kr, p_nuc=pf, include_c0=False)
        assert (om & ~without).any(), "the case does not exercise include_c0"
        Kc, Vc = o.compact(li.K[:, a:b], li.V[:, a:b], gm)
        for h in range(cfg.n_kv_heads):
            n = int(gm[h].sum())
            assert budget[r, h] == n
            assert np.array_equal(Kg[h, a:a + n], Kc[h]) and np.array_equal(Vg[h, a:a + n], Vc[h])
