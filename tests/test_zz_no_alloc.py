"""The allocation-free fit entry point against the ordinary one.

`gvote_fit_static` is for integrations that cannot obtain device memory at the point of the call
(inside an allocator callback, or once a serving process has frozen its memory pool): it takes no
workspace and keeps its partial sums in a fixed array that ships inside the library.  This file
is collected last on purpose, so a run that stops at the first failure has already been through
every other test."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gv():
    from paper_2509_03136_b200 import build as gbuild
    gbuild.build()
    from paper_2509_03136_b200 import gvote
    gvote.load()
    return gvote


def _case(gv, lens, d_h, n_s, seed):
    rng = np.random.default_rng(seed)
    T = sum(lens)
    h = (rng.normal(size=(T, d_h)) * rng.uniform(0.3, 3, size=d_h) + rng.normal(size=d_h) * 5).astype(np.float32)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    p = gv.make_params(d_h=d_h, n_q_heads=2, n_kv_heads=1, d_k=16, rope_theta=1e4, S=2, p_nuc=0.9, n_f=4, n_s=n_s,
                       seed=0)
    return p, torch.from_numpy(h).cuda(), torch.from_numpy(cu).cuda(), (len(lens), T, max(lens))


@pytest.mark.parametrize("lens,d_h,n_s", [((40,), 64, 2), ((33, 64, 17), 72, 4), ((5000, 700), 1024, 4),
                                          ((20000,), 4096, 4)])
def test_static_fit_matches_workspace_fit_twice_in_a_row(gv, lens, d_h, n_s):
    """Two consecutive calls (the shared array still holds the first call's partials during the
    second) must both agree with gvote_fit to the tolerance of the fit parity test: 1e-5 relative
    on the variance, 1e-5 of the largest standard deviation on the mean."""
    p, h, cu, geom = _case(gv, lens, d_h, n_s, seed=21)
    batch, _, max_N = geom
    ws = gv.alloc_workspace(p, *geom)
    mu_ref = torch.empty(batch, d_h, device="cuda"); var_ref = torch.empty_like(mu_ref)
    gv.gvote_fit(p, h, cu, geom, mu_ref, var_ref, ws)
    torch.cuda.synchronize()
    for call in range(2):
        if call == 1:                       # different data through the same array in between
            p2, h2, cu2, geom2 = _case(gv, (777,), d_h, 0, seed=22)
            m2 = torch.empty(1, d_h, device="cuda"); v2 = torch.empty_like(m2)
            gv.gvote_fit_static(p2, h2, cu2, 1, 777, m2, v2)
        mu = torch.full((batch, d_h), float("nan"), device="cuda"); var = torch.full_like(mu, float("nan"))
        gv.gvote_fit_static(p, h, cu, batch, max_N, mu, var)
        torch.cuda.synchronize()
        v, vr = var.cpu().numpy(), var_ref.cpu().numpy()
        m, mr = mu.cpu().numpy(), mu_ref.cpu().numpy()
        assert np.allclose(v, vr, rtol=1e-5, atol=0)
        assert np.abs(m - mr).max() <= 1e-5 * np.sqrt(vr).max() + 1e-6 * np.abs(mr).max()


def test_static_fit_rejects_sizes_beyond_its_array(gv):
    d_h = 4096
    batch = gv.FIT_STATIC_MAX_ENTRIES // d_h + 1
    lens = (8,) * batch
    p, h, cu, geom = _case(gv, lens, d_h, 0, seed=23)
    mu = torch.empty(batch, d_h, device="cuda"); var = torch.empty_like(mu)
    with pytest.raises(gv.GVoteError) as e:
        gv.gvote_fit_static(p, h, cu, batch, 8, mu, var)
    assert e.value.status == -4 and "unsupported shape" in str(e.value)
