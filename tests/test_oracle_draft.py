"""Pins of the draft-stage oracle (Section "Overview": the small model beam-samples W_S beams per
step; Section "Details": each is a sample of q_beam = T o (q / Q) over current beams x V).

The joint and its warping are recomputed here with numpy/scipy, independently of the oracle's C
code; the draws are pinned through their CDF intervals, by a chi-square test of the Philox
stream against that joint, and by special cases."""
import numpy as np
from scipy import stats
from scipy.special import logsumexp, softmax

import oracle


def _joint(z, s, tau, top_k=0, top_p=1.0):
    """q_beam over beams x V by definition: exp(S_a) softmax(z_a / tau), normalised, warped."""
    logq = s[:, None] + (z / tau - logsumexp(z / tau, axis=1, keepdims=True))
    w = np.exp(logq - logsumexp(logq)).ravel()
    if top_k:
        order = np.lexsort((np.arange(w.size), -w))
        keep = order[:top_k]
        if 0.0 < top_p < 1.0:
            wk = w[keep] / w[keep].sum()
            n = int(np.searchsorted(np.cumsum(wk), top_p - 1e-15) + 1)
            keep = keep[:n]
        out = np.zeros_like(w)
        out[keep] = w[keep]
        w = out / out.sum()
    return w


def _problem(rng, beams_per_req, V):
    rbo = np.concatenate([[0], np.cumsum(beams_per_req)]).astype(np.int32)
    n = int(rbo[-1])
    z = rng.normal(0, 2, size=(n, V)).astype(np.float32)
    s = rng.normal(0, 1, size=n)
    return rbo, z, s


def test_draws_fall_in_their_cdf_interval_of_the_joint():
    rng = np.random.default_rng(0)
    rbo, z, s = _problem(rng, [3, 1, 4], 50)
    for top_k, top_p in [(0, 1.0), (10, 1.0), (10, 0.8), (1, 1.0)]:
        prm = dict(V=50, temperature=0.7, seed=5, step=2, top_k=top_k, top_p=top_p)
        u = rng.uniform(size=(3, 6))
        res = oracle.draft_layer(rbo, prm, 2, 6, z, s, inject_u=u)
        assert not res["error"].any()
        for r in range(3):
            w = _joint(z[rbo[r]:rbo[r + 1]].astype(np.float64), s[rbo[r]:rbo[r + 1]], 0.7, top_k, top_p)
            cdf = np.concatenate([[0.0], np.cumsum(w)])
            for k in range(6):
                slot = res["out_off"][r] + k
                cell = (res["out_parent"][slot] - rbo[r]) * 50 + res["out_token"][slot]
                assert w[cell] > 0
                assert cdf[cell] - 1e-12 <= u[r, k] <= cdf[cell + 1] + 1e-12
                a, tok = res["out_parent"][slot], res["out_token"][slot]
                lq = s[a] + float(z[a, tok]) / 0.7 - logsumexp(z[a].astype(np.float64) / 0.7)
                assert abs(res["out_logq"][slot] - lq) < 1e-9


def test_philox_draws_follow_the_joint_chi_square():
    rng = np.random.default_rng(1)
    rbo, z, s = _problem(rng, [3], 8)
    w = _joint(z.astype(np.float64), s, 1.3)
    counts = np.zeros(24)
    W = 50
    for step in range(2000):
        res = oracle.draft_layer(rbo, dict(V=8, temperature=1.3, seed=11, step=step), 1, W, z, s)
        np.add.at(counts, res["out_parent"] * 8 + res["out_token"], 1)
    n = counts.sum()
    assert n == 2000 * W
    keep = w * n >= 5
    chi2 = ((counts[keep] - w[keep] * n) ** 2 / (w[keep] * n)).sum() + \
        ((counts[~keep].sum() - w[~keep].sum() * n) ** 2 / max(w[~keep].sum() * n, 1e-300) if (~keep).any() else 0.0)
    dof = keep.sum() - (0 if (~keep).any() else 1)
    assert chi2 < stats.chi2.ppf(0.999, dof), (chi2, dof)


def test_stream_is_keyed_by_request_layer_and_index():
    rng = np.random.default_rng(2)
    rbo, z, s = _problem(rng, [2, 2], 30)
    prm = dict(V=30, seed=3, step=9)
    res = oracle.draft_layer(rbo, prm, 4, 5, z, s)
    for r in range(2):
        w = _joint(z[rbo[r]:rbo[r + 1]].astype(np.float64), s[rbo[r]:rbo[r + 1]], 1.0)
        cdf = np.concatenate([[0.0], np.cumsum(w)])
        for k in range(5):
            u = oracle.uniform(3, 9, r, (1 << 29) + 4, 3, k)
            slot = res["out_off"][r] + k
            cell = (res["out_parent"][slot] - rbo[r]) * 30 + res["out_token"][slot]
            assert cdf[cell] - 1e-12 <= u <= cdf[cell + 1] + 1e-12


def test_special_cases():
    rng = np.random.default_rng(3)
    rbo, z, s = _problem(rng, [1, 3], 40)
    # top_k = 1: always the most probable cell of the joint
    res = oracle.draft_layer(rbo, dict(V=40, seed=1, top_k=1), 1, 4, z, s)
    for r in range(2):
        w = _joint(z[rbo[r]:rbo[r + 1]].astype(np.float64), s[rbo[r]:rbo[r + 1]], 1.0)
        for k in range(4):
            slot = res["out_off"][r] + k
            assert (res["out_parent"][slot] - rbo[r]) * 40 + res["out_token"][slot] == np.argmax(w)
    # one beam: the joint is the next-token softmax; the beam score only shifts the new score
    u = rng.uniform(size=(2, 3))
    res = oracle.draft_layer(rbo, dict(V=40, temperature=2.0, seed=1), 1, 3, z, s, inject_u=u)
    p = softmax(z[0].astype(np.float64) / 2.0)
    cdf = np.concatenate([[0.0], np.cumsum(p)])
    for k in range(3):
        tok = res["out_token"][k]
        assert res["out_parent"][k] == 0 and cdf[tok] - 1e-12 <= u[0, k] <= cdf[tok + 1] + 1e-12
        assert abs(res["out_logq"][k] - (s[0] + np.log(p[tok]))) < 1e-9
    # a slot range that cannot hold W_S draws is an error of that request only
    res = oracle.draft_layer(rbo, dict(V=40, seed=1), 1, 3, z, s, out_off=[0, 2, 5])
    assert list(res["error"]) == [3, 0]          # 3: capacity
