"""Pins of the width rule: the alpha chain, the residual identities of the proof, the
acceptance-count recursion and its thresholding."""
import itertools

import numpy as np
import pytest

import oracle


def _rand_pair(rng, n, sharp=1.0):
    p = rng.dirichlet(np.full(n, sharp))
    q = rng.dirichlet(np.full(n, sharp))
    return p, q


def test_alpha_chain_matches_definition_and_closed_form():
    rng = np.random.default_rng(0)
    for trial in range(20):
        n, m = int(rng.integers(3, 40)), int(rng.integers(1, 7))
        p, q = _rand_pair(rng, n, sharp=0.5)
        alpha = oracle.alpha_chain(p, q, m)
        # definition: alpha_j = sum q min(p_j/q, 1), p_{k+1} = norm(max(p_k - q, 0))
        pk = p.copy()
        # closed form: p_j = max(p - s_{j-1} q, 0)/c_j, c_{j+1} = F(s_j), alpha_j = 1 - c_{j+1}/c_j
        F = lambda s: np.maximum(p - s * q, 0).sum()
        s, c = 0.0, 1.0
        for j in range(m):
            assert abs(pk.sum() - 1) < 1e-12
            a_def = float((q * np.minimum(pk / q, 1)).sum())
            s_next = s + c
            c_next = F(s_next)
            assert abs(alpha[j] - a_def) < 1e-12
            assert abs(alpha[j] - (1 - c_next / c)) < 1e-10
            assert np.abs(pk - np.maximum(p - s * q, 0) / c).max() < 1e-10
            # identity of the proof: P_{1,j} + P_{2,j} = p_j with p_{j+1} the normalised residual
            res = np.maximum(pk - q, 0)
            if res.sum() <= 1e-300:
                break
            nxt = res / res.sum()
            assert np.abs(np.minimum(pk, q) + (1 - a_def) * nxt - pk).max() < 1e-12
            pk, s, c = nxt, s_next, c_next


def test_alpha_special_cases():
    rng = np.random.default_rng(1)
    p, _ = _rand_pair(rng, 16)
    assert np.allclose(oracle.alpha_chain(p, p, 4), 1.0)            # p == q: always accepted
    q = np.zeros(16); q[:8] = p[8:] / p[8:].sum()
    p2 = p.copy(); p2[:8] = 0; p2 /= p2.sum()
    assert np.allclose(oracle.alpha_chain(p2, q, 4), 0.0)           # disjoint supports


def test_dp_rows_sum_to_one_and_boundaries():
    rng = np.random.default_rng(2)
    for m in range(0, 9):
        alpha = rng.uniform(0, 1, size=m)
        wt, P, G = oracle.width_dp(alpha, 0.7)
        assert P[0, 0] == 1.0
        for n in range(m + 1):
            assert abs(P[n, :n + 1].sum() - 1) < 1e-12
            assert np.all(P[n, n + 1:] == 0)
            assert abs(P[n, 0] - np.prod(1 - alpha[:n])) < 1e-14
        assert G[0] == 1.0 and np.all(np.diff(G[:m + 1]) <= 1e-15)
        assert wt == max(K for K in range(m + 1) if G[K] >= 0.7)


def test_dp_against_brute_force_over_outcomes():
    """P(m, k) by summing over all accept/reject strings: after an accept the chain restarts at
    alpha_1, after j-1 rejections in a row the next draft is accepted with alpha_j."""
    rng = np.random.default_rng(3)
    for m in range(1, 8):
        alpha = rng.uniform(0.05, 0.95, size=m)
        _, P, _ = oracle.width_dp(alpha, 0.5)
        pk = np.zeros(m + 1)
        for bits in itertools.product([0, 1], repeat=m):
            pr, run = 1.0, 0
            for b in bits:
                a = alpha[run]
                pr *= a if b else (1 - a)
                run = 0 if b else run + 1
            pk[sum(bits)] += pr
        assert np.abs(pk - P[m, :]).max() < 1e-12


def test_dp_against_monte_carlo_of_the_accept_chain():
    """The alphas of a concrete (p, q) pair drive a simulated accept/reject chain with iid
    drafts from q; the histogram of accepted counts matches P(m, .)."""
    rng = np.random.default_rng(4)
    n, m, trials = 12, 5, 200000
    p, q = _rand_pair(rng, n, sharp=0.8)
    alpha = oracle.alpha_chain(p, q, m)
    _, P, _ = oracle.width_dp(alpha, 0.5)
    # residual distributions p_1..p_m, computed from the definition
    pj = [p]
    for _ in range(m - 1):
        r = np.maximum(pj[-1] - q, 0)
        pj.append(r / r.sum())
    ratio = np.stack([np.minimum(1, x / q) for x in pj])          # [m, n]
    drafts = rng.choice(n, size=(trials, m), p=q)
    u = rng.uniform(size=(trials, m))
    run = np.zeros(trials, int)
    count = np.zeros(trials, int)
    for i in range(m):
        acc = u[:, i] <= ratio[run, drafts[:, i]]
        count += acc
        run = np.where(acc, 0, run + 1)
    hist = np.bincount(count, minlength=m + 1) / trials
    assert np.abs(hist - P[m]).max() < 4e-3


def test_threshold_rule_special_cases():
    assert oracle.width_dp(np.ones(5), 0.7)[0] == 5        # p == q: W~ = m
    assert oracle.width_dp(np.zeros(5), 0.7)[0] == 0       # disjoint: W~ = 0
    assert oracle.width_dp(np.array([]), 0.7)[0] == 0      # no drafts
    a = np.array([0.6, 0.3, 0.2, 0.1])
    _, P, G = oracle.width_dp(a, 0.0)
    for thresh in (0.05, 0.3, 0.7, 0.95, 1.0):
        wt = oracle.width_dp(a, thresh)[0]
        assert G[wt] >= thresh and (wt == len(a) or G[wt + 1] < thresh)


@pytest.mark.parametrize("seed", [0, 1])
def test_select_width_matches_chain_plus_dp(seed):
    rng = np.random.default_rng(seed)
    V, nA, m = 50, 3, 4
    forest = dict(R=1, B=nA, N=nA, max_depth=1, req_beam_off=[0, nA],
                  beam_node_off=np.arange(nA + 1), parent=[-1] * nA, token=[0] * nA)
    zp = rng.normal(0, 2, size=(nA, V)).astype(np.float32)
    zq = (zp + rng.normal(0, 1, size=(nA, V))).astype(np.float32)
    sp, sq = rng.normal(0, 1, nA), rng.normal(0, 1, nA)
    tau = 0.8
    prm = dict(V=V, temperature=tau, thresh=0.6, W_min=1, W_max=8, W_nom=1)
    width, alpha, tail = oracle.select_width(forest, prm, zp, zq, sp, sq, [0, nA], np.arange(nA), [m])
    sm = lambda z: np.exp(z / tau - (z / tau).max(1, keepdims=True)) / \
        np.exp(z / tau - (z / tau).max(1, keepdims=True)).sum(1, keepdims=True)
    pb = (np.exp(sp) / np.exp(sp).sum())[:, None] * sm(zp.astype(np.float64))
    qb = (np.exp(sq) / np.exp(sq).sum())[:, None] * sm(zq.astype(np.float64))
    a = oracle.alpha_chain(pb, qb, m)
    assert np.abs(a - alpha[0]).max() < 1e-12
    wt, _, G = oracle.width_dp(a, 0.6)
    assert width[0] == min(8, max(1, wt)) and np.abs(G[:m + 1] - tail[0, :m + 1]).max() < 1e-12
