"""Reductions of the verification rule to known algorithms and the worked trace of Fig. 1."""
import numpy as np

import oracle


def _chain_forest(W, gamma, rng, V, zq, tau=1.0):
    """W chains of depth gamma; node order: tree-major, root first. Tokens drawn from q."""
    n_tree = gamma + 1
    N = W * n_tree
    parent = np.full(N, -1, np.int32)
    for n in range(N):
        if n % n_tree:
            parent[n] = n - 1
    token = np.zeros(N, np.int32)
    for n in range(N):
        if parent[n] >= 0:
            z = zq[parent[n]].astype(np.float64) / tau
            pr = np.exp(z - z.max()); pr /= pr.sum()
            token[n] = rng.choice(V, p=pr)
    return dict(R=1, B=W, N=N, max_depth=gamma, req_beam_off=[0, W],
                beam_node_off=np.arange(W + 1) * n_tree, parent=parent, token=token)


def _softmax(z, tau):
    z = z.astype(np.float64) / tau
    e = np.exp(z - z.max())
    return e / e.sum()


def test_width_one_is_vanilla_speculative_decoding():
    """One beam, one chain, widths fixed to 1: token t is kept with probability
    min(1, p(x_t)/q(x_t)); at the first rejection one token comes from norm(max(p - q, 0));
    if all gamma drafts pass, a bonus token comes from p  (Section 2.2).  The reference below
    is that textbook loop driven by the same uniforms."""
    V, gamma, tau = 40, 5, 0.9
    for seed in range(30):
        rng = np.random.default_rng(seed)
        N = gamma + 1
        zp = rng.normal(0, 2, size=(N, V)).astype(np.float32)
        zq = (zp + rng.normal(0, 1.0, size=(N, V))).astype(np.float32)
        forest = _chain_forest(1, gamma, rng, V, zq, tau)
        prm = dict(V=V, temperature=tau, thresh=0.7, W_min=1, W_max=1, W_nom=1, seed=seed, step=3)
        res = oracle.verify_step(forest, prm, zp, zq, [0.0], [0.0])
        # textbook speculative decoding
        kept, final = [], None
        for t in range(1, gamma + 1):
            p, q = _softmax(zp[t - 1], tau), _softmax(zq[t - 1], tau)
            x = forest["token"][t]
            u = oracle.uniform(seed, 3, 0, t, 0, 0)
            if u <= min(1.0, p[x] / q[x]):
                kept.append(x)
                continue
            r = np.maximum(p - q, 0)
            cdf = np.cumsum(r / r.sum())
            final = (t, int(np.searchsorted(cdf, oracle.uniform(seed, 3, 0, t, 1, 0))), 1)
            break
        if final is None:
            cdf = np.cumsum(_softmax(zp[gamma], tau))
            final = (gamma + 1, int(np.searchsorted(cdf, oracle.uniform(seed, 3, 0, gamma + 1, 3, 0))), 3)
        assert res["l_last"][0] == final[0]
        assert res["out_width"][0] == 1
        assert res["out_token"][0] == final[1] and res["out_source"][0] == final[2]
        assert res["out_parent"][0] == final[0] - 1
        acc = [n for n in range(1, N) if res["node_status"][n] == oracle.NODE_ACCEPTED]
        assert acc == list(range(1, len(kept) + 1))


def test_equal_models_accept_everything():
    """p == q: every ratio is 1, alpha_1 = 1, so the width is the number of drafts and all
    gamma layers pass; the outputs come from the extra layer."""
    V, gamma, W = 30, 4, 3
    rng = np.random.default_rng(5)
    N = W * (gamma + 1)
    z = rng.normal(0, 2, size=(N, V)).astype(np.float32)
    forest = _chain_forest(W, gamma, rng, V, z)
    prm = dict(V=V, thresh=0.7, W_min=1, W_max=W, W_nom=W, seed=1)
    s = rng.normal(0, 1, W)
    res = oracle.verify_step(forest, prm, z, z, s, s)
    assert res["l_last"][0] == gamma + 1 and res["out_width"][0] == W
    assert np.all(res["node_status"] == oracle.NODE_ACCEPTED)
    assert np.all(res["layer_width"][0] == W)
    assert np.all(res["out_source"][:W] == oracle.SRC_EXTRA)
    acc = res["trace_kind"] == oracle.TR_ACCEPT
    assert np.allclose(res["trace_a"][acc], 1.0)


def test_figure_1_trace():
    """Fig. 1: W_L = 2, W_S = 3.  Layer 1: 'who are' and 'why do' accepted, 'why is' rejected.
    Layer 2: the child of 'why is' is rejected outright, 'who are they' accepted, 'who are it'
    rejected, then one beam is drawn from the residual.  Uniforms are injected."""
    V = 6
    ARE, IS, DO, THEY, IT, YOU = 0, 1, 2, 3, 4, 5
    # nodes: tree 'who': 0 root, 1 'are', 2 'they', 3 'it'; tree 'why': 4 root, 5 'is', 6 'do', 7 'it'
    parent = np.array([-1, 0, 1, 1, -1, 4, 4, 5], np.int32)
    token = np.array([0, ARE, THEY, IT, 0, IS, DO, IT], np.int32)
    rank = np.array([0, 0, 1, 2, 0, 1, 2, 0], np.int32)      # draw order inside each layer
    forest = dict(R=1, B=2, N=8, max_depth=2, req_beam_off=[0, 2], beam_node_off=[0, 4, 8],
                  parent=parent, token=token, draft_rank=rank)
    zp = np.zeros((8, V), np.float32)
    zq = np.zeros((8, V), np.float32)
    zq[4, IS] = 3.0           # the small model overrates 'why is' -> ratio < 1
    zq[1, IT] = 3.0           # and 'who are it'
    zp[1, YOU] = 2.0
    inj = [[1e-9, 1 - 1e-9, 1e-9,      # layer 1: are (accept), is (reject), do (accept)
            1e-9, 1 - 1e-9,            # layer 2: they (accept), it (reject); 'why is it' untested
            0.2]]                      # residual draw
    prm = dict(V=V, thresh=0.7, W_min=2, W_max=2, W_nom=2)
    res = oracle.verify_step(forest, prm, zp, zq, [0.0, 0.0], [0.0, 0.0], inject_u=inj)
    st = res["node_status"]
    assert [st[1], st[5], st[6]] == [oracle.NODE_ACCEPTED, oracle.NODE_REJECTED, oracle.NODE_ACCEPTED]
    assert st[7] == oracle.NODE_PRUNED
    assert [st[2], st[3]] == [oracle.NODE_ACCEPTED, oracle.NODE_REJECTED]
    assert res["l_last"][0] == 2 and res["out_width"][0] == 2
    assert list(res["out_source"][:2]) == [oracle.SRC_DRAFT, oracle.SRC_RESIDUAL]
    assert res["out_node"][0] == 2 and res["out_token"][0] == THEY
    # the residual beam extends an accepted layer-1 beam; with these logits it is 'who are you'
    assert res["out_parent"][1] == 1 and res["out_token"][1] == YOU
    assert list(res["out_root_beam"][:2]) == [0, 0]
    # accept tests in draw order: 3 in layer 1, 2 in layer 2
    acc = res["trace_kind"] == oracle.TR_ACCEPT
    assert list(res["trace_layer"][acc]) == [1, 1, 1, 2, 2]


def test_draw_order_not_node_order_decides_who_is_tested_first():
    """With draft_rank given, the accept loop walks the drafts in draw order even when the
    tree-major node numbering disagrees."""
    V = 4
    parent = np.array([-1, 0, -1, 2], np.int32)
    token = np.array([0, 1, 0, 2], np.int32)
    zp = np.zeros((4, V), np.float32)
    zq = np.zeros((4, V), np.float32)
    prm = dict(V=V, thresh=0.7, W_min=1, W_max=1, W_nom=1)
    out = []
    for rank in ([0, 1, 0, 0], [0, 0, 0, 1]):
        forest = dict(R=1, B=2, N=4, max_depth=1, req_beam_off=[0, 2], beam_node_off=[0, 2, 4],
                      parent=parent, token=token, draft_rank=np.array(rank, np.int32))
        res = oracle.verify_step(forest, prm, zp, zq, [0.0, 0.0], [0.0, 0.0], inject_u=[[0.5] * 4])
        out.append([int(res["node_status"][1]), int(res["node_status"][3])])
    assert out[0] == [oracle.NODE_CUT, oracle.NODE_ACCEPTED]
    assert out[1] == [oracle.NODE_ACCEPTED, oracle.NODE_CUT]


def test_scores_accumulate_log_probs():
    V, gamma, tau = 20, 3, 0.7
    rng = np.random.default_rng(9)
    N = 2 * (gamma + 1)
    zp = rng.normal(0, 2, size=(N, V)).astype(np.float32)
    zq = rng.normal(0, 2, size=(N, V)).astype(np.float32)
    forest = _chain_forest(2, gamma, rng, V, zq, tau)
    rp, rq = np.array([-0.3, -1.2]), np.array([-0.5, -0.9])
    res = oracle.verify_step(forest, dict(V=V, temperature=tau, W_min=2, W_max=2, W_nom=2),
                             zp, zq, rp, rq)
    for n in range(N):
        path = []
        a = n
        while forest["parent"][a] >= 0:
            path.append(a)
            a = forest["parent"][a]
        b = a // (gamma + 1)
        sp = rp[b] + sum(np.log(_softmax(zp[forest["parent"][k]], tau)[forest["token"][k]]) for k in path)
        sq = rq[b] + sum(np.log(_softmax(zq[forest["parent"][k]], tau)[forest["token"][k]]) for k in path)
        assert abs(res["node_logp"][n] - sp) < 1e-10 and abs(res["node_logq"][n] - sq) < 1e-10
    for s in range(res["out_width"][0]):
        par, tok = res["out_parent"][s], res["out_token"][s]
        assert abs(res["out_logp"][s] - (res["node_logp"][par] + np.log(_softmax(zp[par], tau)[tok]))) < 1e-10
