"""Theorem 1 end to end: 10^6 seeded trials of the paper's process on the toy model.

Each trial draws a draft forest the way the small model would (beam sampling of width
W_S = 3 for gamma = 2 steps from q_beam, numpy generator), then runs the oracle's verification
step on it with its own Philox stream (request id = trial number).  The ordered tuple of
layer-1 output beams must follow the product of p_beam^(1) (chi-square over all cells), and,
given the beams that layer 1 kept, the layer-2 output tuple must follow the product of
p_beam^(2) over those beams.  Seeds are fixed, so the test is deterministic.
"""
import numpy as np
from scipy import stats

import oracle
from toy_model import BEAMS, V, ToyModel

TRIALS = 1_000_000
CHUNK = 100_000
W_S = 3
GAMMA = 2
PARAMS = dict(V=V, thresh=0.6, W_min=1, W_max=2, W_nom=2, seed=2024, step=5)


def _draw(rng, probs, k):
    """k iid draws per row from the rows of probs [R, C] (or one shared row [C])."""
    cdf = np.cumsum(probs, axis=-1)
    cdf = cdf / cdf[..., -1:]
    R = probs.shape[0] if probs.ndim == 2 else None
    u = rng.uniform(size=(len(cdf) if R else k, k) if R else k)
    if R:
        return (u[:, :, None] > cdf[:, None, :]).sum(-1)
    return np.searchsorted(cdf, u)


def _make_chunk(model, rng, R, first_req):
    qb1 = model.beam_dist("q", [(0,), (1,)]).ravel()
    c1 = np.searchsorted(np.cumsum(qb1) / qb1.sum(), rng.uniform(size=(R, W_S)))
    i1, v1 = c1 // V, c1 % V                                            # [R,3]
    logq0, logq1 = model.logq(0), model.logq(1)
    sq = model.root_logq[i1] + logq0[i1, v1]                            # [R,3]
    joint = np.exp(sq[:, :, None] + logq1[i1, v1])                      # [R,3,V]
    c2 = _draw(rng, joint.reshape(R, W_S * V), W_S)                      # [R,3]
    j2, v2 = c2 // V, c2 % V
    # old node ids: 0,1 roots; 2..4 layer-1 drafts; 5..7 layer-2 drafts
    tree = np.concatenate([np.tile([0, 1], (R, 1)), i1, np.take_along_axis(i1, j2, 1)], axis=1)
    depth = np.tile([0, 0, 1, 1, 1, 2, 2, 2], (R, 1))
    rank = np.tile([0, 0, 0, 1, 2, 0, 1, 2], (R, 1))
    par_old = np.concatenate([np.full((R, 2), -1), i1, 2 + j2], axis=1)
    tok_old = np.concatenate([np.zeros((R, 2), int), v1, v2], axis=1)
    order = np.argsort(tree * 100 + depth * 10 + rank, axis=1, kind="stable")   # new -> old
    pos = np.argsort(order, axis=1)                                              # old -> new
    rows = np.arange(R)[:, None]
    base = (np.arange(R) * 8)[:, None]
    par_new_of_old = np.where(par_old >= 0, np.take_along_axis(pos, np.maximum(par_old, 0), 1) + base, -1)
    parent = np.take_along_axis(par_new_of_old, order, 1)
    token = np.take_along_axis(tok_old, order, 1)
    drank = np.take_along_axis(rank, order, 1)
    # logits rows of every node from the context tables
    pv1 = np.take_along_axis(v1, j2, 1)
    pi1 = np.take_along_axis(i1, j2, 1)
    z = {}
    for name, tabs in (("p", model.zp), ("q", model.zq)):
        old = np.concatenate([np.broadcast_to(tabs[0], (R, 2, V)), tabs[1][i1, v1],
                              tabs[2][pi1, pv1, v2]], axis=1)                     # [R,8,V]
        z[name] = np.take_along_axis(old, order[:, :, None], 1).reshape(R * 8, V)
    n0 = (tree == 0).sum(1)
    beam_node_off = np.stack([base[:, 0], base[:, 0] + n0], 1).ravel()
    forest = dict(R=R, B=2 * R, N=8 * R, max_depth=GAMMA,
                  req_beam_off=np.arange(R + 1) * 2,
                  beam_node_off=np.concatenate([beam_node_off, [8 * R]]),
                  parent=parent.ravel(), token=token.ravel(), draft_rank=drank.ravel())
    # contexts of the new nodes, for decoding the outputs: (beam, tok1) of depth-1 nodes
    ctx1_old = i1 * V + v1                                                       # [R,3]
    ctx_of_new = np.full((R, 8), -1)
    np.put_along_axis(ctx_of_new, pos[:, 2:5], ctx1_old, 1)
    prm = dict(PARAMS, req_id=np.arange(first_req, first_req + R))
    res = oracle.verify_step(forest, prm, z["p"], z["q"], np.tile(model.root_logp, R),
                             np.tile(model.root_logq, R), trace=False, threads=8)
    assert not res["error"].any()
    depth_new = np.take_along_axis(depth, order, 1)
    return forest, res, ctx_of_new, depth_new, drank, rows


def _ordered_accepts(status, depth_new, drank, layer, W):
    """new-node ids (local 0..7) of the accepted depth-`layer` nodes in draw order, [R, W]."""
    acc = (status == oracle.NODE_ACCEPTED) & (depth_new == layer)
    key = np.where(acc, drank, 99)
    return np.argsort(key, axis=1, kind="stable")[:, :W]


def _chisq(counts, expect):
    """Pearson chi-square with cells of expectation < 5 merged into one."""
    counts, expect = counts.ravel().astype(float), expect.ravel()
    small = expect < 5
    if small.any():
        counts = np.concatenate([counts[~small], [counts[small].sum()]])
        expect = np.concatenate([expect[~small], [expect[small].sum()]])
    keep = expect > 0
    stat = ((counts[keep] - expect[keep]) ** 2 / expect[keep]).sum()
    return stats.chi2.sf(stat, keep.sum() - 1)


def test_output_law_chi_square():
    model = ToyModel(seed=4)
    rng = np.random.default_rng(77)
    C = BEAMS * V
    o1_all, l_last_all, o2_all, w2_all = [], [], [], []
    for k in range(TRIALS // CHUNK):
        forest, res, ctx_of_new, depth_new, drank, rows = _make_chunk(model, rng, CHUNK, k * CHUNK)
        R = CHUNK
        W1 = int(res["layer_width"][0, 0])
        assert np.all(res["layer_width"][:, 0] == W1)
        status = res["node_status"].reshape(R, 8)
        s0 = res["out_off"][:-1]
        short1 = res["l_last"] == 1
        # layer-1 outputs as cells beam*V + token
        out_cells = np.stack([(res["out_root_beam"][s0 + j] - 2 * np.arange(R)) * V +
                              res["out_token"][s0 + j] for j in range(W1)], 1)
        acc1 = _ordered_accepts(status, depth_new, drank, 1, W1)
        acc_cells = np.take_along_axis(ctx_of_new, acc1, 1)
        o1 = np.where(short1[:, None], out_cells, acc_cells)
        o1_all.append(o1)
        l_last_all.append(res["l_last"].copy())
        # layer-2 outputs as (position of the parent in the ordered layer-1 tuple, token)
        W2 = res["layer_width"][:, 1]
        o2 = np.full((R, 2), -1)
        short2 = res["l_last"] == 2
        acc2 = _ordered_accepts(status, depth_new, drank, 2, 2)
        par_local = forest["parent"].reshape(R, 8) - (np.arange(R) * 8)[:, None]
        tok = forest["token"].reshape(R, 8)
        for j in range(2):
            pn_out = res["out_parent"][s0 + j] - np.arange(R) * 8
            pn_acc = np.take_along_axis(par_local, acc2[:, j:j + 1], 1)[:, 0]
            pn = np.where(short2, pn_out, pn_acc)
            tk = np.where(short2, res["out_token"][s0 + j],
                          np.take_along_axis(tok, acc2[:, j:j + 1], 1)[:, 0])
            which = (pn[:, None] == acc1).argmax(1)        # position in the layer-1 tuple
            o2[:, j] = np.where(j < W2, which * V + tk, -1)
        o2_all.append(o2)
        w2_all.append(W2)
    o1 = np.concatenate(o1_all)
    l_last = np.concatenate(l_last_all)
    o2 = np.concatenate(o2_all)
    w2 = np.concatenate(w2_all)
    W1 = o1.shape[1]

    # layer 1: ordered tuple ~ prod p_beam^(1)
    pb1 = model.beam_dist("p", [(0,), (1,)]).ravel()
    flat = np.ravel_multi_index(tuple(o1.T), (C,) * W1)
    counts = np.bincount(flat, minlength=C ** W1)
    expect = pb1
    for _ in range(W1 - 1):
        expect = np.multiply.outer(expect, pb1)
    assert _chisq(counts, expect * TRIALS) > 1e-3

    # layer 2, given the ordered tuple of beams that layer 1 kept (trials that went on)
    went_on = l_last >= 2
    keys, cnt = np.unique(flat[went_on], return_counts=True)
    tested = 0
    for key in keys[np.argsort(-cnt)]:
        cells = np.unravel_index(key, (C,) * W1)
        if len(set(cells)) < W1:
            continue                                   # skip duplicate beams
        sel = went_on & (flat == key)
        ctxs = [(int(c) // V, int(c) % V) for c in cells]
        pb2 = model.beam_dist("p", ctxs).ravel()
        # the layer-2 width also depends on how many drafts survived the pruning (m enters
        # the acceptance-count recursion), never on their values: condition on it as well
        W2 = int(np.bincount(w2[sel]).argmax())
        sel = sel & (w2 == W2)
        f2 = np.ravel_multi_index(tuple(o2[sel][:, :W2].T), (W1 * V,) * W2)
        c2 = np.bincount(f2, minlength=(W1 * V) ** W2)
        e2 = pb2
        for _ in range(W2 - 1):
            e2 = np.multiply.outer(e2, pb2)
        assert _chisq(c2, e2 * sel.sum()) > 1e-3
        tested += 1
        if tested == 4:
            break
    assert tested == 4
