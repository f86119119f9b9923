"""Theorem 1 by exact enumeration: the ordered tuple of output beams of a verified layer is
distributed as independent draws from the large model's beam-sampling distribution (Eq. 1).

Every ordered tuple of W_S = 3 drafts (each one of 2 beams x 8 tokens, drawn iid from the
small model's q_beam) is enumerated with its probability; for each tuple the oracle's accept
decisions are explored branch by branch by injecting uniforms on either side of the ratio
the oracle reports, and its sample draws enter through the mass vectors it reports.  The
resulting law must equal the product of p_beam, which this file states from Eq. 1 itself.
A wrong ratio direction, a wrong residual, a wrong reset after an accept or a wrong live set
all break the equality by many orders of magnitude more than the tolerance.
"""
import itertools

import numpy as np
import pytest

import oracle
from toy_model import BEAMS, V, ToyModel, build_forest, concat_forests

STRIDE = 16


def _depths(parent):
    d = np.zeros(len(parent), np.int32)
    for n, p in enumerate(parent):
        d[n] = 0 if p < 0 else d[p] + 1
    return d


def _layer_law(model, layer_lists, probs, fixed_prefix, target, params, gamma):
    """Exact law of the ordered output tuple of draft layer `target`.

    layer_lists[i]: the draft layers of enumeration item i; probs[i]: its probability;
    fixed_prefix: injected uniforms that pin the decisions of the layers before `target`."""
    built = [build_forest(model, layers, gamma) for layers in layer_lists]
    states = [(i, list(fixed_prefix), probs[i]) for i in range(len(built))]
    law = None
    width = None
    while states:
        items = [(built[i][0], built[i][1], built[i][2]) for i, _, _ in states]
        forest, zp, zq = concat_forests(items)
        R = len(states)
        inj = np.full((R, STRIDE), 0.5)
        for r, (_, pre, _) in enumerate(states):
            inj[r, :len(pre)] = pre
        prm = dict(params, V=V)
        res = oracle.verify_step(forest, prm, zp, zq,
                                 np.tile(model.root_logp, R), np.tile(model.root_logq, R),
                                 inject_u=inj, trace=True, dist=True)
        assert not res["error"].any()
        depth = _depths(forest["parent"])
        starts = np.searchsorted(res["trace_req"], np.arange(R + 1))
        # lengths of the dumped mass vectors, in trace order
        is_sample = np.isin(res["trace_kind"], (oracle.TR_RESIDUAL, oracle.TR_FILL, oracle.TR_EXTRA))
        nA = np.where(res["trace_layer"] == 1, BEAMS,
                      res["layer_width"][res["trace_req"], np.maximum(res["trace_layer"] - 2, 0)])
        dlen = np.where(is_sample, nA * V, 0)
        doff = np.concatenate([[0], np.cumsum(dlen)])
        nxt = []
        for r, (i, pre, prob) in enumerate(states):
            lo, hi = starts[r], starts[r + 1]
            recs = [t for t in range(lo, hi) if res["trace_kind"][t] not in (oracle.TR_WIDTH, oracle.TR_WARP)]
            k = len(pre)
            if (k < len(recs) and res["trace_kind"][recs[k]] == oracle.TR_ACCEPT
                    and res["trace_layer"][recs[k]] == target):
                ratio = res["trace_a"][recs[k]]
                assert 0.0 <= ratio <= 1.0
                if ratio > 0.0:
                    nxt.append((i, pre + [ratio / 2], prob * ratio))
                if ratio < 1.0:
                    nxt.append((i, pre + [(1 + ratio) / 2], prob * (1 - ratio)))
                continue
            # leaf: every accept decision of the target layer is fixed
            W = int(res["layer_width"][r, target - 1])
            if width is None:
                width = W
                law = np.zeros((BEAMS * V,) * W)
            assert W == width  # the width depends on p and q only, never on the drafts
            n0 = forest["beam_node_off"][forest["req_beam_off"][r]]
            n1 = forest["beam_node_off"][forest["req_beam_off"][r + 1]]
            ids = np.arange(n0, n1)
            if target == 1:
                A = ids[depth[ids] == 0]
            else:
                A = ids[(depth[ids] == target - 1) & (res["node_status"][ids] == oracle.NODE_ACCEPTED)]
            assert len(A) == BEAMS
            acc = ids[(depth[ids] == target) & (res["node_status"][ids] == oracle.NODE_ACCEPTED)]
            acc = acc[np.argsort(forest["draft_rank"][acc])]
            factors = []
            for n in acc:
                e = np.zeros(BEAMS * V)
                e[int(np.where(A == forest["parent"][n])[0][0]) * V + forest["token"][n]] = 1.0
                factors.append(e)
            if res["l_last"][r] == target:
                samples = [t for t in recs if res["trace_layer"][t] == target
                           and res["trace_kind"][t] in (oracle.TR_RESIDUAL, oracle.TR_FILL)]
                assert len(acc) + len(samples) == W
                for t in samples:
                    factors.append(res["dist"][doff[t]:doff[t] + BEAMS * V])
                # the outputs the oracle reports must be the accepted drafts, in order
                s0 = res["out_off"][r]
                for j, n in enumerate(acc):
                    assert res["out_node"][s0 + j] == n and res["out_source"][s0 + j] == oracle.SRC_DRAFT
            else:
                assert res["l_last"][r] > target and len(acc) == W
            contrib = np.array(prob)
            for fct in factors:
                contrib = np.multiply.outer(contrib, fct)
            law += contrib
        states = nxt
    return law, width


def _warp_ref(w, top_k, top_p):
    """The warping by its definition, written independently of the oracle: keep the top_k most
    probable cells, renormalise; keep the shortest most-probable prefix whose mass reaches
    top_p, renormalise.  Ties towards the lower cell index."""
    w = np.asarray(w, dtype=np.float64).ravel()
    order = np.lexsort((np.arange(w.size), -w))
    keep = order[:top_k] if top_k else order
    probs = w[keep] / w[keep].sum()
    if top_p < 1.0:
        n = int(np.searchsorted(np.cumsum(probs), top_p - 1e-15)) + 1
        keep = keep[:n]
    out = np.zeros_like(w)
    out[keep] = w[keep] / w[keep].sum()
    return out


def _product_law(pb, W):
    out = np.array(1.0)
    for _ in range(W):
        out = np.multiply.outer(out, pb.ravel())
    return out


@pytest.mark.parametrize("params", [
    dict(W_min=2, W_max=2, W_nom=2, thresh=0.7),          # fixed width 2, W_S = 3
    dict(W_min=1, W_max=3, W_nom=2, thresh=0.5),          # dynamic width
    dict(W_min=3, W_max=3, W_nom=2, thresh=0.7),          # width 3 with 3 drafts
])
def test_first_layer_law_equals_beam_sampling(params):
    model = ToyModel(seed=1)
    qb = model.beam_dist("q", [(0,), (1,)]).ravel()
    pb = model.beam_dist("p", [(0,), (1,)])
    tuples = list(itertools.product(range(BEAMS * V), repeat=3))
    layer_lists = [[[(c // V, c % V) for c in t]] for t in tuples]
    probs = [float(np.prod(qb[list(t)])) for t in tuples]
    assert abs(sum(probs) - 1) < 1e-12
    law, W = _layer_law(model, layer_lists, probs, [], 1, params, gamma=1)
    assert abs(law.sum() - 1) < 1e-10
    assert np.abs(law - _product_law(pb, W)).max() < 1e-12


@pytest.mark.parametrize("top_k,top_p", [(5, 1.0), (0, 0.7), (6, 0.8), (1, 1.0)])
def test_first_layer_law_with_warped_joints(top_k, top_p):
    """With the warping T on both joints (drafts drawn from T o q_beam) the outputs follow the
    product of T o p_beam."""
    model = ToyModel(seed=5)
    qb = _warp_ref(model.beam_dist("q", [(0,), (1,)]), top_k, top_p)
    pb = _warp_ref(model.beam_dist("p", [(0,), (1,)]), top_k, top_p)
    assert (pb > 0).sum() <= (top_k or 99) and abs(pb.sum() - 1) < 1e-12
    assert np.abs(oracle.warp(model.beam_dist("p", [(0,), (1,)]), top_k, top_p).ravel() - pb).max() < 1e-15
    support = np.nonzero(qb)[0]
    tuples = list(itertools.product(support, repeat=3))
    layer_lists = [[[(int(c) // V, int(c) % V) for c in t]] for t in tuples]
    probs = [float(np.prod(qb[list(t)])) for t in tuples]
    assert abs(sum(probs) - 1) < 1e-12
    params = dict(W_min=2, W_max=2, W_nom=2, thresh=0.7, top_k=top_k, top_p=top_p)
    law, W = _layer_law(model, layer_lists, probs, [], 1, params, gamma=1)
    assert abs(law.sum() - 1) < 1e-10
    assert np.abs(law - _product_law(pb, W)).max() < 1e-12


def test_inverted_ratio_would_fail():
    """Sanity of the pin itself: the law of the FIRST output under the inverted acceptance
    ratio min(1, q/p') (as the running text prints it) is far from p_beam, so the test above
    can tell the two readings apart.  Computed here by hand for one draft."""
    model = ToyModel(seed=1)
    qb = model.beam_dist("q", [(0,), (1,)]).ravel()
    pb = model.beam_dist("p", [(0,), (1,)]).ravel()
    acc = qb * np.minimum(1.0, qb / pb)                 # inverted rule, one draft
    res = np.maximum(pb - qb, 0)
    law = acc + (1 - acc.sum()) * res / res.sum()
    assert np.abs(law - pb).max() > 1e-2
    acc = qb * np.minimum(1.0, pb / qb)                 # the rule the proof uses
    law = acc + (1 - acc.sum()) * res / res.sum()
    assert np.abs(law - pb).max() < 1e-14


@pytest.mark.parametrize("case", ["two_accepted", "one_rejected_child_pruned"])
def test_second_layer_law_equals_beam_sampling(case):
    model = ToyModel(seed=2)
    if case == "two_accepted":
        layer1 = [(0, 3), (1, 5)]
        prefix = [1e-12, 1e-12]                       # both accepted
        live_parents = [0, 1]
        pruned = []
        params = dict(W_min=2, W_max=2, W_nom=2, thresh=0.7)
    else:
        # find a middle draft whose ratio is < 1 so that a large uniform rejects it
        pb1 = model.beam_dist("p", [(0,), (1,)]).ravel()
        qb1 = model.beam_dist("q", [(0,), (1,)]).ravel()
        cand = int(np.argmin(pb1 / qb1))
        assert pb1[cand] / qb1[cand] < 0.9
        best = int(np.argmax(pb1 / qb1))                # survives the residual update
        layer1 = [(0, 2), (cand // V, cand % V), (best // V, best % V)]
        prefix = [1e-12, 1 - 1e-12, 1e-12]            # accept, reject, accept
        live_parents = [0, 2]
        pruned = [(1, 4)]                             # a draft under the rejected beam
        params = dict(W_min=2, W_max=2, W_nom=2, thresh=0.7)
    # the layer-2 drafts are iid from q_beam over (accepted layer-1 beams) x V
    live_ctx = [(layer1[j][0], layer1[j][1]) for j in live_parents]
    qb = model.beam_dist("q", live_ctx).ravel()
    cells = list(range(len(live_parents) * V))
    tuples = list(itertools.product(cells, repeat=3))
    layer_lists, probs = [], []
    for t in tuples:
        drafts = [(live_parents[c // V], c % V) for c in t]
        layer_lists.append([layer1, drafts[:1] + pruned + drafts[1:]])
        probs.append(float(np.prod(qb[list(t)])))
    law, W = _layer_law(model, layer_lists, probs, prefix, 2, params, gamma=2)
    assert W == 2 and abs(law.sum() - 1) < 1e-10
    # cells of the law follow the live set in ascending node id; build_forest stores the
    # nodes of a tree in draw order, trees in beam order
    order = sorted(range(len(live_parents)),
                   key=lambda j: (layer1[live_parents[j]][0], live_parents[j]))
    pb = model.beam_dist("p", [live_ctx[j] for j in order])
    assert np.abs(law - _product_law(pb, W)).max() < 1e-12


def _warped_case(seed, top_k, top_p, need=3):
    """A toy model and three layer-1 drafts inside the common support of the two warped joints:
    the two with the largest ratio (accepted by tiny injected uniforms) and the one with the
    smallest (cut once the width of 2 is reached, so its children are pruned)."""
    model = ToyModel(seed=seed)
    pb1 = _warp_ref(model.beam_dist("p", [(0,), (1,)]), top_k, top_p)
    qb1 = _warp_ref(model.beam_dist("q", [(0,), (1,)]), top_k, top_p)
    both = np.nonzero((pb1 > 0) & (qb1 > 0))[0]
    order = both[np.argsort(-(pb1[both] / qb1[both]))]
    cells = [int(order[0]), int(order[1]), int(order[-1])][:need]
    assert len(set(cells)) == need
    return model, [(c // V, c % V) for c in cells]


def _second_layer_law(model, layer1, params, drafter_beams, live=(0, 1)):
    """Exact law of the ordered layer-2 outputs when every layer-2 draft is an iid draw from the
    warped q joint over the layer-1 drafts `drafter_beams` (x V) and layer 1 accepted the drafts
    `live`; also returns the product of the warped p joint over the accepted beams."""
    top_k, top_p = params.get("top_k", 0), params.get("top_p", 1.0)
    ctx = [(layer1[j][0], layer1[j][1]) for j in drafter_beams]
    qd = _warp_ref(model.beam_dist("q", ctx), top_k, top_p)
    support = np.nonzero(qd)[0]
    layer_lists, probs = [], []
    for t in itertools.product(support, repeat=3):
        layer_lists.append([layer1, [(drafter_beams[int(c) // V], int(c) % V) for c in t]])
        probs.append(float(np.prod(qd[list(t)])))
    assert abs(sum(probs) - 1) < 1e-12
    law, W = _layer_law(model, layer_lists, probs, [1e-12, 1e-12], 2, params, gamma=2)
    live_ctx = [(layer1[j][0], layer1[j][1]) for j in live]
    order = sorted(range(len(live)), key=lambda j: (layer1[live[j]][0], live[j]))
    pb = _warp_ref(model.beam_dist("p", [live_ctx[j] for j in order]), top_k, top_p)
    assert abs(law.sum() - 1) < 1e-10
    return law, _product_law(pb.reshape(len(live), V), W)


@pytest.mark.parametrize("seed,top_k,top_p", [(2, 6, 0.9), (5, 6, 0.8), (7, 4, 1.0), (2, 0, 0.7)])
def test_second_layer_law_with_warped_joints(seed, top_k, top_p):
    """Layer 2 with the warping T (Section "Details": p_beam = T o (p/P), q_beam = T o (q/Q) at
    every layer): when the live drafts are iid draws from the q_beam the verification itself
    uses -- T applied to the joint over the ACCEPTED layer-1 beams -- the outputs follow the
    product of T o p_beam^(2) exactly.  This pins the accept / residual arithmetic with warped
    joints beyond the first layer."""
    model, layer1 = _warped_case(seed, top_k or 16, top_p)
    params = dict(W_min=2, W_max=2, W_nom=2, thresh=0.7, top_k=top_k, top_p=top_p)
    law, expected = _second_layer_law(model, layer1, params, drafter_beams=[0, 1])
    assert np.abs(law - expected).max() < 1e-12


def test_warping_does_not_commute_with_pruning():
    """The small model drafts layer 2 from T applied to the joint over ALL its layer-1 beams;
    the verification prunes the children of rejected beams and applies T to the joint over the
    accepted beams only.  Without warping the two agree (a restriction of the joint is the
    joint of the restriction) and the outputs are exact.  With warping they do not: the top-k
    cells of the large joint, restricted, are not the top-k cells of the restricted joint, so
    the live drafts are not draws from the verification's q_beam and the output law misses the
    product of T o p_beam^(2).  The size of the miss on this toy problem is recorded here so
    that a change of reading shows up."""
    model, layer1 = _warped_case(2, 16, 1.0)
    unwarped = dict(W_min=2, W_max=2, W_nom=2, thresh=0.7)
    law, expected = _second_layer_law(model, layer1, unwarped, drafter_beams=[0, 1, 2])
    assert np.abs(law - expected).max() < 1e-12
    worst = 0.0
    for seed, top_k, top_p in [(2, 6, 0.9), (5, 6, 0.8), (7, 4, 1.0)]:
        model, layer1 = _warped_case(seed, top_k, top_p)
        params = dict(unwarped, top_k=top_k, top_p=top_p)
        law, expected = _second_layer_law(model, layer1, params, drafter_beams=[0, 1, 2])
        tv = 0.5 * np.abs(law - expected).sum()
        assert 1e-3 < tv < 0.5
        worst = max(worst, tv)
    assert worst > 0.05            # total variation 0.10 .. 0.19 on these three cases


@pytest.mark.parametrize("top_k,top_p", [(0, 1.0), (5, 0.9)])
def test_extra_layer_draws_follow_the_warped_joint(top_k, top_p):
    """All drafts of the only layer accepted: the extra layer's W_nom beams are draws from
    T o p_beam over (accepted beams x V), each realised by inverse CDF over that vector."""
    model, layer1 = _warped_case(3, top_k or 16, top_p, need=2)
    forest, zp, zq, _, _ = build_forest(model, [layer1], gamma=1)
    prm = dict(V=V, W_min=2, W_max=2, W_nom=3, thresh=0.7, top_k=top_k, top_p=top_p)
    base = oracle.verify_step(forest, prm, zp, zq, model.root_logp, model.root_logq,
                              inject_u=[[1e-12, 1e-12] + [0.5] * 6], dist=True)
    assert base["l_last"][0] == 2 and base["out_width"][0] == 3
    assert np.all(base["out_source"][:3] == oracle.SRC_EXTRA)
    # accepted beams in node order, with the p joint of Eq. 1 over them
    acc = np.nonzero((base["node_status"] == oracle.NODE_ACCEPTED) & (forest["parent"] >= 0))[0]
    ctxs = []
    for n in acc:
        tree = int(np.searchsorted(forest["beam_node_off"], n, side="right") - 1)
        ctxs.append((tree, int(forest["token"][n])))
    pb = _warp_ref(model.beam_dist("p", ctxs), top_k, top_p)
    extra = np.nonzero(base["trace_kind"] == oracle.TR_EXTRA)[0]
    assert len(extra) == 3
    for k in range(3):
        w = base["dist"][k * len(acc) * V:(k + 1) * len(acc) * V]
        assert np.abs(w - pb).max() < 1e-14
    cdf = np.concatenate([[0], np.cumsum(pb)])
    for cell in np.nonzero(pb)[0]:
        u = (cdf[cell] + cdf[cell + 1]) / 2
        res = oracle.verify_step(forest, prm, zp, zq, model.root_logp, model.root_logq,
                                 inject_u=[[1e-12, 1e-12, u, 0.5, 0.5] + [0.5] * 3])
        assert res["out_parent"][0] == acc[cell // V] and res["out_token"][0] == cell % V


def test_sampler_realises_the_reported_mass_vector():
    """Inverse-CDF draws: a uniform in the middle of cell i's CDF interval yields cell i, and
    the interval the oracle reports is the cumulative sum of the vector it reports."""
    model = ToyModel(seed=3)
    forest, zp, zq, _, _ = build_forest(model, [[(0, 1)]], gamma=1)
    prm = dict(V=V, W_min=2, W_max=2, W_nom=2, thresh=0.7)
    base = oracle.verify_step(forest, prm, zp, zq, model.root_logp, model.root_logq,
                              inject_u=[[1 - 1e-12] + [0.5] * 7], dist=True)
    assert base["l_last"][0] == 1 and base["out_source"][0] == oracle.SRC_RESIDUAL
    w = base["dist"][:BEAMS * V]
    cdf = np.concatenate([[0], np.cumsum(w)])
    pb = model.beam_dist("p", [(0,), (1,)]).ravel()
    qb = model.beam_dist("q", [(0,), (1,)]).ravel()
    assert np.abs(w - np.maximum(pb - qb, 0) / np.maximum(pb - qb, 0).sum()).max() < 1e-14
    for cell in range(BEAMS * V):
        if w[cell] <= 0:
            continue
        u = (cdf[cell] + cdf[cell + 1]) / 2
        res = oracle.verify_step(forest, prm, zp, zq, model.root_logp, model.root_logq,
                                 inject_u=[[1 - 1e-12, u] + [0.5] * 6])
        assert res["out_parent"][0] * V + res["out_token"][0] == \
            (0 if cell < V else forest["beam_node_off"][1]) * V + cell % V
        t = np.where(res["trace_kind"] == oracle.TR_RESIDUAL)[0][0]
        assert abs(res["trace_a"][t] - cdf[cell]) < 1e-14
        assert abs(res["trace_b"][t] - cdf[cell + 1]) < 1e-14
