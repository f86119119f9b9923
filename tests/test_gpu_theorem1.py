"""Theorem 1 on the GPU path itself, without the oracle: drafts drawn by dsbd_draft_layer and
verified by dsbd_verify_step must leave W_L layer-1 beams that are iid samples of the LARGE
model's beam-sampling distribution p_beam, whatever the small model is.  40 000 independent
requests (each with its own Philox stream) share one toy problem -- 2 input beams with unequal
scores, V = 8, W_S = 3 drafts, W_L = 2 -- and the ordered pair of layer-1 beams is tested
against p_beam x p_beam with a chi-square test at the 0.001 level."""
import numpy as np
import pytest
import torch
from scipy import stats
from scipy.special import softmax

import paper_2409_16560_b200 as dsbd

pytestmark = pytest.mark.gpu

V, W_S, W_L = 8, 3, 2


def _run(R, seed, sigma_n, top_k=0, top_p=1.0):
    rng = np.random.default_rng(seed)
    zp = rng.normal(0, 1.5, size=(2, V)).astype(np.float32)
    zq = (zp + rng.normal(0, sigma_n, size=(2, V))).astype(np.float32)
    sp = np.array([-1.0, -1.7], np.float32)
    sq = np.array([-1.3, -1.1], np.float32)
    i32 = lambda a: torch.as_tensor(np.ascontiguousarray(a, dtype=np.int32)).cuda()
    f32 = lambda a: torch.as_tensor(np.ascontiguousarray(a, dtype=np.float32)).cuda()
    # ---- draft stage: W_S draws per request from q_beam over (2 beams x V)
    rbo = (2 * np.arange(R + 1)).astype(np.int32)
    off = (W_S * np.arange(R + 1)).astype(np.int32)
    d = dsbd.draft_layer(i32(rbo), rbo, dict(V=V, seed=seed, step=3, top_k=top_k, top_p=top_p), 1, W_S, f32(np.tile(zq, (R, 1))),
                         f32(np.tile(sq, R)), i32(off), W_S * R)
    torch.cuda.synchronize()
    assert int(d["status"].item()) == 0
    dpar = d["out_parent"].cpu().numpy().reshape(R, W_S) - 2 * np.arange(R)[:, None]     # 0 / 1: which root
    dtok = d["out_token"].cpu().numpy().reshape(R, W_S)
    # ---- forest: per request [root0, its drafts in draw order, root1, its drafts]
    N = 5 * R
    parent = np.full((R, 5), -1, np.int64)
    token = np.zeros((R, 5), np.int64)
    rank = np.zeros((R, 5), np.int64)
    is_root1 = np.zeros((R, 5), bool)
    n0 = (dpar == 0).sum(1)                                  # drafts under root 0
    base = 5 * np.arange(R)
    bno = np.zeros(2 * R + 1, np.int64)
    bno[1::2] = base + 1 + n0
    bno[2::2] = base + 5
    for r_sel, c in ((dpar == 0), 0), ((dpar == 1), 1):
        pos_in_tree = np.cumsum(r_sel, axis=1) - 1           # position among the drafts of that root
        for k in range(W_S):
            rows = np.nonzero(r_sel[:, k])[0]
            local = (1 + pos_in_tree[rows, k]) if c == 0 else (1 + n0[rows] + 1 + pos_in_tree[rows, k])
            parent[rows, local] = base[rows] + (0 if c == 0 else 1 + n0[rows])
            token[rows, local] = dtok[rows, k]
            rank[rows, local] = k
    is_root1[np.arange(R), 1 + n0] = True
    forest = dict(R=R, B=2 * R, N=N, max_depth=1, req_beam_off=rbo, beam_node_off=bno.astype(np.int32),
                  parent=parent.reshape(-1).astype(np.int32), token=token.reshape(-1).astype(np.int32),
                  draft_rank=rank.reshape(-1).astype(np.int32))
    # ---- logits rows: the two root rows; draft rows only feed the extra layer (any values)
    lp = rng.normal(0, 1, size=(R, 5, V)).astype(np.float32)
    lq = rng.normal(0, 1, size=(R, 5, V)).astype(np.float32)
    lp[:, 0], lq[:, 0] = zp[0], zq[0]
    lp[is_root1], lq[is_root1] = zp[1], zq[1]
    prm = dict(V=V, thresh=0.5, W_min=W_L, W_max=W_L, W_nom=W_L, seed=seed + 1, step=0, top_k=top_k, top_p=top_p)
    f = dsbd.Forest(forest, "cuda")
    out = dsbd.alloc_verify_out(f, dsbd.default_out_off(forest, prm), "cuda")
    st = dsbd.verify_step(f, prm, f32(lp.reshape(N, V)), f32(lq.reshape(N, V)), f32(np.tile(sp, R)),
                          f32(np.tile(sq, R)), out)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    res = {k: v.cpu().numpy() for k, v in out.items()}
    # ---- the W_L layer-1 beams of every request, as cells (root, token)
    cells = np.zeros((R, W_L), np.int64)
    oo = np.asarray(dsbd.default_out_off(forest, prm))
    status = res["node_status"].reshape(R, 5)
    for r in range(R):
        if res["l_last"][r] == 1:                            # short layer: its completed beams
            s = oo[r]
            assert res["out_width"][r] == W_L
            roots = (res["out_parent"][s:s + W_L] - 5 * r != 0).astype(np.int64)
            cells[r] = roots * V + res["out_token"][s:s + W_L]
        else:                                                # layer passed: the accepted drafts, test order
            acc = [i for i in range(5) if parent[r, i] >= 0 and status[r, i] == 1]
            acc.sort(key=lambda i: rank[r, i])
            assert len(acc) == W_L
            cells[r] = [(0 if parent[r, i] == 5 * r else 1) * V + token[r, i] for i in acc]
    w = softmax(sp.astype(np.float64))
    p_beam = np.concatenate([w[a] * softmax(zp[a].astype(np.float64)) for a in range(2)])
    if top_k:
        # the warping T of the joint: top-k cells, then the shortest prefix reaching top_p
        order = np.lexsort((np.arange(p_beam.size), -p_beam))[:top_k]
        kept = p_beam[order] / p_beam[order].sum()
        if 0.0 < top_p < 1.0:
            n = int(np.searchsorted(np.cumsum(kept), top_p - 1e-12) + 1)
            order, kept = order[:n], kept[:n] / kept[:n].sum()
        p_beam = np.zeros_like(p_beam)
        p_beam[order] = kept
    return cells, p_beam, float((res["l_last"] == 1).mean())


def _chi_square(cells, p_beam):
    R = len(cells)
    joint = np.outer(p_beam, p_beam).ravel()
    counts = np.bincount(cells[:, 0] * (2 * V) + cells[:, 1], minlength=joint.size).astype(np.float64)
    big = joint * R >= 5
    chi2 = ((counts[big] - joint[big] * R) ** 2 / (joint[big] * R)).sum()
    dof = int(big.sum()) - 1
    if (~big).any():
        e = joint[~big].sum() * R
        chi2 += (counts[~big].sum() - e) ** 2 / e
        dof += 1
    return chi2, dof


@pytest.mark.parametrize("seed,sigma_n", [(11, 0.7), (12, 2.0)])
def test_layer_one_beams_are_iid_p_beam(seed, sigma_n):
    cells, p_beam, short = _run(40000, seed, sigma_n)
    assert 0.02 < short < 0.98                # both outcomes of the layer occur
    chi2, dof = _chi_square(cells, p_beam)
    assert chi2 < stats.chi2.ppf(0.999, dof), (chi2, dof)
    # each beam alone follows p_beam as well
    for k in range(W_L):
        c = np.bincount(cells[:, k], minlength=2 * V)
        x = ((c - p_beam * len(cells)) ** 2 / (p_beam * len(cells))).sum()
        assert x < stats.chi2.ppf(0.999, 2 * V - 1), (k, x)


def test_warped_joints_top_k_top_p():
    cells, p_beam, short = _run(40000, 13, 1.0, top_k=6, top_p=0.85)
    assert 0.02 < short < 0.98
    support = p_beam > 0
    assert 2 <= support.sum() <= 6
    assert support[cells].all()                    # nothing outside the warped support is ever output
    keep = np.nonzero(support)[0]
    remap = -np.ones(2 * V, np.int64); remap[keep] = np.arange(len(keep))
    joint = np.outer(p_beam[keep], p_beam[keep]).ravel()
    counts = np.bincount(remap[cells[:, 0]] * len(keep) + remap[cells[:, 1]], minlength=joint.size)
    R = len(cells)
    big = joint * R >= 5
    chi2 = ((counts[big] - joint[big] * R) ** 2 / (joint[big] * R)).sum()
    dof = int(big.sum()) - 1
    if (~big).any():
        e = joint[~big].sum() * R
        chi2 += (counts[~big].sum() - e) ** 2 / e
        dof += 1
    assert chi2 < stats.chi2.ppf(0.999, dof), (chi2, dof)


def test_the_test_has_power():
    """The same statistic rejects when the small model's drafts are accepted unverified: the
    pairs then follow q_beam, not p_beam."""
    cells, p_beam, _ = _run(40000, 12, 2.0)
    rng = np.random.default_rng(0)
    zq_like = softmax(rng.normal(0, 2, size=2 * V))
    fake = rng.choice(2 * V, size=cells.shape, p=zq_like)
    chi2, dof = _chi_square(fake, p_beam)
    assert chi2 > 10 * stats.chi2.ppf(0.999, dof)
