"""Pins of the oracle's forest attention: library attention on the cases where the forest
mask reduces to a standard one, and the locality properties of the mask."""
import numpy as np
import torch
import torch.nn.functional as F

import oracle


def _rand_problem(rng, tree_parents, L, Hq, Hkv, d):
    """tree_parents: list (one per tree) of local parent arrays (-1 root, parent < index)."""
    B = len(tree_parents)
    sizes = [len(t) for t in tree_parents]
    node_off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    parent = np.concatenate([np.where(np.array(t) >= 0, np.array(t) + node_off[b], -1)
                             for b, t in enumerate(tree_parents)]).astype(np.int32)
    N = int(node_off[-1])
    forest = dict(R=1, B=B, N=N, max_depth=max(N, 1), req_beam_off=[0, B], beam_node_off=node_off,
                  parent=parent, token=np.zeros(N, np.int32))
    prefix_off = np.concatenate([[0], np.cumsum(L)]).astype(np.int64)
    q = rng.normal(size=(N, Hq, d)).astype(np.float32)
    kn = rng.normal(size=(N, Hkv, d)).astype(np.float32)
    vn = rng.normal(size=(N, Hkv, d)).astype(np.float32)
    kp = [rng.normal(size=(Hkv, l, d)).astype(np.float32) for l in L]
    vp = [rng.normal(size=(Hkv, l, d)).astype(np.float32) for l in L]
    return forest, prefix_off, q, kn, vn, kp, vp


def _run(forest, prefix_off, q, kn, vn, kp, vp, Hq, Hkv, d, scale):
    return oracle.forest_attention(forest, Hq, Hkv, d, scale, q, kn, vn,
                                   np.concatenate([x.ravel() for x in kp]),
                                   np.concatenate([x.ravel() for x in vp]), prefix_off)


def _sdpa_tree(q, kn, vn, kp, vp, local_parent, Hq, Hkv, scale):
    """One tree through torch's scaled_dot_product_attention with an explicit boolean mask:
    keys = prefix ++ tree nodes; node i may see the prefix and the reflexive-transitive
    closure of the parent relation (built here by repeated squaring of the adjacency)."""
    n = len(local_parent)
    adj = np.eye(n, dtype=bool)
    for i, p in enumerate(local_parent):
        if p >= 0:
            adj[i, p] = True
    clo = adj.copy()
    for _ in range(n):
        clo = (clo.astype(int) @ adj.astype(int)) > 0
    L = kp.shape[1]
    mask = torch.from_numpy(np.concatenate([np.ones((n, L), bool), clo], axis=1))
    g = Hq // Hkv
    K = torch.from_numpy(np.concatenate([kp, kn.transpose(1, 0, 2)], axis=1)).double()   # [Hkv, L+n, d]
    Vv = torch.from_numpy(np.concatenate([vp, vn.transpose(1, 0, 2)], axis=1)).double()
    K = K.repeat_interleave(g, dim=0)
    Vv = Vv.repeat_interleave(g, dim=0)
    Q = torch.from_numpy(q.transpose(1, 0, 2)).double()                                    # [Hq, n, d]
    o = F.scaled_dot_product_attention(Q[None], K[None], Vv[None], attn_mask=mask, scale=scale)[0]
    return o.permute(1, 0, 2).numpy()


def test_general_forest_against_library_attention():
    rng = np.random.default_rng(0)
    trees = [[-1, 0, 0, 1, 1, 2, 2, 3], [-1], [-1, 0, 1, 2], [-1, 0, 0, 0, 2]]
    L = [7, 12, 1, 30]
    for (Hq, Hkv, d) in [(4, 4, 16), (8, 2, 32)]:
        scale = 1 / np.sqrt(d)
        forest, poff, q, kn, vn, kp, vp = _rand_problem(rng, trees, L, Hq, Hkv, d)
        out = _run(forest, poff, q, kn, vn, kp, vp, Hq, Hkv, d, scale)
        no = forest["beam_node_off"]
        for b, t in enumerate(trees):
            s = slice(no[b], no[b + 1])
            ref = _sdpa_tree(q[s], kn[s], vn[s], kp[b], vp[b], t, Hq, Hkv, scale)
            assert np.abs(out[s] - ref).max() < 1e-12


def test_single_node_tree_is_decode_attention_and_chain_is_causal():
    rng = np.random.default_rng(1)
    Hq = Hkv = 2
    d = 8
    scale = 0.3
    # single node: plain decode attention over prefix ++ self, no mask at all
    forest, poff, q, kn, vn, kp, vp = _rand_problem(rng, [[-1]], [9], Hq, Hkv, d)
    out = _run(forest, poff, q, kn, vn, kp, vp, Hq, Hkv, d, scale)
    K = torch.from_numpy(np.concatenate([kp[0], kn.transpose(1, 0, 2)], axis=1)).double()
    Vv = torch.from_numpy(np.concatenate([vp[0], vn.transpose(1, 0, 2)], axis=1)).double()
    Q = torch.from_numpy(q.transpose(1, 0, 2)).double()
    ref = F.scaled_dot_product_attention(Q[None], K[None], Vv[None], scale=scale)[0].permute(1, 0, 2)
    assert np.abs(out - ref.numpy()).max() < 1e-12
    # chain of 5: causal attention over the sequence prefix ++ chain (last 5 query rows)
    forest, poff, q, kn, vn, kp, vp = _rand_problem(rng, [[-1, 0, 1, 2, 3]], [6], Hq, Hkv, d)
    out = _run(forest, poff, q, kn, vn, kp, vp, Hq, Hkv, d, scale)
    K = torch.from_numpy(np.concatenate([kp[0], kn.transpose(1, 0, 2)], axis=1)).double()
    Vv = torch.from_numpy(np.concatenate([vp[0], vn.transpose(1, 0, 2)], axis=1)).double()
    Qfull = torch.zeros(Hq, 11, d, dtype=torch.float64)
    Qfull[:, 6:] = torch.from_numpy(q.transpose(1, 0, 2)).double()
    ref = F.scaled_dot_product_attention(Qfull[None], K[None], Vv[None], is_causal=True, scale=scale)[0]
    assert np.abs(out - ref[:, 6:].permute(1, 0, 2).numpy()).max() < 1e-12


def test_mask_locality():
    """Other trees never matter; a subtree moved under another parent changes only its rows;
    siblings do not see each other."""
    rng = np.random.default_rng(2)
    Hq, Hkv, d = 4, 2, 8
    trees = [[-1, 0, 0, 1], [-1, 0, 1]]
    forest, poff, q, kn, vn, kp, vp = _rand_problem(rng, trees, [5, 4], Hq, Hkv, d)
    base = _run(forest, poff, q, kn, vn, kp, vp, Hq, Hkv, d, 0.25)
    # perturb everything that belongs to tree 1: tree 0's rows are unchanged
    kn2, vn2 = kn.copy(), vn.copy()
    kn2[4:] += 1.0
    vn2[4:] -= 2.0
    kp2 = [kp[0], kp[1] + 1.0]
    out = _run(forest, poff, q, kn2, vn2, kp2, vp, Hq, Hkv, d, 0.25)
    assert np.array_equal(out[:4], base[:4]) and not np.allclose(out[4:], base[4:])
    # node 2 is a sibling of node 1: changing node 2's key/value leaves nodes 0, 1, 3 alone
    kn3, vn3 = kn.copy(), vn.copy()
    kn3[2] += 3.0
    vn3[2] += 3.0
    out = _run(forest, poff, q, kn3, vn3, kp, vp, Hq, Hkv, d, 0.25)
    assert np.array_equal(out[[0, 1, 3]], base[[0, 1, 3]]) and not np.allclose(out[2], base[2])
    # re-hang node 3 from node 1 to node 2: only row 3 changes
    f2 = dict(forest, parent=np.array([-1, 0, 0, 2, -1, 4, 5], np.int32))
    out = _run(f2, poff, q, kn, vn, kp, vp, Hq, Hkv, d, 0.25)
    assert np.array_equal(out[[0, 1, 2, 4, 5, 6]], base[[0, 1, 2, 4, 5, 6]])
    assert not np.allclose(out[3], base[3])
