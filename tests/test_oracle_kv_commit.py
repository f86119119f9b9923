"""Pins of the KV-commit oracle (Section "Forest-based Parallel Decoding": the caches are
updated according to the output beams; Section "Reducing Memory Cost": keep one beam).

The committed cache of an output beam must hold exactly what its parent node attended to, so
ordinary decode attention over the committed cache has to reproduce the forest attention of
that node (the attention oracle is pinned on its own against library attention)."""
import numpy as np

import oracle
from oracle import kv_commit as kvc


def _problem(rng, trees, L, Hq, Hkv, d, R_split=None):
    B = len(trees)
    sizes = [len(t) for t in trees]
    node_off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    parent = np.concatenate([np.where(np.array(t) >= 0, np.array(t) + node_off[b], -1)
                             for b, t in enumerate(trees)]).astype(np.int32)
    N = int(node_off[-1])
    rbo = np.asarray(R_split if R_split is not None else [0, B], np.int32)
    forest = dict(R=len(rbo) - 1, B=B, N=N, max_depth=max(sizes), req_beam_off=rbo, beam_node_off=node_off,
                  parent=parent, token=np.zeros(N, np.int32))
    prefix_off = np.concatenate([[0], np.cumsum(L)]).astype(np.int64)
    q = rng.normal(size=(N, Hq, d)).astype(np.float32)
    kn = rng.normal(size=(N, Hkv, d)).astype(np.float32)
    vn = rng.normal(size=(N, Hkv, d)).astype(np.float32)
    kp = np.concatenate([rng.normal(size=(Hkv, l, d)).astype(np.float32).ravel() for l in L])
    vp = np.concatenate([rng.normal(size=(Hkv, l, d)).astype(np.float32).ravel() for l in L])
    return forest, prefix_off, q, kn, vn, kp, vp


def _random_outputs(rng, forest, width):
    """`width` output beams per request, each extending a random node of the request."""
    rbo, bno = forest["req_beam_off"], forest["beam_node_off"]
    R = forest["R"]
    out_off = (np.arange(R + 1) * (width + 1)).astype(np.int32)      # one spare slot per request
    out_width = np.full(R, width, np.int32)
    slots = int(out_off[-1])
    out_parent = np.full(slots, -1, np.int32)
    out_root = np.full(slots, -1, np.int32)
    out_logp = rng.normal(size=slots).astype(np.float32) - 5.0
    for r in range(R):
        for k in range(width):
            b = rng.integers(rbo[r], rbo[r + 1])
            n = rng.integers(bno[b], bno[b + 1])
            out_parent[out_off[r] + k] = n
            out_root[out_off[r] + k] = b
    return out_off, out_width, out_parent, out_root, out_logp


TREES = [[-1, 0, 0, 1, 1, 2], [-1, 0, 1, 2], [-1], [-1, 0, 0, 0, 3]]


def test_committed_cache_is_what_the_parent_node_attended_to():
    rng = np.random.default_rng(0)
    Hq, Hkv, d, scale = 4, 2, 16, 0.25
    L = [7, 3, 5, 9]
    forest, poff, q, kn, vn, kp, vp = _problem(rng, TREES, L, Hq, Hkv, d, R_split=[0, 2, 4])
    ref = oracle.forest_attention(forest, Hq, Hkv, d, scale, q, kn, vn, kp, vp, poff)
    oo, ow, op, orb, olp = _random_outputs(rng, forest, 3)
    res = kvc.kv_commit(forest, Hkv, d, oo, ow, op, orb, olp, kn, vn, kp, vp, poff)
    assert len(res["new_beam_slot"]) == 6 and list(res["new_req_beam_off"]) == [0, 3, 6]
    for j, s in enumerate(res["new_beam_slot"]):
        n = int(op[s])
        Lj = int(res["new_prefix_off"][j + 1] - res["new_prefix_off"][j])
        base = int(res["new_prefix_off"][j]) * Hkv * d
        kc = res["k_cache"][base:base + Hkv * Lj * d].reshape(Hkv, Lj, d)
        vc = res["v_cache"][base:base + Hkv * Lj * d].reshape(Hkv, Lj, d)
        # decode attention of node n's query: prefix = committed cache without its last
        # entry, own key/value = that last entry
        one = dict(R=1, B=1, N=1, max_depth=0, req_beam_off=[0, 1], beam_node_off=[0, 1],
                   parent=np.array([-1], np.int32), token=np.zeros(1, np.int32))
        o = oracle.forest_attention(one, Hq, Hkv, d, scale, q[n:n + 1],
                                    np.ascontiguousarray(kc[:, -1, :])[None], np.ascontiguousarray(vc[:, -1, :])[None],
                                    np.ascontiguousarray(kc[:, :-1, :]).ravel(),
                                    np.ascontiguousarray(vc[:, :-1, :]).ravel(),
                                    np.array([0, Lj - 1], np.int64))
        assert np.allclose(o[0], ref[n], atol=1e-12, rtol=0), (j, n)


def test_single_chain_is_a_plain_append():
    rng = np.random.default_rng(1)
    Hkv, d, L = 2, 8, 6
    forest, poff, q, kn, vn, kp, vp = _problem(rng, [[-1, 0, 1, 2]], [L], 2, Hkv, d)
    for n in range(4):            # output beam extends node n: cache grows by the nodes 0..n
        res = kvc.kv_commit(forest, Hkv, d, [0, 1], [1], [n], [0], [-1.0], kn, vn, kp, vp, poff)
        want_k = np.concatenate([kp.reshape(Hkv, L, d), kn[:n + 1].transpose(1, 0, 2)], axis=1)
        want_v = np.concatenate([vp.reshape(Hkv, L, d), vn[:n + 1].transpose(1, 0, 2)], axis=1)
        assert np.array_equal(res["k_cache"], want_k.ravel())
        assert np.array_equal(res["v_cache"], want_v.ravel())
        assert list(res["new_prefix_off"]) == [0, L + n + 1]


def test_lengths_and_offsets():
    rng = np.random.default_rng(2)
    Hkv, d = 2, 4
    L = [4, 6, 2, 3]
    forest, poff, q, kn, vn, kp, vp = _problem(rng, TREES, L, 2, Hkv, d, R_split=[0, 1, 4])
    oo, ow, op, orb, olp = _random_outputs(rng, forest, 2)
    ow[0] = 0                                            # a request without output beams
    res = kvc.kv_commit(forest, Hkv, d, oo, ow, op, orb, olp, kn, vn, kp, vp, poff)
    assert list(res["new_req_beam_off"]) == [0, 0, 2]
    depth = np.zeros(forest["N"], int)
    for n, p in enumerate(forest["parent"]):
        depth[n] = 0 if p < 0 else depth[p] + 1
    for j, s in enumerate(res["new_beam_slot"]):
        want = L[orb[s]] + depth[op[s]] + 1
        assert res["new_prefix_off"][j + 1] - res["new_prefix_off"][j] == want
    assert res["k_cache"].size == res["new_prefix_off"][-1] * Hkv * d


def test_keep_best_takes_the_lowest_perplexity():
    rng = np.random.default_rng(3)
    Hkv, d = 1, 4
    L = [5, 5, 9, 2]
    forest, poff, q, kn, vn, kp, vp = _problem(rng, TREES, L, 1, Hkv, d, R_split=[0, 2, 4])
    depth = np.zeros(forest["N"], int)
    for n, p in enumerate(forest["parent"]):
        depth[n] = 0 if p < 0 else depth[p] + 1
    for trial in range(20):
        oo, ow, op, orb, olp = _random_outputs(rng, forest, 3)
        res = kvc.kv_commit(forest, Hkv, d, oo, ow, op, orb, olp, kn, vn, kp, vp, poff, keep_best=True)
        assert list(res["new_req_beam_off"]) == [0, 1, 2]
        for r in range(2):
            slots = np.arange(oo[r], oo[r] + ow[r])
            length = np.array([L[orb[s]] + depth[op[s]] + 2 for s in slots], float)
            ppl = np.exp(-olp[slots].astype(np.float64) / length)
            assert res["new_beam_slot"][r] == slots[np.argmin(ppl)]
    # equal lengths: lowest perplexity = highest log-probability
    oo, ow = np.array([0, 3, 6], np.int32), np.array([3, 3], np.int32)
    op = np.array([0, 0, 0, 10, 10, 10], np.int32)
    orb = np.array([0, 0, 0, 2, 2, 2], np.int32)
    olp = np.array([-3, -1, -2, -9, -9.5, -8], np.float32)
    res = kvc.kv_commit(forest, Hkv, d, oo, ow, op, orb, olp, kn, vn, kp, vp, poff, keep_best=True)
    assert list(res["new_beam_slot"]) == [1, 5]
