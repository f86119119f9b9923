"""Pins of the paged KV-cache oracle: a paged cache means its gathered content, so every commit
is checked against the packed oracle (itself pinned through the attention), over several decode
steps so that pages are shared, freed and reused; plus the allocator's invariants."""
import numpy as np

from oracle import kv_commit as kvc
from oracle import kv_paged as kvp


def _forest_on(rng, req_beam_off, max_nodes):
    """Random trees (root first, parent < node) on the given beams."""
    B = int(req_beam_off[-1])
    sizes = rng.integers(1, max_nodes + 1, size=B)
    node_off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    parent = np.full(node_off[-1], -1, np.int32)
    for b in range(B):
        for i in range(1, sizes[b]):
            parent[node_off[b] + i] = node_off[b] + rng.integers(0, i)
    return dict(R=len(req_beam_off) - 1, B=B, N=int(node_off[-1]), max_depth=max_nodes,
                req_beam_off=np.asarray(req_beam_off, np.int32), beam_node_off=node_off, parent=parent,
                token=np.zeros(node_off[-1], np.int32))


def _outputs(rng, forest, width):
    rbo, bno = forest["req_beam_off"], forest["beam_node_off"]
    R = forest["R"]
    out_off = (np.arange(R + 1) * width).astype(np.int32)
    out_width = rng.integers(1, width + 1, size=R).astype(np.int32)
    out_parent = np.zeros(R * width, np.int32)
    out_root = np.zeros(R * width, np.int32)
    for r in range(R):
        for k in range(width):
            b = rng.integers(rbo[r], rbo[r + 1])
            out_parent[r * width + k] = rng.integers(bno[b], bno[b + 1])
            out_root[r * width + k] = b
    return out_off, out_width, out_parent, out_root, rng.normal(size=R * width).astype(np.float32) - 9


def test_pages_round_trip():
    rng = np.random.default_rng(0)
    Hkv, d = 2, 4
    L = [130, 64, 1, 200]
    poff = np.concatenate([[0], np.cumsum(L)]).astype(np.int64)
    kp = rng.normal(size=poff[-1] * Hkv * d).astype(np.float32)
    vp = rng.normal(size=poff[-1] * Hkv * d).astype(np.float32)
    kpool, vpool, table, page_off, free, nfree = kvp.pack_into_pages(kp, vp, poff, Hkv, d, 20, rng)
    assert list(np.diff(page_off)) == [3, 1, 1, 4] and nfree == 11
    k2, v2 = kvp.gather(kpool, vpool, table, page_off, poff)
    assert np.array_equal(k2, kp) and np.array_equal(v2, vp)


def test_commits_over_several_steps_match_the_packed_oracle():
    rng = np.random.default_rng(1)
    Hkv, d, n_pages = 2, 4, 64
    rbo = np.array([0, 2, 3, 6], np.int32)
    L = [100, 100, 63, 129, 129, 129]                 # beams of a request share a length
    poff = np.concatenate([[0], np.cumsum(L)]).astype(np.int64)
    kp = rng.normal(size=poff[-1] * Hkv * d).astype(np.float32)
    vp = rng.normal(size=poff[-1] * Hkv * d).astype(np.float32)
    kpool, vpool, table, page_off, free, nfree = kvp.pack_into_pages(kp, vp, poff, Hkv, d, n_pages, rng)
    shared_seen = False
    for step in range(6):
        forest = _forest_on(rng, rbo, 5)
        kn = rng.normal(size=(forest["N"], Hkv, d)).astype(np.float32)
        vn = rng.normal(size=(forest["N"], Hkv, d)).astype(np.float32)
        outs = _outputs(rng, forest, 3)
        keep_best = step == 4
        ref = kvc.kv_commit(forest, Hkv, d, *outs, kn, vn, kp, vp, poff, keep_best=keep_best)
        res = kvp.kv_commit_paged(forest, *outs, kn, vn, kpool, vpool, table, page_off, poff, free, nfree,
                                  keep_best=keep_best)
        assert res["error"] == 0
        assert np.array_equal(res["new_req_beam_off"], ref["new_req_beam_off"])
        assert np.array_equal(res["new_prefix_off"], ref["new_prefix_off"])
        assert np.array_equal(res["new_beam_slot"], ref["new_beam_slot"])
        k2, v2 = kvp.gather(res["k_pool"], res["v_pool"], res["new_page_table"], res["new_page_off"],
                            res["new_prefix_off"])
        assert np.array_equal(k2, ref["k_cache"]) and np.array_equal(v2, ref["v_cache"])
        # allocator invariants: every page is free or referenced, never both; a page referenced
        # by two beams sits at the same position of both tables and is a full page
        used = set(res["new_page_table"].tolist())
        freeset = set(res["free_stack"][:res["free_count"]].tolist())
        assert not (used & freeset) and len(used) + len(freeset) == n_pages
        assert list(res["free_stack"][:res["free_count"]]) == sorted(freeset)
        where = {}
        nb = len(res["new_beam_slot"])
        for j in range(nb):
            Lj = int(res["new_prefix_off"][j + 1] - res["new_prefix_off"][j])
            pages = res["new_page_table"][res["new_page_off"][j]:res["new_page_off"][j + 1]]
            assert len(pages) == -(-Lj // kvp.PAGE)
            for i, pg in enumerate(pages):
                if pg in where:
                    shared_seen = True
                    assert where[pg] == i and (i + 1) * kvp.PAGE <= Lj
                where[pg] = i
        # next step starts from these beams
        rbo, poff = res["new_req_beam_off"], res["new_prefix_off"]
        kp, vp = ref["k_cache"], ref["v_cache"]
        kpool, vpool, table, page_off = res["k_pool"], res["v_pool"], res["new_page_table"], res["new_page_off"]
        free, nfree = res["free_stack"], res["free_count"]
    assert shared_seen


def test_pool_without_enough_free_pages():
    rng = np.random.default_rng(2)
    Hkv, d = 1, 2
    rbo = np.array([0, 1], np.int32)
    poff = np.array([0, 10], np.int64)
    kp = rng.normal(size=10 * d).astype(np.float32)
    kpool, vpool, table, page_off, free, nfree = kvp.pack_into_pages(kp, kp, poff, Hkv, d, 2)
    forest = _forest_on(rng, rbo, 2)
    kn = rng.normal(size=(forest["N"], Hkv, d)).astype(np.float32)
    outs = (np.array([0, 2], np.int32), np.array([2], np.int32), np.array([0, 0], np.int32),
            np.array([0, 0], np.int32), np.zeros(2, np.float32))
    assert kvp.kv_commit_paged(forest, *outs, kn, kn, kpool, vpool, table, page_off, poff, free, nfree)["error"] == 3
    assert kvp.kv_commit_paged(forest, *outs, kn, kn, kpool, vpool, table, page_off, poff, free, nfree,
                               keep_best=True)["error"] == 0
