"""Pins of the forest-assembly oracle: the built forest must be the genealogy the draws
describe (checked by following every draw's chain of parents independently), in a layout the
other oracles accept, and for chains it must reduce to the obvious numbering."""
import numpy as np

import oracle
from oracle import forest_build as fb


def _draws(rng, rbo, gamma, W_S):
    R = len(rbo) - 1
    dp = np.zeros((gamma, R * W_S), np.int32)
    for r in range(R):
        dp[0, r * W_S:(r + 1) * W_S] = rng.integers(rbo[r], rbo[r + 1], size=W_S)
        for l in range(1, gamma):
            dp[l, r * W_S:(r + 1) * W_S] = r * W_S + rng.integers(0, W_S, size=W_S)
    return dp, rng.integers(0, 1000, size=(gamma, R * W_S)).astype(np.int32)


def test_forest_is_the_genealogy_of_the_draws():
    rng = np.random.default_rng(0)
    rbo = np.array([0, 3, 4, 9], np.int32)
    gamma, W_S = 4, 5
    dp, dt = _draws(rng, rbo, gamma, W_S)
    f = fb.forest_build(rbo, gamma, W_S, dp, dt)
    assert f["N"] == 9 + 4 * 3 * 5 and sorted(f["node_of_draw"].ravel()) == sorted(set(f["node_of_draw"].ravel()))
    bno = f["beam_node_off"]
    tree_of_node = np.searchsorted(bno, np.arange(f["N"]), side="right") - 1
    for l in range(1, gamma + 1):
        for i in range(dp.shape[1]):
            n = f["node_of_draw"][l - 1, i]
            r, k = divmod(i, W_S)
            assert f["token"][n] == dt[l - 1, i] and f["draft_rank"][n] == k
            # token sequence and root found by walking the forest == by walking the draws
            seq_f, m = [], n
            while f["parent"][m] >= 0:
                assert f["parent"][m] < m and tree_of_node[f["parent"][m]] == tree_of_node[m]
                seq_f.append(int(f["token"][m])); m = f["parent"][m]
            seq_d, ll, ii = [], l, i
            while ll >= 1:
                seq_d.append(int(dt[ll - 1, ii]))
                p = dp[ll - 1, ii]
                ll, ii = ll - 1, p
            assert seq_f == seq_d and m == bno[ii] and len(seq_f) == l      # ii is now the input beam
    # every non-root node is some draw; roots are the beams
    assert set(range(f["N"])) - set(f["node_of_draw"].ravel()) == set(bno[:-1].tolist())
    # a layout the verification oracle accepts: run it
    V = 50
    z = rng.normal(size=(f["N"], V)).astype(np.float32)
    f["token"] = (f["token"] % V).astype(np.int32)
    out = oracle.verify_step(f, dict(V=V, W_min=2, W_max=3, W_nom=3, seed=1), z, z + 0.1, np.zeros(9), np.zeros(9))
    assert not out["error"].any()


def test_chains_number_the_obvious_way():
    # W_S = number of beams, draw k extends beam / draw k: every tree is a chain
    rbo = np.array([0, 3], np.int32)
    gamma, W_S = 3, 3
    dp = np.array([[0, 1, 2], [0, 1, 2], [0, 1, 2]], np.int32)
    dt = np.arange(9, dtype=np.int32).reshape(3, 3)
    f = fb.forest_build(rbo, gamma, W_S, dp, dt)
    assert list(f["beam_node_off"]) == [0, 4, 8, 12]
    assert list(f["parent"]) == [-1, 0, 1, 2, -1, 4, 5, 6, -1, 8, 9, 10]
    assert list(f["token"]) == [0, 0, 3, 6, 0, 1, 4, 7, 0, 2, 5, 8]
