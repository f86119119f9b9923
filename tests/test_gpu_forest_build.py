"""GPU parity of dsbd_forest_build against the oracle (integer work: bit for bit) and its error
paths."""
import numpy as np
import pytest
import torch

from oracle import forest_build as ofb
import paper_2409_16560_b200 as dsbd

pytestmark = pytest.mark.gpu


def _draws(rng, rbo, gamma, W_S):
    R = len(rbo) - 1
    dp = np.zeros((gamma, R * W_S), np.int32)
    for r in range(R):
        dp[0, r * W_S:(r + 1) * W_S] = rng.integers(rbo[r], rbo[r + 1], size=W_S)
        for l in range(1, gamma):
            dp[l, r * W_S:(r + 1) * W_S] = r * W_S + rng.integers(0, W_S, size=W_S)
    return dp, rng.integers(0, 50000, size=(gamma, R * W_S)).astype(np.int32)


def _run(rbo, gamma, W_S, dp, dt):
    i32 = lambda a: torch.as_tensor(np.ascontiguousarray(a, dtype=np.int32)).cuda()
    f, nod, st = dsbd.forest_build(i32(rbo), rbo, gamma, W_S, i32(dp), i32(dt))
    torch.cuda.synchronize()
    return f, nod, int(st.item())


@pytest.mark.parametrize("R,max_beams,gamma,W_S", [(1, 1, 1, 1), (50, 8, 6, 12), (7, 64, 2, 64), (300, 3, 8, 8),
                                                   (3, 5, 16, 64)])
def test_against_the_oracle(R, max_beams, gamma, W_S):
    rng = np.random.default_rng(R * 1000 + gamma)
    rbo = np.concatenate([[0], np.cumsum(rng.integers(1, max_beams + 1, size=R))]).astype(np.int32)
    dp, dt = _draws(rng, rbo, gamma, W_S)
    ref = ofb.forest_build(rbo, gamma, W_S, dp, dt)
    f, nod, status = _run(rbo, gamma, W_S, dp, dt)
    assert status == 0
    for k in ("beam_node_off", "parent", "token", "draft_rank"):
        assert np.array_equal(f.dev[k].cpu().numpy(), ref[k]), k
    assert np.array_equal(nod.cpu().numpy(), ref["node_of_draw"])
    # the size of the largest tree, read back on request
    i32 = lambda a: torch.as_tensor(np.ascontiguousarray(a, dtype=np.int32)).cuda()
    f2, _, _ = dsbd.forest_build(i32(rbo), rbo, gamma, W_S, i32(dp), i32(dt), exact=True)
    assert f2.max_tree_nodes == int(np.diff(ref["beam_node_off"]).max())
    assert f.max_tree_nodes == 1 + gamma * W_S


def test_errors():
    rbo = np.array([0, 2, 4], np.int32)
    dp = np.array([[0, 1, 2, 3], [0, 1, 2, 3]], np.int32)
    dt = np.zeros((2, 4), np.int32)
    assert _run(rbo, 2, 2, dp, dt)[2] == 0
    bad = dp.copy(); bad[0, 0] = 2                      # request 0 names a beam of request 1
    assert _run(rbo, 2, 2, bad, dt)[2] == 4
    bad = dp.copy(); bad[1, 3] = 0                      # request 1 names a draw of request 0
    assert _run(rbo, 2, 2, bad, dt)[2] == 4
    with pytest.raises(dsbd.DsbdError):                 # more than 1024 draws per request
        _run(rbo, 17, 64, np.zeros((17, 128), np.int32), np.zeros((17, 128), np.int32))
