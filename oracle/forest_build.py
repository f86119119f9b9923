"""Oracle of the draft-forest assembly.

TEST INFRASTRUCTURE, NOT PRODUCT CODE (plain Python loops; shares nothing with the CUDA library).

Section "Overview": the small model's beam sampling of width W_S over gamma steps traces a
forest of W_L trees, one per input beam; every later layer holds W_S nodes.  The draws of layer l
name their parents -- an input beam for l = 1, a draw of layer l-1 afterwards -- and this puts
them into the node layout the attention and the verification read: trees beam-major, a tree's
nodes contiguous, root first, then its draws in (layer, draw) order.  The order inside a tree is
a convention ("parity unpinned": any topological order is a valid forest); what the tests pin is
that the result IS the forest the draws describe (same parent/child relation, same tokens).
"""
import numpy as np


def forest_build(req_beam_off, gamma, W_S, draw_parent, draw_token):
    """draw_parent, draw_token: [gamma, R*W_S].  Returns dict(R, B, N, max_depth, req_beam_off,
    beam_node_off, parent, token, draft_rank, node_of_draw)."""
    rbo = np.asarray(req_beam_off, np.int64)
    R, B = len(rbo) - 1, int(rbo[-1])
    dp = np.asarray(draw_parent).reshape(gamma, R * W_S)
    dt = np.asarray(draw_token).reshape(gamma, R * W_S)
    N = B + gamma * R * W_S
    parent = np.full(N, -1, np.int32)
    token = np.zeros(N, np.int32)
    rank = np.zeros(N, np.int32)
    node_of_draw = np.full((gamma, R * W_S), -1, np.int32)
    beam_node_off = np.zeros(B + 1, np.int32)
    node = 0
    for r in range(R):
        # tree of every draw
        tree = {}
        for l in range(1, gamma + 1):
            for k in range(W_S):
                p = int(dp[l - 1, r * W_S + k])
                if l == 1:
                    assert rbo[r] <= p < rbo[r + 1]
                    tree[(l, k)] = p
                else:
                    assert r * W_S <= p < (r + 1) * W_S
                    tree[(l, k)] = tree[(l - 1, p - r * W_S)]
        for b in range(int(rbo[r]), int(rbo[r + 1])):
            beam_node_off[b] = node
            root = node
            node += 1
            for l in range(1, gamma + 1):
                for k in range(W_S):
                    if tree[(l, k)] != b:
                        continue
                    p = int(dp[l - 1, r * W_S + k])
                    parent[node] = root if l == 1 else node_of_draw[l - 2, p]
                    token[node] = dt[l - 1, r * W_S + k]
                    rank[node] = k
                    node_of_draw[l - 1, r * W_S + k] = node
                    node += 1
    beam_node_off[B] = node
    assert node == N
    return dict(R=R, B=B, N=N, max_depth=gamma, req_beam_off=rbo.astype(np.int32), beam_node_off=beam_node_off,
                parent=parent, token=token, draft_rank=rank, node_of_draw=node_of_draw)
