"""A tiny context-table language-model pair for the exactness tests.

Every context up to depth 2 (V = 8 tokens, 2 input beams) has its own seeded logits row for
the large model (p) and the small model (q).  The helpers here build forests over it and
state the beam-sampling distribution straight from its definition (Eq. 1); none of this
code is shared with the oracle or with the CUDA library.
"""
import numpy as np

V = 8
BEAMS = 2


class ToyModel:
    def __init__(self, seed=0, noise=0.7, root_gap=0.9):
        rng = np.random.default_rng(seed)
        # logits after the contexts (beam), (beam, v), (beam, v, v'); float32 like the real path
        self.zp = [rng.normal(0, 1.5, size=(BEAMS,) + (V,) * (k + 1)).astype(np.float32)
                   for k in range(3)]
        self.zq = [(z + rng.normal(0, noise, size=z.shape)).astype(np.float32) for z in self.zp]
        # unequal cumulative scores of the two input beams, different under p and q
        self.root_logp = np.array([-1.0, -1.0 - root_gap])
        self.root_logq = np.array([-1.3, -0.8 - root_gap])

    @staticmethod
    def _logsoftmax(z):
        z = z.astype(np.float64)
        m = z.max(axis=-1, keepdims=True)
        return z - m - np.log(np.exp(z - m).sum(axis=-1, keepdims=True))

    def logp(self, k):
        """log p(next token | context of depth k), shape (BEAMS,)+(V,)*(k+1)."""
        return self._logsoftmax(self.zp[k])

    def logq(self, k):
        return self._logsoftmax(self.zq[k])

    def row(self, which, ctx):
        """logits row of the node whose context is ctx = (beam, tok1, ..)."""
        table = (self.zp if which == "p" else self.zq)[len(ctx) - 1]
        return table[tuple(ctx)]

    def seq_logprob(self, which, ctx):
        """log of the model's probability of the sequence ctx (root score + token log-probs)."""
        root = (self.root_logp if which == "p" else self.root_logq)[ctx[0]]
        lp = self.logp if which == "p" else self.logq
        s = root
        for k in range(1, len(ctx)):
            s = s + lp(k - 1)[tuple(ctx[:k + 1])]
        return s

    def beam_dist(self, which, contexts):
        """Eq. 1: the joint over (contexts x V), p(ctx, v) / sum over all (ctx', v').
        contexts: list of equal-depth contexts.  Returns an array [len(contexts), V]."""
        lp = self.logp if which == "p" else self.logq
        k = len(contexts[0]) - 1
        joint = np.array([np.exp(self.seq_logprob(which, c) + lp(k)[tuple(c)]) for c in contexts])
        return joint / joint.sum()


def build_forest(model, layers, gamma):
    """One request.  layers[l] = list of drafts of draft layer l+1, each (parent, token) with
    parent an index into the previous layer's draft list (layer 0: the beam index), listed in
    the order the small model drew them.  Returns (forest dict, logits_p, logits_q, contexts)
    with nodes stored tree-major in breadth-first order and draft_rank = draw order."""
    nodes = [dict(ctx=(b,), depth=0, rank=0, tree=b, parent=None) for b in range(BEAMS)]
    prev = list(range(BEAMS))
    for l, drafts in enumerate(layers):
        cur = []
        for rank, (par, tok) in enumerate(drafts):
            pn = nodes[prev[par]]
            nodes.append(dict(ctx=pn["ctx"] + (tok,), depth=l + 1, rank=rank, tree=pn["tree"],
                              parent=prev[par]))
            cur.append(len(nodes) - 1)
        prev = cur
    order = sorted(range(len(nodes)), key=lambda i: (nodes[i]["tree"], nodes[i]["depth"],
                                                     nodes[i]["rank"]))
    pos = {old: new for new, old in enumerate(order)}
    N = len(nodes)
    parent = np.full(N, -1, np.int32)
    token = np.zeros(N, np.int32)
    rank = np.zeros(N, np.int32)
    ctxs = [None] * N
    for old in range(N):
        n = pos[old]
        nd = nodes[old]
        ctxs[n] = nd["ctx"]
        rank[n] = nd["rank"]
        if nd["parent"] is not None:
            parent[n] = pos[nd["parent"]]
            token[n] = nd["ctx"][-1]
    tree_sizes = [sum(1 for nd in nodes if nd["tree"] == b) for b in range(BEAMS)]
    forest = dict(R=1, B=BEAMS, N=N, max_depth=gamma,
                  req_beam_off=np.array([0, BEAMS], np.int32),
                  beam_node_off=np.concatenate([[0], np.cumsum(tree_sizes)]).astype(np.int32),
                  parent=parent, token=token, draft_rank=rank)
    zp = np.stack([model.row("p", c) if len(c) <= 3 else np.zeros(V, np.float32) for c in ctxs])
    zq = np.stack([model.row("q", c) if len(c) <= 3 else np.zeros(V, np.float32) for c in ctxs])
    return forest, zp, zq, ctxs, pos


def concat_forests(items):
    """Stack single-request forests (forest, zp, zq) into one batch of R requests."""
    R = len(items)
    req_beam_off = np.zeros(R + 1, np.int32)
    beam_node_off = [np.zeros(1, np.int32)]
    parent, token, rank, zp, zq = [], [], [], [], []
    n_base = 0
    for r, (f, a, b) in enumerate(items):
        req_beam_off[r + 1] = req_beam_off[r] + f["B"]
        beam_node_off.append(f["beam_node_off"][1:] + n_base)
        parent.append(np.where(f["parent"] >= 0, f["parent"] + n_base, -1))
        token.append(f["token"])
        rank.append(f["draft_rank"])
        zp.append(a)
        zq.append(b)
        n_base += f["N"]
    forest = dict(R=R, B=int(req_beam_off[-1]), N=n_base, max_depth=items[0][0]["max_depth"],
                  req_beam_off=req_beam_off,
                  beam_node_off=np.concatenate(beam_node_off).astype(np.int32),
                  parent=np.concatenate(parent).astype(np.int32),
                  token=np.concatenate(token).astype(np.int32),
                  draft_rank=np.concatenate(rank).astype(np.int32))
    return forest, np.concatenate(zp), np.concatenate(zq)
