"""Shared helpers of the GPU parity tests: run the CUDA library and the oracle on the same
bytes and compare them under the stated bars.

Bars
  attention : |gpu - oracle| <= 1e-2 + 2e-2 * |oracle| element-wise for bf16 inputs (fp32
              accumulation); 1e-4 + 1e-4 * |oracle| for fp32 inputs.
  verify    : widths, node statuses, l_last, output parents / nodes / tokens / sources
              bit-exact.  The only exception: a request whose first differing layer holds a
              decision of the kind that differs which the oracle flags as a near tie.  Such a
              request is compared up to that layer only and counted in one of two classes:
                "decision" -- an accept test with |u - ratio| < 1e-5, a layer width whose
                    threshold lies within 1e-5 of the tail probability, or a top-k / top-p cut
                    within 1e-5 (relative) of a tie.  At most 1e-4 of the decisions, rounded
                    DOWN: none at all in a test with fewer than 10 000 decisions.
                "draw" -- the statuses and widths agree and only a sampled token differs, the
                    uniform lying within 1e-6 of a boundary of the oracle's cell in the
                    cumulative distribution.  The CUDA path evaluates cell masses in fp32, the
                    oracle in fp64, and a large vocabulary has thousands of cells narrower than
                    the difference, so this class cannot be emptied; it is counted on its own
                    and must stay below 1e-3 of the decisions (rounded up per test).
              The session's totals are printed at its end and checked against the same bars.
              Scores: 1e-4 + 1e-5 * |oracle|.
"""
import math

import numpy as np
import torch

import oracle
import paper_2409_16560_b200 as dsbd

OUT_KEYS = ("out_parent", "out_node", "out_root_beam", "out_token", "out_source")


def to_host_f32(t):
    return t.detach().float().cpu().numpy()


def sub_forest(forest, reqs):
    """Forest arrays restricted to the listed requests (nodes renumbered); returns the arrays,
    the kept node ids and the kept beam ids."""
    rbo, bno = np.asarray(forest["req_beam_off"]), np.asarray(forest["beam_node_off"])
    beams = np.concatenate([np.arange(rbo[r], rbo[r + 1]) for r in reqs])
    nodes = np.concatenate([np.arange(bno[b], bno[b + 1]) for b in beams])
    remap = np.full(forest["N"], -1, np.int64)
    remap[nodes] = np.arange(len(nodes))
    par = np.asarray(forest["parent"])[nodes]
    sub = dict(R=len(reqs), B=len(beams), N=len(nodes), max_depth=forest["max_depth"],
               req_beam_off=np.concatenate([[0], np.cumsum([rbo[r + 1] - rbo[r] for r in reqs])]).astype(np.int32),
               beam_node_off=np.concatenate([[0], np.cumsum(bno[beams + 1] - bno[beams])]).astype(np.int32),
               parent=np.where(par >= 0, remap[np.maximum(par, 0)], -1).astype(np.int32),
               token=np.asarray(forest["token"])[nodes].astype(np.int32))
    if forest.get("draft_rank") is not None:
        sub["draft_rank"] = np.asarray(forest["draft_rank"])[nodes].astype(np.int32)
    return sub, nodes, beams


def run_gpu_verify(forest_arrays, params, zp, zq, root_logp, root_logq, device="cuda", row_stride=None):
    """Calls dsbd_verify_step through the binding; returns (dict of numpy outputs, status)."""
    f = dsbd.Forest(forest_arrays, device)
    prm = dict(params)
    for k in ("W_min_r", "W_max_r", "W_nom_r"):
        if prm.get(k) is not None:
            prm[k] = torch.as_tensor(np.asarray(prm[k], dtype=np.int32)).to(device)
    out_off = oracle.default_out_off(forest_arrays, params)
    out = dsbd.alloc_verify_out(f, out_off, device)
    status = dsbd.verify_step(f, prm, zp, zq, root_logp, root_logq, out, row_stride=row_stride)
    torch.cuda.synchronize()
    res = {k: v.cpu().numpy() for k, v in out.items()}
    res["layer_width"] = res["layer_width"].reshape(f.R, f.max_depth + 1)
    return res, int(status.item())


def compare_verify(ref, gpu, forest, req_ids=None):
    """Compares oracle result `ref` (over a forest whose requests are the GPU's requests
    `req_ids`, or all of them) with the GPU outputs.  Returns (exempt, decisions); raises
    AssertionError on any mismatch that no near tie explains."""
    R = int(forest["R"])
    rbo, bno = np.asarray(forest["req_beam_off"]), np.asarray(forest["beam_node_off"])
    parent = np.asarray(forest["parent"])
    depth = np.zeros(forest["N"], np.int64)
    for n, p in enumerate(parent):
        depth[n] = 0 if p < 0 else depth[p] + 1
    gamma = int(forest["max_depth"])
    exempt = Exempt()
    tr_start = np.searchsorted(ref["trace_req"], np.arange(R + 1))
    for r in range(R):
        n0, n1 = bno[rbo[r]], bno[rbo[r + 1]]
        s0 = ref["out_off"][r]
        assert ref["error"][r] == 0 and gpu["req_error"][r] == 0, (r, ref["error"][r], gpu["req_error"][r])

        def layer_equal(l):
            if ref["layer_width"][r, l - 1] != gpu["layer_width"][r, l - 1]:
                return False
            ids = np.arange(n0, n1)[depth[n0:n1] == l]
            if not np.array_equal(ref["node_status"][ids], gpu["node_status"][ids]):
                return False
            rl, gl = ref["l_last"][r] == l, gpu["l_last"][r] == l
            if rl != gl:
                return False
            if rl:
                w = ref["out_width"][r]
                if w != gpu["out_width"][r]:
                    return False
                for k in OUT_KEYS:
                    if not np.array_equal(ref[k][s0:s0 + w], gpu[k][s0:s0 + w]):
                        return False
            return True

        first_bad = None
        for l in range(1, gamma + 2):
            if not layer_equal(l):
                first_bad = l
                break
            if ref["l_last"][r] == l:
                break
        if first_bad is None:
            ids = np.arange(n0, n1)
            fin = np.isfinite(ref["node_logp"][ids])
            for a, b in (("node_logp", "node_logp"), ("node_logq", "node_logq"), ("lse_p", "lse_p"),
                         ("lse_q", "lse_q")):
                x, y = ref[a][ids][fin], gpu[b][ids][fin]
                assert np.all(np.abs(x - y) <= 1e-4 + 1e-5 * np.abs(x)), (r, a, np.abs(x - y).max())
            w = ref["out_width"][r]
            for k in ("out_logp", "out_logq"):
                x, y = ref[k][s0:s0 + w], gpu[k][s0:s0 + w]
                assert np.all(np.abs(x - y) <= 1e-4 + 1e-5 * np.abs(x)), (r, k)
            continue
        recs = np.arange(tr_start[r], tr_start[r + 1])
        recs = recs[ref["trace_layer"][recs] == first_bad]
        kind, near = ref["trace_kind"][recs], ref["trace_near"][recs] != 0
        l = first_bad
        ids = np.arange(n0, n1)[depth[n0:n1] == l]
        warp_tie = bool(np.any(near & (kind == oracle.TR_WARP)))
        if l <= gamma and ref["layer_width"][r, l - 1] != gpu["layer_width"][r, l - 1]:
            ok, cls = warp_tie or bool(np.any(near & (kind == oracle.TR_WIDTH))), "decision"
        elif l <= gamma and not np.array_equal(ref["node_status"][ids], gpu["node_status"][ids]):
            ok, cls = warp_tie or bool(np.any(near & (kind == oracle.TR_ACCEPT))), "decision"
        else:
            # same statuses and width: a sampled token differs
            draws = recs[np.isin(kind, (oracle.TR_RESIDUAL, oracle.TR_FILL, oracle.TR_EXTRA))]
            u, lo, hi = ref["trace_u"][draws], ref["trace_a"][draws], ref["trace_b"][draws]
            tight = bool(np.any(np.minimum(np.abs(u - lo), np.abs(u - hi)) < DRAW_BAND))
            ok, cls = tight or warp_tie, ("draw" if tight else "decision")
        assert ok, (
            "request %d diverges at layer %d with no near tie of that kind there: "
            "oracle width %s gpu width %s, l_last %d/%d" % (
                r if req_ids is None else req_ids[r], first_bad, ref["layer_width"][r],
                gpu["layer_width"][r], ref["l_last"][r], gpu["l_last"][r]))
        exempt[cls] += 1
    return exempt, len(ref["trace_req"])


DRAW_BAND = 1e-6       # distance of a draw's uniform from a cell boundary inside which tokens may differ
DRAW_RATE = 1e-3       # allowed "draw" class divergences per decision

# exempt requests and decisions of every check_exempt call of this session
TOTALS = {"decision": 0, "draw": 0, "decisions": 0, "checks": 0}


class Exempt(dict):
    """Counts of exempt requests by class; adds like a vector."""

    def __init__(self, decision=0, draw=0):
        super().__init__(decision=decision, draw=draw)

    def __add__(self, other):
        return Exempt(self["decision"] + other["decision"], self["draw"] + other["draw"])

    __radd__ = lambda self, other: self if other == 0 else self.__add__(other)


def check_exempt(exempt, decisions):
    """The near-tie allowance of one test (see the module docstring); feeds the session totals."""
    TOTALS["decision"] += exempt["decision"]
    TOTALS["draw"] += exempt["draw"]
    TOTALS["decisions"] += int(decisions)
    TOTALS["checks"] += 1
    assert exempt["decision"] <= math.floor(1e-4 * decisions), \
        "%d exempt decisions in %d decisions" % (exempt["decision"], decisions)
    assert exempt["draw"] <= math.ceil(DRAW_RATE * decisions), \
        "%d draws differ inside a tie in %d decisions" % (exempt["draw"], decisions)


def attention_close(gpu, ref, bf16):
    gpu = np.asarray(gpu, dtype=np.float64)
    atol, rtol = (1e-2, 2e-2) if bf16 else (1e-4, 1e-4)
    err = np.abs(gpu - ref)
    bad = err > atol + rtol * np.abs(ref)
    assert not bad.any(), "max abs err %.3e, %d elements outside the bar" % (err.max(), bad.sum())
    return float(err.max())
