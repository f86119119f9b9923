"""ctypes front end of the DSBD oracle.

TEST INFRASTRUCTURE, NOT PRODUCT CODE.  Only tests, the smoke check and the benchmark's
CPU-baseline leg import this package; the CUDA library never does.  The arithmetic lives in
``dsbd_oracle.c`` (plain C, double precision, written from the paper); this file only
marshals numpy arrays.

A forest is passed as a plain dict of numpy arrays:
``R, B, N, max_depth, req_beam_off[R+1], beam_node_off[B+1], parent[N], token[N]`` and
optionally ``draft_rank[N]``.
"""
import ctypes as C

import numpy as np

from . import build as _build

_lib = None

NODE_UNREACHED, NODE_ACCEPTED, NODE_REJECTED, NODE_CUT, NODE_PRUNED = 0, 1, 2, 3, 4
SRC_DRAFT, SRC_RESIDUAL, SRC_FILL, SRC_EXTRA = 0, 1, 2, 3
TR_ACCEPT, TR_RESIDUAL, TR_FILL, TR_EXTRA, TR_WIDTH, TR_WARP = 0, 1, 2, 3, 4, 5

_i32p = C.POINTER(C.c_int32)
_i64p = C.POINTER(C.c_int64)
_f32p = C.POINTER(C.c_float)
_f64p = C.POINTER(C.c_double)
_i8p = C.POINTER(C.c_int8)


class _Forest(C.Structure):
    _fields_ = [("R", C.c_int32), ("B", C.c_int32), ("N", C.c_int32), ("max_depth", C.c_int32),
                ("req_beam_off", _i32p), ("beam_node_off", _i32p), ("parent", _i32p),
                ("token", _i32p), ("draft_rank", _i32p)]


class _Params(C.Structure):
    _fields_ = [("V", C.c_int32), ("temperature", C.c_double), ("thresh", C.c_double),
                ("W_min", C.c_int32), ("W_max", C.c_int32), ("W_nom", C.c_int32),
                ("W_min_r", _i32p), ("W_max_r", _i32p), ("W_nom_r", _i32p),
                ("seed", C.c_uint64), ("step", C.c_uint64), ("req_id", _i32p),
                ("top_k", C.c_int32), ("top_p", C.c_double)]


class _VerifyOut(C.Structure):
    _fields_ = [("l_last", _i32p), ("out_width", _i32p), ("out_off", _i32p),
                ("out_parent", _i32p), ("out_node", _i32p), ("out_root_beam", _i32p),
                ("out_token", _i32p), ("out_logp", _f64p), ("out_logq", _f64p),
                ("out_source", _i32p), ("node_status", _i8p), ("layer_width", _i32p),
                ("node_logp", _f64p), ("node_logq", _f64p), ("lse_p", _f64p), ("lse_q", _f64p),
                ("error", _i32p),
                ("trace_cap", C.c_int64), ("trace_len", _i64p),
                ("trace_req", _i32p), ("trace_layer", _i32p), ("trace_kind", _i32p),
                ("trace_index", _i32p), ("trace_near", _i32p),
                ("trace_u", _f64p), ("trace_a", _f64p), ("trace_b", _f64p),
                ("dist_cap", C.c_int64), ("dist_len", _i64p), ("dist", _f64p)]


def lib():
    """Load (building if needed) the oracle's shared library."""
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.dsbd_oracle_uniform.restype = C.c_double
        _lib.dsbd_oracle_uniform.argtypes = [C.c_uint64, C.c_uint64, C.c_uint32, C.c_uint32,
                                             C.c_uint32, C.c_uint32]
        _lib.dsbd_oracle_width_dp.restype = C.c_int32
    return _lib


def _p(a, typ):
    return a.ctypes.data_as(typ) if a is not None else typ()


def _arr(x, dtype):
    return np.ascontiguousarray(x, dtype=dtype)


def _forest(forest, keep):
    f = _Forest()
    f.R, f.B, f.N, f.max_depth = (int(forest[k]) for k in ("R", "B", "N", "max_depth"))
    for name in ("req_beam_off", "beam_node_off", "parent", "token"):
        a = _arr(forest[name], np.int32)
        keep.append(a)
        setattr(f, name, _p(a, _i32p))
    rank = forest.get("draft_rank")
    if rank is not None:
        a = _arr(rank, np.int32)
        keep.append(a)
        f.draft_rank = _p(a, _i32p)
    return f


def _params(params, R, keep):
    p = _Params()
    p.V = int(params["V"])
    p.temperature = float(params.get("temperature", 1.0))
    p.thresh = float(params.get("thresh", 0.7))
    p.W_min = int(params.get("W_min", 1))
    p.W_max = int(params.get("W_max", 1 << 30))
    p.W_nom = int(params.get("W_nom", 1))
    for name in ("W_min_r", "W_max_r", "W_nom_r", "req_id"):
        v = params.get(name)
        if v is not None:
            a = _arr(v, np.int32)
            assert a.shape == (R,)
            keep.append(a)
            setattr(p, name, _p(a, _i32p))
    p.seed = int(params.get("seed", 0))
    p.step = int(params.get("step", 0))
    p.top_k = int(params.get("top_k", 0))
    p.top_p = float(params.get("top_p", 1.0))
    return p


def philox4x32_10(ctr, key):
    c = (C.c_uint32 * 4)(*[int(x) for x in ctr])
    k = (C.c_uint32 * 2)(*[int(x) for x in key])
    o = (C.c_uint32 * 4)()
    lib().dsbd_oracle_philox4x32_10(c, k, o)
    return np.array(list(o), dtype=np.uint32)


def uniform(seed, step, request, layer, purpose, index):
    return float(lib().dsbd_oracle_uniform(seed, step, request, layer, purpose, index))


def forest_attention(forest, Hq, Hkv, d, scale, q, k_new, v_new, k_prefix, v_prefix,
                     prefix_off, threads=1):
    """O[N,Hq,d] (float64) by the definition of forest attention."""
    keep = []
    f = _forest(forest, keep)
    q, k_new, v_new = (_arr(x, np.float32) for x in (q, k_new, v_new))
    k_prefix, v_prefix = _arr(k_prefix, np.float32), _arr(v_prefix, np.float32)
    prefix_off = _arr(prefix_off, np.int64)
    N = f.N
    assert q.size == N * Hq * d and k_new.size == N * Hkv * d and v_new.size == N * Hkv * d
    assert k_prefix.size == int(prefix_off[-1]) * Hkv * d == v_prefix.size
    out = np.zeros((N, Hq, d), dtype=np.float64)
    rc = lib().dsbd_oracle_forest_attention(
        C.byref(f), C.c_int32(Hq), C.c_int32(Hkv), C.c_int32(d), C.c_double(scale),
        _p(q, _f32p), _p(k_new, _f32p), _p(v_new, _f32p), _p(k_prefix, _f32p),
        _p(v_prefix, _f32p), _p(prefix_off, _i64p), _p(out, _f64p), C.c_int32(threads))
    if rc:
        raise ValueError("oracle forest_attention: error %d" % rc)
    return out


def alpha_chain(p_beam, q_beam, m):
    p_beam, q_beam = _arr(p_beam, np.float64).ravel(), _arr(q_beam, np.float64).ravel()
    alpha = np.zeros(max(m, 1), dtype=np.float64)
    lib().dsbd_oracle_alpha_chain(_p(p_beam, _f64p), _p(q_beam, _f64p),
                                  C.c_int64(p_beam.size), C.c_int32(m), _p(alpha, _f64p))
    return alpha[:m]


def width_dp(alpha, thresh):
    """Returns (W~, P[(m+1),(m+1)], G[m+2])."""
    alpha = _arr(alpha, np.float64)
    m = alpha.size
    P = np.zeros((m + 1, m + 1), dtype=np.float64)
    G = np.zeros(m + 2, dtype=np.float64)
    a = alpha if m else np.zeros(1)
    wt = lib().dsbd_oracle_width_dp(_p(a, _f64p), C.c_int32(m), C.c_double(thresh),
                                    _p(P, _f64p), _p(G, _f64p))
    return int(wt), P, G


def default_out_off(forest, params):
    """Slot ranges large enough for any outcome: a layer's width never exceeds
    max(W_min, min(W_max, nodes of the request)) and the extra layer yields W_nom beams."""
    R = int(forest["R"])

    def per_req(name):
        v = params.get(name + "_r")
        if v is not None:
            return np.asarray(v, dtype=np.int64)
        return np.full(R, int(params.get(name, {"W_min": 1, "W_max": 1 << 30, "W_nom": 1}[name])),
                       dtype=np.int64)

    nodes = np.diff(np.asarray(forest["beam_node_off"])[np.asarray(forest["req_beam_off"])])
    cap = np.maximum(np.maximum(per_req("W_nom"), per_req("W_min")),
                     np.minimum(per_req("W_max"), nodes))
    return np.concatenate([[0], np.cumsum(cap)]).astype(np.int32)


def warp(w, top_k=0, top_p=1.0):
    """T o w: the warped copy of the joint distribution w (any shape; cells in C order)."""
    w = np.array(w, dtype=np.float64)
    flat = np.ascontiguousarray(w.ravel())
    lib().dsbd_oracle_warp(_p(flat, _f64p), C.c_int64(flat.size), C.c_int32(int(top_k)), C.c_double(float(top_p)),
                           _f64p(), _f64p())
    return flat.reshape(w.shape)


def verify_step(forest, params, logits_p, logits_q, root_logp, root_logq, out_off=None,
                inject_u=None, trace=True, dist=False, threads=1, row_stride=None):
    """One verification step for every request; returns a dict of numpy arrays."""
    keep = []
    f = _forest(forest, keep)
    R, B, N, gamma = f.R, f.B, f.N, f.max_depth
    prm = _params(params, R, keep)
    logits_p, logits_q = _arr(logits_p, np.float32), _arr(logits_q, np.float32)
    stride = int(row_stride) if row_stride is not None else prm.V
    assert logits_p.size >= (N - 1) * stride + prm.V and logits_q.size == logits_p.size
    root_logp, root_logq = _arr(root_logp, np.float64), _arr(root_logq, np.float64)
    assert root_logp.shape == (B,) and root_logq.shape == (B,)
    if out_off is None:
        out_off = default_out_off(forest, params)
    out_off = _arr(out_off, np.int32)
    S = int(out_off[-1])
    res = {
        "l_last": np.zeros(R, np.int32), "out_width": np.zeros(R, np.int32), "out_off": out_off,
        "out_parent": np.full(S, -1, np.int32), "out_node": np.full(S, -1, np.int32),
        "out_root_beam": np.full(S, -1, np.int32), "out_token": np.full(S, -1, np.int32),
        "out_logp": np.zeros(S, np.float64), "out_logq": np.zeros(S, np.float64),
        "out_source": np.full(S, -1, np.int32), "node_status": np.zeros(N, np.int8),
        "layer_width": np.full(R * (gamma + 1), -1, np.int32),
        "node_logp": np.zeros(N, np.float64), "node_logq": np.zeros(N, np.float64),
        "lse_p": np.zeros(N, np.float64), "lse_q": np.zeros(N, np.float64),
        "error": np.zeros(R, np.int32),
    }
    o = _VerifyOut()
    for name, typ in (("l_last", _i32p), ("out_width", _i32p), ("out_off", _i32p),
                      ("out_parent", _i32p), ("out_node", _i32p), ("out_root_beam", _i32p),
                      ("out_token", _i32p), ("out_logp", _f64p), ("out_logq", _f64p),
                      ("out_source", _i32p), ("node_status", _i8p), ("layer_width", _i32p),
                      ("node_logp", _f64p), ("node_logq", _f64p), ("lse_p", _f64p),
                      ("lse_q", _f64p), ("error", _i32p)):
        setattr(o, name, _p(res[name], typ))
    tlen = np.zeros(1, np.int64)
    dlen = np.zeros(1, np.int64)
    if trace:
        nodes = N
        cap = 4 * nodes + 12 * R * (gamma + 2) + int(out_off[-1]) + 64
        o.trace_cap = cap
        o.trace_len = _p(tlen, _i64p)
        for name in ("trace_req", "trace_layer", "trace_kind", "trace_index", "trace_near"):
            res[name] = np.zeros(cap, np.int32)
            setattr(o, name, _p(res[name], _i32p))
        for name in ("trace_u", "trace_a", "trace_b"):
            res[name] = np.zeros(cap, np.float64)
            setattr(o, name, _p(res[name], _f64p))
    if dist:
        max_live = int(np.max(np.diff(np.asarray(forest["beam_node_off"])[np.asarray(forest["req_beam_off"])])))
        dcap = int(out_off[-1]) * max_live * prm.V + 16
        res["dist"] = np.zeros(dcap, np.float64)
        o.dist_cap = dcap
        o.dist_len = _p(dlen, _i64p)
        o.dist = _p(res["dist"], _f64p)
    inj = None
    inj_stride = 0
    if inject_u is not None:
        inj = _arr(inject_u, np.float64).reshape(R, -1)
        inj_stride = inj.shape[1]
    rc = lib().dsbd_oracle_verify_step(
        C.byref(f), C.byref(prm), _p(logits_p, _f32p), _p(logits_q, _f32p), C.c_int64(stride),
        _p(root_logp, _f64p), _p(root_logq, _f64p), _p(inj, _f64p), C.c_int64(inj_stride),
        C.byref(o), C.c_int32(threads))
    if rc:
        raise ValueError("oracle verify_step: error %d" % rc)
    if trace:
        n = int(tlen[0])
        assert n <= o.trace_cap, "oracle trace truncated"
        for name in ("trace_req", "trace_layer", "trace_kind", "trace_index", "trace_near",
                     "trace_u", "trace_a", "trace_b"):
            res[name] = res[name][:n]
    if dist:
        n = int(dlen[0])
        assert n <= o.dist_cap, "oracle dist dump truncated"
        res["dist"] = res["dist"][:n]
    res["layer_width"] = res["layer_width"].reshape(R, gamma + 1)
    return res


def select_width(forest, params, logits_p, logits_q, node_logp, node_logq, live_off, live_nodes,
                 m, row_stride=None):
    """Width of one layer for a given live set; returns (width[R], alpha[R,mmax], tail[R,mmax+1])."""
    keep = []
    f = _forest(forest, keep)
    prm = _params(params, f.R, keep)
    logits_p, logits_q = _arr(logits_p, np.float32), _arr(logits_q, np.float32)
    stride = int(row_stride) if row_stride is not None else prm.V
    node_logp, node_logq = _arr(node_logp, np.float64), _arr(node_logq, np.float64)
    live_off, live_nodes, m = (_arr(x, np.int32) for x in (live_off, live_nodes, m))
    mmax = int(m.max()) if m.size else 0
    width = np.zeros(f.R, np.int32)
    alpha = np.zeros((f.R, mmax + 1), np.float64)
    tail = np.zeros((f.R, mmax + 1), np.float64)
    rc = lib().dsbd_oracle_select_width(
        C.byref(f), C.byref(prm), _p(logits_p, _f32p), _p(logits_q, _f32p), C.c_int64(stride),
        _p(node_logp, _f64p), _p(node_logq, _f64p), _p(live_off, _i32p), _p(live_nodes, _i32p),
        _p(m, _i32p), _p(width, _i32p), _p(alpha, _f64p), _p(tail, _f64p), C.c_int32(mmax + 1))
    if rc:
        raise ValueError("oracle select_width: error %d" % rc)
    return width, alpha[:, :mmax], tail


def draft_layer(req_beam_off, params, layer, W_S, logits_q, beam_logq, out_off=None, inject_u=None):
    """One beam-sampling step of the small model: W_S (int or [R] array) iid draws per request
    from q_beam over its current beams x V.  params: V, temperature, seed, step, top_k, top_p,
    req_id.  Returns dict(out_off, out_parent, out_token, out_logq, cdf_lo, cdf_hi, error)."""
    rbo = _arr(req_beam_off, np.int32)
    R = len(rbo) - 1
    keep = []
    p = _params(params, R, keep)
    W_r = np.full(R, int(W_S), np.int32) if np.isscalar(W_S) else _arr(W_S, np.int32)
    if out_off is None:
        out_off = np.concatenate([[0], np.cumsum(W_r)])
    out_off = _arr(out_off, np.int32)
    z = _arr(logits_q, np.float32)
    assert z.ndim == 2 and z.shape[0] == rbo[-1]
    s = _arr(beam_logq, np.float64)
    slots = int(out_off[-1])
    res = dict(out_off=out_off, out_parent=np.full(slots, -1, np.int32), out_token=np.full(slots, -1, np.int32),
               out_logq=np.zeros(slots), cdf_lo=np.zeros(slots), cdf_hi=np.zeros(slots),
               error=np.zeros(R, np.int32))
    inj, stride = None, 0
    if inject_u is not None:
        inj = _arr(inject_u, np.float64).reshape(R, -1)
        stride = inj.shape[1]
    rc = lib().dsbd_oracle_draft_layer(
        C.c_int32(R), _p(rbo, _i32p), C.byref(p), C.c_int32(int(layer)), _p(W_r, _i32p), C.c_int32(0),
        _p(z, _f32p), C.c_int64(z.shape[1]), _p(s, _f64p), _p(inj, _f64p), C.c_int64(stride),
        _p(out_off, _i32p), _p(res["out_parent"], _i32p), _p(res["out_token"], _i32p),
        _p(res["out_logq"], _f64p), _p(res["cdf_lo"], _f64p), _p(res["cdf_hi"], _f64p), _p(res["error"], _i32p))
    if rc:
        raise RuntimeError("dsbd_oracle_draft_layer: %d" % rc)
    return res
