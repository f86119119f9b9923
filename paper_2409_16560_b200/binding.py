"""ctypes binding of libdsbd.so: argument marshalling only.

Every step of the hot path runs in the CUDA library; this module turns torch tensors into the
device pointers of the C ABI declared in ``include/dsbd.h`` and checks return codes.  There is
no CPU fallback: without the built library, or without a CUDA device, calls raise.
"""
import ctypes as C
import os

import numpy as np
import torch

from . import build as _build

OK = 0
DTYPE_BF16, DTYPE_F32 = 0, 1
NODE_UNREACHED, NODE_ACCEPTED, NODE_REJECTED, NODE_CUT, NODE_PRUNED = 0, 1, 2, 3, 4
SRC_DRAFT, SRC_RESIDUAL, SRC_FILL, SRC_EXTRA = 0, 1, 2, 3
MAX_TREE_NODES = 64          # DSBD_MAX_TREE_NODES: the CUDA-core attention kernel
MAX_TREE_NODES_TC = 128      # DSBD_MAX_TREE_NODES_TC: the tensor-core kernel (bf16, d = 128)
MAX_LIVE = 64
REQ_STATS = 8                # DSBD_REQ_STATS: counters per request in req_stats

EXPORTS = ["dsbd_forest_attention", "dsbd_forest_attention_workspace", "dsbd_forest_attention_launches", "dsbd_verify_step",
           "dsbd_verify_workspace", "dsbd_select_width", "dsbd_node_stats", "dsbd_node_stats_static",
           "dsbd_kv_commit", "dsbd_kv_commit_workspace", "dsbd_draft_layer", "dsbd_draft_workspace",
           "dsbd_forest_attention_paged", "dsbd_forest_attention_paged_workspace", "dsbd_kv_commit_paged", "dsbd_kv_commit_paged_workspace",
           "dsbd_forest_build",
           "dsbd_status_string"]

_vp = C.c_void_p


class ForestT(C.Structure):
    _fields_ = [("R", C.c_int32), ("B", C.c_int32), ("N", C.c_int32), ("max_depth", C.c_int32),
                ("req_beam_off", _vp), ("beam_node_off", _vp), ("parent", _vp), ("token", _vp),
                ("draft_rank", _vp),
                ("max_tree_nodes", C.c_int32), ("max_req_beams", C.c_int32),
                ("max_layer_nodes", C.c_int32)]


class AttnDescT(C.Structure):
    _fields_ = [("Hq", C.c_int32), ("Hkv", C.c_int32), ("d", C.c_int32), ("dtype", C.c_int32),
                ("scale", C.c_float), ("total_prefix", C.c_int64), ("max_prefix", C.c_int64)]


class VerifyParamsT(C.Structure):
    _fields_ = [("V", C.c_int32), ("temperature", C.c_float), ("thresh", C.c_float),
                ("W_min", C.c_int32), ("W_max", C.c_int32), ("W_nom", C.c_int32),
                ("W_min_r", _vp), ("W_max_r", _vp), ("W_nom_r", _vp),
                ("seed", C.c_uint64), ("step", C.c_uint64), ("top_k", C.c_int32), ("top_p", C.c_float)]


_OUT_FIELDS = ["l_last", "out_width", "out_off", "out_parent", "out_node", "out_root_beam",
               "out_token", "out_logp", "out_logq", "out_source", "node_status", "layer_width",
               "node_logp", "node_logq", "lse_p", "lse_q", "req_error", "req_stats"]


class VerifyOutT(C.Structure):
    _fields_ = [(n, _vp) for n in _OUT_FIELDS]


_lib = None


def lib_path():
    return _build.LIB_PATH


def load():
    """Load libdsbd.so (building it when a compiler is at hand and it is missing or stale)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB_PATH
    if not os.path.exists(path) or _build.stale():
        path = _build.build()
    _lib = _declare(C.CDLL(path))
    return _lib


def use_library(path):
    """Route every call of this module through another build of the library (a measuring build
    such as the one `build.build_phase_timing()` makes).  For tools; call it before anything else."""
    global _lib
    _lib = _declare(C.CDLL(path))
    return _lib


def _declare(lib):
    lib.dsbd_status_string.restype = C.c_char_p
    lib.dsbd_status_string.argtypes = [C.c_int]
    lib.dsbd_forest_attention_workspace.restype = C.c_size_t
    lib.dsbd_forest_attention_workspace.argtypes = [_vp, _vp]
    lib.dsbd_forest_attention_launches.restype = C.c_int
    lib.dsbd_forest_attention_launches.argtypes = [_vp, _vp]
    lib.dsbd_verify_workspace.restype = C.c_size_t
    lib.dsbd_verify_workspace.argtypes = [_vp, _vp]
    lib.dsbd_forest_attention.restype = C.c_int
    lib.dsbd_forest_attention.argtypes = [_vp] * 10 + [C.c_size_t, _vp, _vp]
    lib.dsbd_verify_step.restype = C.c_int
    lib.dsbd_verify_step.argtypes = [_vp, _vp, _vp, _vp, C.c_int64, _vp, _vp, _vp, _vp, C.c_size_t,
                                     _vp, _vp]
    lib.dsbd_node_stats.restype = C.c_int
    lib.dsbd_node_stats.argtypes = [_vp, _vp, _vp, _vp, C.c_int64, _vp, _vp, _vp, C.c_size_t, _vp]
    lib.dsbd_node_stats_static.restype = C.c_int
    lib.dsbd_node_stats_static.argtypes = [_vp, _vp, _vp, _vp, C.c_int64, _vp, _vp, _vp]
    lib.dsbd_select_width.restype = C.c_int
    lib.dsbd_select_width.argtypes = [_vp, _vp, _vp, _vp, C.c_int64, _vp, _vp, _vp, _vp, _vp, _vp,
                                      _vp, _vp, C.c_int32, _vp, C.c_size_t, _vp, _vp]
    lib.dsbd_kv_commit_workspace.restype = C.c_size_t
    lib.dsbd_kv_commit_workspace.argtypes = [_vp, _vp]
    lib.dsbd_kv_commit.restype = C.c_int
    lib.dsbd_kv_commit.argtypes = [_vp] * 19 + [C.c_size_t, _vp, _vp]
    lib.dsbd_forest_attention_paged_workspace.restype = C.c_size_t
    lib.dsbd_forest_attention_paged_workspace.argtypes = [_vp, _vp, _vp]
    lib.dsbd_forest_attention_paged.restype = C.c_int
    lib.dsbd_forest_attention_paged.argtypes = [_vp] * 11 + [C.c_size_t, _vp, _vp]
    lib.dsbd_kv_commit_paged_workspace.restype = C.c_size_t
    lib.dsbd_kv_commit_paged_workspace.argtypes = [_vp, _vp, C.c_int64]
    lib.dsbd_kv_commit_paged.restype = C.c_int
    lib.dsbd_kv_commit_paged.argtypes = [_vp] * 22 + [C.c_size_t, _vp, _vp]
    lib.dsbd_forest_build.restype = C.c_int
    lib.dsbd_forest_build.argtypes = [C.c_int32, C.c_int32, C.c_int32] + [_vp] * 11
    lib.dsbd_draft_workspace.restype = C.c_size_t
    lib.dsbd_draft_workspace.argtypes = [C.c_int32, C.c_int32, _vp]
    lib.dsbd_draft_layer.restype = C.c_int
    lib.dsbd_draft_layer.argtypes = [C.c_int32, C.c_int32, _vp, _vp, _vp, C.c_int64, _vp, _vp, _vp, _vp, _vp, _vp,
                                     _vp, C.c_size_t, _vp, _vp]
    return lib


def status_string(code):
    return load().dsbd_status_string(int(code)).decode()


class DsbdError(RuntimeError):
    def __init__(self, where, code):
        super().__init__("%s: %s (%d)" % (where, status_string(code), code))
        self.code = code


def _ptr(t):
    if t is None:
        return None
    assert t.is_contiguous()
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def _require_cuda(*tensors):
    for t in tensors:
        if t is not None and not t.is_cuda:
            raise RuntimeError("dsbd: device tensors required; there is no CPU path")


def _node_depths(parent):
    """Depth of every node (roots 0) by pointer doubling: O(N log depth) array work, no Python
    loop over the nodes.  A malformed array (a cycle) ends after 32 rounds with wrong depths;
    the kernels check the forest themselves."""
    parent = np.asarray(parent, dtype=np.int64)
    jump = parent.copy()                      # ancestor 2^k levels up, -1 past the root
    depth = (parent >= 0).astype(np.int64)    # levels climbed so far
    for _ in range(32):
        live = jump >= 0
        if not live.any():
            break
        j = jump[live]
        depth[live] += depth[j]
        jump[live] = jump[j]
    return depth


class Forest:
    """Device copy of a draft forest plus the host-side facts the launches are sized by."""

    @classmethod
    def from_device(cls, R, B, N, max_depth, dev_arrays, max_tree_nodes, max_req_beams, max_layer_nodes):
        """A forest whose arrays are already on the device; the launch facts are given as bounds."""
        self = cls.__new__(cls)
        self.R, self.B, self.N, self.max_depth = int(R), int(B), int(N), int(max_depth)
        self.host = None
        self.dev = dict(dev_arrays)
        self.dev.setdefault("draft_rank", None)
        self.max_tree_nodes, self.max_req_beams = int(max_tree_nodes), int(max_req_beams)
        self.max_layer_nodes = int(max_layer_nodes)
        return self

    def __init__(self, arrays, device):
        a = {k: np.ascontiguousarray(arrays[k], dtype=np.int32)
             for k in ("req_beam_off", "beam_node_off", "parent", "token")}
        self.R, self.B, self.N = (int(arrays[k]) for k in ("R", "B", "N"))
        self.max_depth = int(arrays["max_depth"])
        self.host = a
        rank = arrays.get("draft_rank")
        self.dev = {k: torch.from_numpy(v).to(device) for k, v in a.items()}
        self.dev["draft_rank"] = (torch.from_numpy(np.ascontiguousarray(rank, dtype=np.int32)).to(device)
                                  if rank is not None else None)
        tree_sizes = np.diff(a["beam_node_off"])
        self.max_tree_nodes = int(tree_sizes.max())
        self.max_req_beams = int(np.diff(a["req_beam_off"]).max())
        # nodes per (request, depth)
        depth = _node_depths(a["parent"])
        tree_of = np.repeat(np.arange(self.B), tree_sizes)
        req_of = np.searchsorted(a["req_beam_off"], tree_of, side="right") - 1
        nz = depth > 0
        if nz.any():
            key = req_of[nz] * (int(depth.max()) + 1) + depth[nz]
            self.max_layer_nodes = int(np.bincount(key).max())
        else:
            self.max_layer_nodes = 0
        self.depth = depth
        self.tree_of = tree_of
        self.req_of = req_of
        self.device = device

    def struct(self):
        f = ForestT()
        f.R, f.B, f.N, f.max_depth = self.R, self.B, self.N, self.max_depth
        for k in ("req_beam_off", "beam_node_off", "parent", "token", "draft_rank"):
            setattr(f, k, _ptr(self.dev[k]))
        f.max_tree_nodes = self.max_tree_nodes
        f.max_req_beams = self.max_req_beams
        f.max_layer_nodes = self.max_layer_nodes
        return f


def _attn_desc(Hq, Hkv, d, dtype, scale, prefix_off_host):
    desc = AttnDescT()
    desc.Hq, desc.Hkv, desc.d = Hq, Hkv, d
    desc.dtype = DTYPE_BF16 if dtype == torch.bfloat16 else DTYPE_F32
    desc.scale = float(scale)
    desc.total_prefix = int(prefix_off_host[-1])
    desc.max_prefix = int(np.diff(prefix_off_host).max()) if len(prefix_off_host) > 1 else 0
    return desc


def forest_attention_workspace(forest, Hq, Hkv, d, dtype, scale, prefix_off_host):
    f = forest.struct()
    desc = _attn_desc(Hq, Hkv, d, dtype, scale, prefix_off_host)
    return int(load().dsbd_forest_attention_workspace(C.addressof(f), C.addressof(desc)))


def forest_attention_launches(forest, Hq, Hkv, d, dtype, scale, prefix_off_host):
    f = forest.struct()
    desc = _attn_desc(Hq, Hkv, d, dtype, scale, prefix_off_host)
    return int(load().dsbd_forest_attention_launches(C.addressof(f), C.addressof(desc)))


def forest_attention(forest, Hq, Hkv, d, scale, q, k_new, v_new, k_prefix, v_prefix, prefix_off,
                     prefix_off_host, out=None, workspace=None, status=None, stream=None):
    """dsbd_forest_attention; returns (out, status tensor)."""
    _require_cuda(q, k_new, v_new, k_prefix, v_prefix, prefix_off)
    assert q.dtype in (torch.bfloat16, torch.float32)
    f = forest.struct()
    desc = _attn_desc(Hq, Hkv, d, q.dtype, scale, prefix_off_host)
    if out is None:
        out = torch.empty_like(q)
    need = int(load().dsbd_forest_attention_workspace(C.addressof(f), C.addressof(desc)))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=q.device)
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=q.device)
    rc = load().dsbd_forest_attention(C.addressof(f), C.addressof(desc), _ptr(q), _ptr(k_new), _ptr(v_new),
                                      _ptr(k_prefix), _ptr(v_prefix), _ptr(prefix_off), _ptr(out),
                                      _ptr(workspace), workspace.numel(), _ptr(status), _stream(stream))
    if rc != OK:
        raise DsbdError("dsbd_forest_attention", rc)
    return out, status


def forest_build(req_beam_off, req_beam_off_host, gamma, W_S, draw_parent, draw_token, status=None, stream=None,
                 exact=False):
    """dsbd_forest_build.  draw_parent / draw_token: int32 device tensors [gamma, R*W_S].  Returns a
    Forest whose arrays live on the device, node_of_draw and the status tensor.  The host-side
    launch facts are the static bounds 1 + gamma*W_S nodes per tree and W_S nodes per layer; with
    exact=True the size of the largest tree is read back (4 bytes, one synchronisation of the
    stream), which lets the attention use its shape for small trees."""
    _require_cuda(req_beam_off, draw_parent, draw_token)
    dev = draw_parent.device
    rbo = np.asarray(req_beam_off_host)
    R, B = len(rbo) - 1, int(rbo[-1])
    N = B + gamma * R * W_S
    i32 = lambda n: torch.empty(n, dtype=torch.int32, device=dev)
    arrays = dict(req_beam_off=req_beam_off, beam_node_off=i32(B + 1), parent=i32(N), token=i32(N),
                  draft_rank=i32(N))
    node_of_draw = torch.empty(gamma, R * W_S, dtype=torch.int32, device=dev)
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=dev)
    largest = torch.zeros(1, dtype=torch.int32, device=dev) if exact else None
    rc = load().dsbd_forest_build(R, gamma, W_S, _ptr(req_beam_off), _ptr(draw_parent), _ptr(draw_token),
                                  _ptr(arrays["beam_node_off"]), _ptr(arrays["parent"]), _ptr(arrays["token"]),
                                  _ptr(arrays["draft_rank"]), _ptr(node_of_draw),
                                  _ptr(largest) if exact else None, _ptr(status), _stream(stream))
    if rc != OK:
        raise DsbdError("dsbd_forest_build", rc)
    f = Forest.from_device(R, B, N, gamma, arrays,
                           max_tree_nodes=int(largest.item()) if exact else 1 + gamma * W_S,
                           max_req_beams=int(np.diff(rbo).max()), max_layer_nodes=W_S)
    return f, node_of_draw, status


class KvPagesT(C.Structure):
    _fields_ = [("page_table", _vp), ("page_off", _vp), ("n_pages", C.c_int64), ("n_layers", C.c_int32),
                ("pool_layer_stride", C.c_int64), ("new_layer_stride", C.c_int64), ("q_layer_stride", C.c_int64)]


def forest_attention_paged(forest, Hq, Hkv, d, scale, q, k_new, v_new, k_pool, v_pool, page_table, page_off,
                           prefix_off, prefix_off_host, out=None, workspace=None, status=None, stream=None):
    """dsbd_forest_attention_paged; k_pool / v_pool: [n_pages, Hkv, 64, d]; returns (out, status).
    Several transformer layers in one call: pools [n_layers, n_pages, Hkv, 64, d], q [n_layers, N,
    Hq, d], k_new / v_new [n_layers, N, Hkv, d]; the leading strides are passed on as they are."""
    _require_cuda(q, k_new, v_new, k_pool, v_pool, page_table, page_off, prefix_off)
    assert page_table.dtype == torch.int32 and page_off.dtype == torch.int64
    f = forest.struct()
    desc = _attn_desc(Hq, Hkv, d, q.dtype, scale, prefix_off_host)
    pages = KvPagesT()
    pages.page_table, pages.page_off, pages.n_pages = _ptr(page_table), _ptr(page_off), int(k_pool.shape[-4])
    if out is None:
        out = torch.empty_like(q)
    if k_pool.dim() == 5:
        pages.n_layers = int(k_pool.shape[0])
        assert q.dim() == 4 and k_new.dim() == 4 and q.shape[0] == k_new.shape[0] == pages.n_layers
        assert v_pool.stride(0) == k_pool.stride(0) and v_new.stride(0) == k_new.stride(0)
        assert out.stride(0) == q.stride(0)
        pages.pool_layer_stride, pages.new_layer_stride = int(k_pool.stride(0)), int(k_new.stride(0))
        pages.q_layer_stride = int(q.stride(0))
    need = int(load().dsbd_forest_attention_paged_workspace(C.addressof(f), C.addressof(desc), C.addressof(pages)))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=q.device)
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=q.device)
    rc = load().dsbd_forest_attention_paged(C.addressof(f), C.addressof(desc), _ptr(q), _ptr(k_new), _ptr(v_new),
                                            _ptr(k_pool), _ptr(v_pool), C.addressof(pages), _ptr(prefix_off),
                                            _ptr(out), _ptr(workspace), workspace.numel(), _ptr(status),
                                            _stream(stream))
    if rc != OK:
        raise DsbdError("dsbd_forest_attention_paged", rc)
    return out, status


class DraftParamsT(C.Structure):
    _fields_ = [("V", C.c_int32), ("temperature", C.c_float), ("W_S", C.c_int32), ("W_S_r", _vp),
                ("seed", C.c_uint64), ("step", C.c_uint64), ("layer", C.c_int32), ("top_k", C.c_int32),
                ("top_p", C.c_float), ("n_slots", C.c_int32), ("max_req_beams", C.c_int32)]


def draft_layer(req_beam_off, req_beam_off_host, params, layer, W_S, logits_q, beam_logq, out_off, n_slots,
                row_stride=None, workspace=None, status=None, stream=None, out=None):
    """dsbd_draft_layer (out: the dict of an earlier call, to reuse its tensors).  req_beam_off, out_off: int32 device tensors; W_S: int or int32 device
    tensor [R]; params: V, temperature, seed, step, top_k, top_p.  Returns dict(out_parent,
    out_token, out_logq, req_error, status) on the device."""
    _require_cuda(req_beam_off, logits_q, beam_logq, out_off)
    assert logits_q.dtype == torch.float32 and beam_logq.dtype == torch.float32
    dev = logits_q.device
    rbo = np.asarray(req_beam_off_host)
    R, n_beams = len(rbo) - 1, int(rbo[-1])
    p = DraftParamsT()
    p.V = int(params["V"])
    p.temperature = float(params.get("temperature", 1.0))
    if torch.is_tensor(W_S):
        _require_cuda(W_S)
        assert W_S.dtype == torch.int32
        p.W_S, p.W_S_r = 0, _ptr(W_S)
    else:
        p.W_S = int(W_S)
    p.seed, p.step, p.layer = int(params.get("seed", 0)), int(params.get("step", 0)), int(layer)
    p.top_k, p.top_p = int(params.get("top_k", 0)), float(params.get("top_p", 1.0))
    p.n_slots = int(n_slots)
    p.max_req_beams = int(np.diff(rbo).max())
    need = int(load().dsbd_draft_workspace(R, n_beams, C.addressof(p)))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=dev)
    res = out if out is not None else dict(
        out_parent=torch.full((int(n_slots),), -1, dtype=torch.int32, device=dev),
        out_token=torch.full((int(n_slots),), -1, dtype=torch.int32, device=dev),
        out_logq=torch.zeros(int(n_slots), dtype=torch.float32, device=dev),
        req_error=torch.zeros(R, dtype=torch.int32, device=dev))
    res["status"], res["workspace"] = status, workspace
    stride = int(row_stride) if row_stride is not None else int(logits_q.stride(0))
    rc = load().dsbd_draft_layer(R, n_beams, _ptr(req_beam_off), C.addressof(p), _ptr(logits_q), stride,
                                 _ptr(beam_logq), _ptr(out_off), _ptr(res["out_parent"]), _ptr(res["out_token"]),
                                 _ptr(res["out_logq"]), _ptr(res["req_error"]), _ptr(workspace), workspace.numel(),
                                 _ptr(status), _stream(stream))
    if rc != OK:
        raise DsbdError("dsbd_draft_layer", rc)
    return res


class CommitParamsT(C.Structure):
    _fields_ = [("n_slots", C.c_int32), ("keep_best", C.c_int32), ("dst_capacity", C.c_int64),
                ("n_layers", C.c_int32), ("pool_layer_stride", C.c_int64), ("new_layer_stride", C.c_int64)]


def kv_commit(forest, Hkv, d, out_off, out_width, out_parent, out_root_beam, out_logp, k_new, v_new,
              k_prefix, v_prefix, prefix_off, prefix_off_host, n_slots, dst_capacity, keep_best=False,
              k_dst=None, v_dst=None, workspace=None, status=None, stream=None, out=None):
    """dsbd_kv_commit; returns a dict with k_dst, v_dst, new_req_beam_off, new_prefix_off,
    new_beam_slot and the status tensor (all on the device, nothing is synchronised)."""
    _require_cuda(out_off, out_width, out_parent, out_root_beam, k_new, v_new, k_prefix, v_prefix, prefix_off)
    dev = k_new.device
    f = forest.struct()
    desc = _attn_desc(Hkv, Hkv, d, k_new.dtype, 1.0, prefix_off_host)
    p = CommitParamsT()
    p.n_slots, p.keep_best, p.dst_capacity = int(n_slots), int(bool(keep_best)), int(dst_capacity)
    if k_dst is None:
        k_dst = torch.empty(int(dst_capacity) * Hkv * d, dtype=k_new.dtype, device=dev)
    if v_dst is None:
        v_dst = torch.empty(int(dst_capacity) * Hkv * d, dtype=k_new.dtype, device=dev)
    need = int(load().dsbd_kv_commit_workspace(C.addressof(f), C.addressof(p)))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=dev)
    if out is not None:
        new_req_beam_off, new_prefix_off, new_beam_slot = (out[k] for k in ("new_req_beam_off", "new_prefix_off",
                                                                              "new_beam_slot"))
    else:
        new_req_beam_off = torch.empty(forest.R + 1, dtype=torch.int32, device=dev)
        new_prefix_off = torch.empty(int(n_slots) + 1, dtype=torch.int64, device=dev)
        new_beam_slot = torch.empty(int(n_slots), dtype=torch.int32, device=dev)
    rc = load().dsbd_kv_commit(C.addressof(f), C.addressof(desc), C.addressof(p), _ptr(out_off), _ptr(out_width),
                               _ptr(out_parent), _ptr(out_root_beam), _ptr(out_logp) if out_logp is not None else None,
                               _ptr(k_new), _ptr(v_new), _ptr(k_prefix), _ptr(v_prefix), _ptr(prefix_off),
                               _ptr(k_dst), _ptr(v_dst), _ptr(new_req_beam_off), _ptr(new_prefix_off),
                               _ptr(new_beam_slot), _ptr(workspace), workspace.numel(), _ptr(status),
                               _stream(stream))
    if rc != OK:
        raise DsbdError("dsbd_kv_commit", rc)
    return dict(k_dst=k_dst, v_dst=v_dst, new_req_beam_off=new_req_beam_off, new_prefix_off=new_prefix_off,
                new_beam_slot=new_beam_slot, status=status, workspace=workspace)


def kv_commit_paged(forest, Hkv, d, out_off, out_width, out_parent, out_root_beam, out_logp, k_new, v_new,
                    k_pool, v_pool, page_table, page_off, prefix_off, prefix_off_host, free_stack, free_count,
                    n_slots, table_capacity, keep_best=False, workspace=None, status=None, stream=None, out=None):
    """dsbd_kv_commit_paged; the pools, free_stack and free_count are updated in place.  Pools of
    shape [n_layers, n_pages, Hkv, 64, d] with k_new / v_new [n_layers, N, Hkv, d] update all
    layers in one call (the layers share the page tables).  Returns a
    dict with new_req_beam_off, new_prefix_off, new_page_off, new_page_table, new_beam_slot and the
    status tensor (device tensors, nothing is synchronised)."""
    _require_cuda(out_off, out_width, out_parent, out_root_beam, k_new, v_new, k_pool, v_pool, page_table,
                  page_off, prefix_off, free_stack, free_count)
    dev = k_new.device
    f = forest.struct()
    desc = _attn_desc(Hkv, Hkv, d, k_new.dtype, 1.0, prefix_off_host)
    p = CommitParamsT()
    p.n_slots, p.keep_best, p.dst_capacity = int(n_slots), int(bool(keep_best)), int(table_capacity)
    pages = KvPagesT()
    if k_pool.dim() == 5:
        p.n_layers = int(k_pool.shape[0])
        p.pool_layer_stride = int(k_pool.stride(0))
        p.new_layer_stride = int(k_new.stride(0))
        assert k_new.dim() == 4 and k_new.shape[0] == p.n_layers
    pages.page_table, pages.page_off = _ptr(page_table), _ptr(page_off)
    pages.n_pages = int(k_pool.shape[-4])
    need = int(load().dsbd_kv_commit_paged_workspace(C.addressof(f), C.addressof(p), pages.n_pages))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=dev)
    res = out if out is not None else dict(
        new_req_beam_off=torch.empty(forest.R + 1, dtype=torch.int32, device=dev),
        new_prefix_off=torch.empty(int(n_slots) + 1, dtype=torch.int64, device=dev),
        new_page_off=torch.empty(int(n_slots) + 1, dtype=torch.int64, device=dev),
        new_page_table=torch.full((int(table_capacity),), -1, dtype=torch.int32, device=dev),
        new_beam_slot=torch.empty(int(n_slots), dtype=torch.int32, device=dev))
    res["status"], res["workspace"] = status, workspace
    rc = load().dsbd_kv_commit_paged(
        C.addressof(f), C.addressof(desc), C.addressof(p), _ptr(out_off), _ptr(out_width), _ptr(out_parent),
        _ptr(out_root_beam), _ptr(out_logp) if out_logp is not None else None, _ptr(k_new), _ptr(v_new),
        _ptr(k_pool), _ptr(v_pool), C.addressof(pages), _ptr(prefix_off), _ptr(free_stack), _ptr(free_count),
        _ptr(res["new_req_beam_off"]), _ptr(res["new_prefix_off"]), _ptr(res["new_page_off"]),
        _ptr(res["new_page_table"]), _ptr(res["new_beam_slot"]), _ptr(workspace), workspace.numel(), _ptr(status),
        _stream(stream))
    if rc != OK:
        raise DsbdError("dsbd_kv_commit_paged", rc)
    return res


def _params(params, keep):
    p = VerifyParamsT()
    p.V = int(params["V"])
    p.temperature = float(params.get("temperature", 1.0))
    p.thresh = float(params.get("thresh", 0.7))
    p.W_min = int(params.get("W_min", 1))
    p.W_max = int(params.get("W_max", 1 << 30))
    p.W_nom = int(params.get("W_nom", 1))
    for name in ("W_min_r", "W_max_r", "W_nom_r"):
        t = params.get(name)
        if t is not None:
            _require_cuda(t)
            assert t.dtype == torch.int32
            keep.append(t)
            setattr(p, name, _ptr(t))
    p.seed = int(params.get("seed", 0))
    p.step = int(params.get("step", 0))
    p.top_k = int(params.get("top_k", 0))
    p.top_p = float(params.get("top_p", 1.0))
    return p


def verify_workspace(forest, params):
    keep = []
    f = forest.struct()
    p = _params(params, keep)
    return int(load().dsbd_verify_workspace(C.addressof(f), C.addressof(p)))


def default_out_off(arrays, params):
    """Output slot ranges that hold any outcome: max(W_nom, W_min, min(W_max, nodes)) per request."""
    R = int(arrays["R"])
    nodes = np.diff(np.asarray(arrays["beam_node_off"])[np.asarray(arrays["req_beam_off"])])

    def per_request(name, default):
        v = params.get(name + "_r")
        if v is not None:
            return np.asarray(v.cpu() if torch.is_tensor(v) else v, dtype=np.int64)
        return np.full(R, int(params.get(name, default)), dtype=np.int64)

    cap = np.maximum(np.maximum(per_request("W_nom", 1), per_request("W_min", 1)),
                     np.minimum(per_request("W_max", 1 << 30), nodes))
    return np.concatenate([[0], np.cumsum(cap)]).astype(np.int32)


def alloc_verify_out(forest, out_off_host, device):
    """Output buffers of dsbd_verify_step as a dict of device tensors."""
    R, N, g = forest.R, forest.N, forest.max_depth
    S = int(out_off_host[-1])
    i32, f32 = torch.int32, torch.float32
    o = {
        "l_last": torch.zeros(R, dtype=i32, device=device),
        "out_width": torch.zeros(R, dtype=i32, device=device),
        "out_off": torch.from_numpy(np.ascontiguousarray(out_off_host, dtype=np.int32)).to(device),
        "out_parent": torch.full((S,), -1, dtype=i32, device=device),
        "out_node": torch.full((S,), -1, dtype=i32, device=device),
        "out_root_beam": torch.full((S,), -1, dtype=i32, device=device),
        "out_token": torch.full((S,), -1, dtype=i32, device=device),
        "out_logp": torch.zeros(S, dtype=f32, device=device),
        "out_logq": torch.zeros(S, dtype=f32, device=device),
        "out_source": torch.full((S,), -1, dtype=i32, device=device),
        "node_status": torch.zeros(N, dtype=torch.int8, device=device),
        "layer_width": torch.full((R * (g + 1),), -1, dtype=i32, device=device),
        "node_logp": torch.zeros(N, dtype=f32, device=device),
        "node_logq": torch.zeros(N, dtype=f32, device=device),
        "lse_p": torch.zeros(N, dtype=f32, device=device),
        "lse_q": torch.zeros(N, dtype=f32, device=device),
        "req_error": torch.zeros(R, dtype=i32, device=device),
        "req_stats": torch.zeros(R * REQ_STATS, dtype=i32, device=device),
    }
    return o


def verify_step(forest, params, logits_p, logits_q, root_logp, root_logq, out, workspace=None,
                status=None, stream=None, row_stride=None):
    """dsbd_verify_step; `out` from alloc_verify_out.  Returns the status tensor."""
    _require_cuda(logits_p, logits_q, root_logp, root_logq)
    assert logits_p.dtype == torch.float32 and logits_q.dtype == torch.float32
    keep = []
    f = forest.struct()
    p = _params(params, keep)
    o = VerifyOutT()
    for name in _OUT_FIELDS:
        setattr(o, name, _ptr(out[name]))
    need = int(load().dsbd_verify_workspace(C.addressof(f), C.addressof(p)))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=logits_p.device)
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=logits_p.device)
    stride = int(row_stride) if row_stride is not None else logits_p.stride(0)
    rc = load().dsbd_verify_step(C.addressof(f), C.addressof(p), _ptr(logits_p), _ptr(logits_q), stride,
                                 _ptr(root_logp), _ptr(root_logq), C.addressof(o), _ptr(workspace),
                                 workspace.numel(), _ptr(status), _stream(stream))
    if rc != OK:
        raise DsbdError("dsbd_verify_step", rc)
    return status


def node_stats(forest, params, logits_p, logits_q, lse_p=None, lse_q=None, workspace=None, stream=None):
    """dsbd_node_stats; returns (lse_p[N], lse_q[N])."""
    _require_cuda(logits_p, logits_q)
    keep = []
    f = forest.struct()
    p = _params(params, keep)
    dev = logits_p.device
    if lse_p is None:
        lse_p = torch.empty(forest.N, dtype=torch.float32, device=dev)
    if lse_q is None:
        lse_q = torch.empty(forest.N, dtype=torch.float32, device=dev)
    need = int(load().dsbd_verify_workspace(C.addressof(f), C.addressof(p)))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
    rc = load().dsbd_node_stats(C.addressof(f), C.addressof(p), _ptr(logits_p), _ptr(logits_q),
                                logits_p.stride(0), _ptr(lse_p), _ptr(lse_q), _ptr(workspace),
                                workspace.numel(), _stream(stream))
    if rc != OK:
        raise DsbdError("dsbd_node_stats", rc)
    return lse_p, lse_q


STATIC_SCRATCH_BYTES = 8 << 20


def node_stats_static(forest, params, logits_p, logits_q, lse_p, lse_q, stream=None):
    """dsbd_node_stats_static: dsbd_node_stats without a workspace, for callers that cannot
    allocate device memory; the outputs lse_p, lse_q ([N] fp32 each) are the caller's.  The
    binding itself allocates nothing either.  Problems that need more than
    STATIC_SCRATCH_BYTES of scratch raise DsbdError (workspace too small).  Calls share one
    scratch array per GPU: do not let two of them overlap on the device."""
    _require_cuda(logits_p, logits_q, lse_p, lse_q)
    keep = []
    f = forest.struct()
    p = _params(params, keep)
    rc = load().dsbd_node_stats_static(C.addressof(f), C.addressof(p), _ptr(logits_p), _ptr(logits_q),
                                       logits_p.stride(0), _ptr(lse_p), _ptr(lse_q), _stream(stream))
    if rc != OK:
        raise DsbdError("dsbd_node_stats_static", rc)
    return lse_p, lse_q


def select_width(forest, params, logits_p, logits_q, node_logp, node_logq, live_off, live_nodes, m,
                 out_stride, workspace=None, status=None, stream=None, want_alpha=True):
    """dsbd_select_width; returns (width[R], alpha[R,out_stride], tail[R,out_stride], status)."""
    _require_cuda(logits_p, logits_q, node_logp, node_logq, live_off, live_nodes, m)
    keep = []
    f = forest.struct()
    p = _params(params, keep)
    dev = logits_p.device
    width = torch.zeros(forest.R, dtype=torch.int32, device=dev)
    alpha = torch.zeros(forest.R, out_stride, dtype=torch.float32, device=dev) if want_alpha else None
    tail = torch.zeros(forest.R, out_stride, dtype=torch.float32, device=dev) if want_alpha else None
    need = int(load().dsbd_verify_workspace(C.addressof(f), C.addressof(p)))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
    if status is None:
        status = torch.zeros(1, dtype=torch.int32, device=dev)
    rc = load().dsbd_select_width(C.addressof(f), C.addressof(p), _ptr(logits_p), _ptr(logits_q),
                                  logits_p.stride(0), _ptr(node_logp), _ptr(node_logq), _ptr(live_off),
                                  _ptr(live_nodes), _ptr(m), _ptr(width), _ptr(alpha), _ptr(tail),
                                  int(out_stride), _ptr(workspace), workspace.numel(), _ptr(status),
                                  _stream(stream))
    if rc != OK:
        raise DsbdError("dsbd_select_width", rc)
    return width, alpha, tail, status
