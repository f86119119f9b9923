"""GPU parity of dsbd_forest_attention against the oracle (through the C ABI)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2409_16560_b200 as dsbd
from paper_2409_16560_b200 import inputs
from parity_util import attention_close, to_host_f32

pytestmark = pytest.mark.gpu


def _gpu(forest, spec, t, prefix_off):
    f = dsbd.Forest(forest, "cuda")
    poff = torch.as_tensor(prefix_off).cuda()
    out, status = dsbd.forest_attention(f, spec["Hq"], spec["Hkv"], spec["d"], inputs.default_scale(spec["d"]),
                                        t["q"], t["k_new"], t["v_new"], t["k_prefix"], t["v_prefix"], poff,
                                        prefix_off)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return out


def _oracle_beams(forest, spec, t, prefix_off, beams, threads=8):
    """Oracle attention of the listed trees only (their nodes, their KV prefixes)."""
    bno = np.asarray(forest["beam_node_off"])
    Hkv, d = spec["Hkv"], spec["d"]
    nodes = np.concatenate([np.arange(bno[b], bno[b + 1]) for b in beams])
    remap = np.full(forest["N"], -1, np.int64)
    remap[nodes] = np.arange(len(nodes))
    par = np.asarray(forest["parent"])[nodes]
    sub = dict(R=1, B=len(beams), N=len(nodes), max_depth=forest["max_depth"],
               req_beam_off=np.array([0, len(beams)], np.int32),
               beam_node_off=np.concatenate([[0], np.cumsum(bno[np.asarray(beams) + 1] - bno[beams])]).astype(np.int32),
               parent=np.where(par >= 0, remap[np.maximum(par, 0)], -1).astype(np.int32),
               token=np.zeros(len(nodes), np.int32))
    L = np.diff(prefix_off)[beams]
    sub_off = np.concatenate([[0], np.cumsum(L)]).astype(np.int64)
    idx = torch.as_tensor(nodes).cuda()
    kp = torch.cat([t["k_prefix"][prefix_off[b] * Hkv * d: prefix_off[b + 1] * Hkv * d] for b in beams])
    vp = torch.cat([t["v_prefix"][prefix_off[b] * Hkv * d: prefix_off[b + 1] * Hkv * d] for b in beams])
    ref = oracle.forest_attention(sub, spec["Hq"], Hkv, d, inputs.default_scale(d), to_host_f32(t["q"][idx]),
                                  to_host_f32(t["k_new"][idx]), to_host_f32(t["v_new"][idx]),
                                  to_host_f32(kp), to_host_f32(vp), sub_off, threads=threads)
    return nodes, ref


def _spread(B, n):
    """n tree ids spread evenly over 0..B-1 (all of them when n is None or >= B): the work units
    of consecutive trees go to consecutive CTAs, so an even spread meets every CTA's every round."""
    if n is None or n >= B:
        return list(range(B))
    return sorted(set(int(round(i * (B - 1) / (n - 1))) for i in range(n)))


@pytest.mark.parametrize("name,n_beams", [("C1", None), ("C2", None), ("C3", None), ("C4", 24), ("C5", 74),
                                          ("C6", None)])
def test_configs_full_size(name, n_beams):
    """The GPU runs the full configuration; the oracle checks all trees (C1-C3, C6) or an even
    spread of trees (C4: 24 of about 72, C5: 74 of 512; all nodes and heads of those trees)."""
    spec = inputs.config(name)
    t = inputs.generate(spec, "cuda", parts=("attention",))
    forest, poff = t["forest"], t["prefix_off"]
    out = _gpu(forest, spec, t, poff)
    beams = _spread(forest["B"], n_beams)
    nodes, ref = _oracle_beams(forest, spec, t, poff, beams, threads=16)
    attention_close(to_host_f32(out[torch.as_tensor(nodes).cuda()]), ref, bf16=spec["dtype"] == "bf16")
    assert torch.isfinite(out.float()).all()


def _custom(rng, trees, L, Hq, Hkv, d, dtype):
    sizes = [len(x) for x in trees]
    bno = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    parent = np.concatenate([np.where(np.array(x) >= 0, np.array(x) + bno[b], -1) for b, x in enumerate(trees)])
    N, B = int(bno[-1]), len(trees)
    forest = dict(R=1, B=B, N=N, max_depth=max(sizes), req_beam_off=np.array([0, B], np.int32),
                  beam_node_off=bno, parent=parent.astype(np.int32), token=np.zeros(N, np.int32))
    poff = np.concatenate([[0], np.cumsum(L)]).astype(np.int64)
    g = torch.Generator(device="cuda"); g.manual_seed(int(rng.integers(1 << 30)))
    mk = lambda *s: torch.randn(*s, generator=g, device="cuda").to(dtype)
    t = dict(q=mk(N, Hq, d), k_new=mk(N, Hkv, d), v_new=mk(N, Hkv, d),
             k_prefix=mk(max(int(poff[-1]) * Hkv * d, 8)), v_prefix=mk(max(int(poff[-1]) * Hkv * d, 8)))
    spec = dict(Hq=Hq, Hkv=Hkv, d=d, dtype="bf16" if dtype == torch.bfloat16 else "f32")
    return forest, spec, t, poff


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("Hq,Hkv,d", [(8, 2, 128), (4, 4, 64), (8, 1, 64)])
def test_ragged_prefixes_and_tree_shapes(dtype, Hq, Hkv, d):
    rng = np.random.default_rng(Hq * 100 + d)
    rand_tree = lambda n: [-1] + [int(rng.integers(0, i)) for i in range(1, n)]
    trees = [[-1], rand_tree(7), rand_tree(33), rand_tree(64), [-1, 0, 1, 2, 3], rand_tree(20)]
    L = [0, 1, 31, 33, 257, 1000]          # empty prefix, one token, around the tile size, ragged
    forest, spec, t, poff = _custom(rng, trees, L, Hq, Hkv, d, dtype)
    out = _gpu(forest, spec, t, poff)
    nodes, ref = _oracle_beams(forest, spec, t, poff, list(range(len(trees))))
    attention_close(to_host_f32(out), ref, bf16=dtype == torch.bfloat16)


@pytest.mark.parametrize("Hq,Hkv,max_nodes", [(8, 2, 32), (16, 2, 16), (4, 4, 64), (32, 8, 9), (40, 40, 20)])
def test_tensor_core_kernel_row_counts(Hq, Hkv, max_nodes):
    """bf16, d = 128: the tcgen05 kernel with 64-row and with 128-row query tiles (nodes x group
    up to 128), ragged prefixes around its 64-token tiles."""
    rng = np.random.default_rng(Hq * 7 + max_nodes)
    rand_tree = lambda n: [-1] + [int(rng.integers(0, i)) for i in range(1, n)]
    trees = [rand_tree(max_nodes), [-1], rand_tree(max(2, max_nodes // 2)), rand_tree(max_nodes), rand_tree(3)]
    L = [63, 64, 65, 700, 1]
    forest, spec, t, poff = _custom(rng, trees, L, Hq, Hkv, 128, torch.bfloat16)
    out = _gpu(forest, spec, t, poff)
    nodes, ref = _oracle_beams(forest, spec, t, poff, list(range(len(trees))))
    attention_close(to_host_f32(out), ref, bf16=True)


@pytest.mark.parametrize("L", [[5000, 3000], [9000]])
def test_few_units_long_prefix_is_split_and_merged(L):
    """Fewer (beam, KV head) units than CTAs: the prefix of each unit is cut into parts that
    different CTAs process, and their partial results are merged."""
    rng = np.random.default_rng(len(L))
    trees = [[-1, 0, 0, 1, 2, 2, 4][:7] for _ in L]
    forest, spec, t, poff = _custom(rng, trees, L, 8, 2, 128, torch.bfloat16)
    out = _gpu(forest, spec, t, poff)
    nodes, ref = _oracle_beams(forest, spec, t, poff, list(range(len(trees))))
    attention_close(to_host_f32(out), ref, bf16=True)


@pytest.mark.parametrize("Hq,Hkv,sizes,L", [
    (32, 2, [40, 1, 9, 64], [300, 64, 1000, 77]),        # 16 query heads per KV head: up to 1024 rows, 8 row blocks
    (16, 4, [64, 33, 5], [129, 700, 63]),                # 256 and 132 rows next to a small tree
    (8, 2, [50, 60], [6000, 4000]),                      # few units: row blocks of split units are merged
    (24, 8, [45, 2, 45, 7, 30, 64, 12, 1], [900, 100, 2500, 64, 1, 333, 1500, 4000]),   # ragged: planned order
    (8, 2, [128, 65, 100, 3], [500, 64, 1, 2000]),       # more than 64 nodes: two tiles of the tree's own K/V
    (4, 4, [127, 66], [7000, 9000]),                     # the same with split units
])
def test_trees_with_more_than_128_query_rows(Hq, Hkv, sizes, L):
    """nodes x (query heads per KV head) > 128: the tensor-core kernel cuts the tree's query rows
    into blocks of 128, each block an item of its own over the same keys and values."""
    rng = np.random.default_rng(Hq + len(L))
    rand_tree = lambda n: [-1] + [int(rng.integers(0, i)) for i in range(1, n)]
    trees = [rand_tree(n) for n in sizes]
    forest, spec, t, poff = _custom(rng, trees, L, Hq, Hkv, 128, torch.bfloat16)
    assert dsbd.forest_attention_launches(dsbd.Forest(forest, "cuda"), Hq, Hkv, 128, torch.bfloat16, 0.1, poff) >= 1
    out = _gpu(forest, spec, t, poff)
    nodes, ref = _oracle_beams(forest, spec, t, poff, list(range(len(trees))))
    attention_close(to_host_f32(out), ref, bf16=True)


def test_host_side_errors():
    rng = np.random.default_rng(0)
    forest, spec, t, poff = _custom(rng, [[-1, 0]], [8], 4, 4, 64, torch.bfloat16)
    f = dsbd.Forest(forest, "cuda")
    pd = torch.as_tensor(poff).cuda()
    with pytest.raises(dsbd.DsbdError) as e:      # head dim the kernels do not cover
        dsbd.forest_attention(f, 4, 4, 96, 0.1, t["q"], t["k_new"], t["v_new"], t["k_prefix"], t["v_prefix"], pd, poff)
    assert e.value.code == -2
    with pytest.raises(dsbd.DsbdError) as e:      # Hq not a multiple of Hkv
        dsbd.forest_attention(f, 4, 3, 64, 0.1, t["q"], t["k_new"], t["v_new"], t["k_prefix"], t["v_prefix"], pd, poff)
    assert e.value.code == -1
