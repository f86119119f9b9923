"""GPU parity of the paged KV-cache path: dsbd_forest_attention_paged against the oracle's
attention on the same caches (the pages are cut from the packed caches on the host, with
shuffled page ids), and dsbd_kv_commit_paged against the paged oracle."""
import numpy as np
import pytest
import torch

from oracle import kv_paged as kvp
import paper_2409_16560_b200 as dsbd
from paper_2409_16560_b200 import inputs
from parity_util import attention_close, to_host_f32
from test_gpu_attention import _custom, _oracle_beams

pytestmark = pytest.mark.gpu


def _bits(t):
    t = t.detach().cpu().contiguous()
    return t.view(torch.int16 if t.element_size() == 2 else torch.int32).numpy().reshape(-1)


def _from_bits(a, dtype):
    return torch.from_numpy(np.ascontiguousarray(a)).view(dtype)


def _paged(t, poff, Hkv, d, extra_pages, rng):
    need = int(sum(-(-int(l) // kvp.PAGE) for l in np.diff(poff)))
    n = int(poff[-1]) * Hkv * d
    kpool, vpool, table, page_off, free, nfree = kvp.pack_into_pages(
        _bits(t["k_prefix"])[:n], _bits(t["v_prefix"])[:n], poff, Hkv, d, need + extra_pages, rng)
    dt = t["k_prefix"].dtype
    return dict(k_pool=_from_bits(kpool, dt).cuda(), v_pool=_from_bits(vpool, dt).cuda(),
                table=torch.as_tensor(table).cuda(), page_off=torch.as_tensor(page_off).cuda(),
                free=free, nfree=nfree, host=(kpool, vpool, table, page_off))


def _gpu_paged(forest, spec, t, poff, pg):
    f = dsbd.Forest(forest, "cuda")
    out, st = dsbd.forest_attention_paged(f, spec["Hq"], spec["Hkv"], spec["d"], inputs.default_scale(spec["d"]),
                                          t["q"], t["k_new"], t["v_new"], pg["k_pool"], pg["v_pool"], pg["table"],
                                          pg["page_off"], torch.as_tensor(poff).cuda(), poff)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    return out


@pytest.mark.parametrize("name,kw,n_beams", [("C2", {}, None), ("C3", {}, 3), ("C4", {}, 4), ("C5", dict(R=3), 2),
                                             ("C6", {}, 8)])
def test_paged_attention_configs(name, kw, n_beams):
    spec = inputs.config(name, **kw)
    t = inputs.generate(spec, "cuda", parts=("attention",))
    forest, poff = t["forest"], t["prefix_off"]
    pg = _paged(t, poff, spec["Hkv"], spec["d"], 5, np.random.default_rng(1))
    out = _gpu_paged(forest, spec, t, poff, pg)
    beams = list(range(forest["B"])) if n_beams is None else \
        sorted(np.random.default_rng(2).choice(forest["B"], size=n_beams, replace=False).tolist())
    nodes, ref = _oracle_beams(forest, spec, t, poff, beams)
    attention_close(to_host_f32(out[torch.as_tensor(nodes).cuda()]), ref, bf16=True)
    assert torch.isfinite(out.float()).all()


@pytest.mark.parametrize("L", [[1, 63, 64, 65, 700], [5000, 3000, 128, 129, 2]])
def test_partial_pages_and_split_units(L):
    rng = np.random.default_rng(len(L) + L[0])
    rand_tree = lambda n: [-1] + [int(rng.integers(0, i)) for i in range(1, n)]
    trees = [rand_tree(9), [-1], rand_tree(16), rand_tree(5), rand_tree(2)]
    forest, spec, t, poff = _custom(rng, trees, L, 8, 2, 128, torch.bfloat16)
    pg = _paged(t, poff, 2, 128, 4, rng)
    out = _gpu_paged(forest, spec, t, poff, pg)
    nodes, ref = _oracle_beams(forest, spec, t, poff, list(range(len(trees))))
    attention_close(to_host_f32(out), ref, bf16=True)


def test_paged_attention_with_row_blocks():
    rng = np.random.default_rng(12)
    rand_tree = lambda n: [-1] + [int(rng.integers(0, i)) for i in range(1, n)]
    trees = [rand_tree(64), rand_tree(3), rand_tree(40), rand_tree(101)]
    L = [200, 4000, 65, 130]
    forest, spec, t, poff = _custom(rng, trees, L, 16, 2, 128, torch.bfloat16)        # up to 512 query rows
    pg = _paged(t, poff, 2, 128, 4, rng)
    out = _gpu_paged(forest, spec, t, poff, pg)
    nodes, ref = _oracle_beams(forest, spec, t, poff, list(range(len(trees))))
    attention_close(to_host_f32(out), ref, bf16=True)


@pytest.mark.parametrize("L,sizes,Hq,Hkv,n_layers", [
    ([700, 64, 65, 130, 1], [9, 1, 16, 5, 2], 8, 2, 3),       # 64-row tile, units in plain order
    ([6000, 4000], [7, 7], 8, 2, 4),                          # few units: split prefixes, merged per layer
    ([900, 100, 2500, 64, 333], [45, 2, 30, 64, 12], 16, 4, 2),   # row blocks and a planned order
    ([300, 200, 257, 40], [5, 5, 5, 5], 40, 40, 5),           # 40 heads of 128 (the Llama-2-13B shape)
])
def test_attention_of_several_layers_in_one_call(L, sizes, Hq, Hkv, n_layers):
    """All transformer layers of a step in one launch: every layer has its own pools, new
    keys/values and queries, all share the forest and the page tables.  Each layer must match the
    oracle's attention on that layer's caches."""
    rng = np.random.default_rng(n_layers * 10 + len(L))
    rand_tree = lambda n: [-1] + [int(rng.integers(0, i)) for i in range(1, n)]
    trees = [rand_tree(n) for n in sizes]
    layers = [_custom(rng, trees, L, Hq, Hkv, 128, torch.bfloat16) for _ in range(n_layers)]
    forest, spec, _, poff = layers[0]
    pgs = [_paged(t, poff, Hkv, 128, 4, np.random.default_rng(5)) for _, _, t, _ in layers]   # same page ids
    assert all(torch.equal(pg["table"], pgs[0]["table"]) for pg in pgs)
    stack = lambda key: torch.stack([t[key] for _, _, t, _ in layers]).contiguous()
    k_pool = torch.stack([pg["k_pool"] for pg in pgs]).contiguous()
    v_pool = torch.stack([pg["v_pool"] for pg in pgs]).contiguous()
    f = dsbd.Forest(forest, "cuda")
    out, st = dsbd.forest_attention_paged(f, Hq, Hkv, 128, inputs.default_scale(128), stack("q"), stack("k_new"),
                                          stack("v_new"), k_pool, v_pool, pgs[0]["table"], pgs[0]["page_off"],
                                          torch.as_tensor(poff).cuda(), poff)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    for l, (_, _, t, _) in enumerate(layers):
        nodes, ref = _oracle_beams(forest, spec, t, poff, list(range(len(trees))))
        attention_close(to_host_f32(out[l]), ref, bf16=True)
        # and bit for bit what a call for this layer alone gives
        single = _gpu_paged(forest, spec, t, poff, pgs[l])
        assert torch.equal(single, out[l])


def test_layer_strides_are_validated():
    """A layer stride that is not a whole number of tensor-map rows, or shorter than one layer's
    tensor, is refused before anything is launched (the workspace query answers 0)."""
    import ctypes as C
    from paper_2409_16560_b200 import binding as bd
    rng = np.random.default_rng(3)
    forest, spec, t, poff = _custom(rng, [[-1, 0]], [100], 8, 2, 128, torch.bfloat16)
    pg = _paged(t, poff, 2, 128, 1, rng)
    f = dsbd.Forest(forest, "cuda").struct()
    desc = bd._attn_desc(8, 2, 128, torch.bfloat16, 0.1, poff)
    n_pages = int(pg["k_pool"].shape[0])
    pool, new, q = n_pages * 2 * 64 * 128, forest["N"] * 2 * 128, forest["N"] * 8 * 128

    def query(n_layers, ps, ns, qs):
        pages = bd.KvPagesT()
        pages.page_table, pages.page_off, pages.n_pages = bd._ptr(pg["table"]), bd._ptr(pg["page_off"]), n_pages
        pages.n_layers, pages.pool_layer_stride, pages.new_layer_stride, pages.q_layer_stride = n_layers, ps, ns, qs
        return int(bd.load().dsbd_forest_attention_paged_workspace(C.addressof(f), C.addressof(desc),
                                                                   C.addressof(pages)))
    assert query(2, pool, new, q) > 0
    assert query(1, 0, 0, 0) > 0                      # one layer: strides ignored
    assert query(2, pool + 64, new, q) == 0           # not a whole 64-token page row
    assert query(2, pool - 64 * 128, new, q) == 0     # layers would overlap
    assert query(2, pool, new + 128, q) == 0          # not a whole row of the new keys
    assert query(2, pool, new, q - 8) == 0
    assert query(-1, pool, new, q) == 0


def test_unsupported_shapes_are_refused():
    rng = np.random.default_rng(0)
    forest, spec, t, poff = _custom(rng, [[-1, 0]], [100], 4, 4, 64, torch.float32)
    pg = _paged(t, poff, 4, 64, 1, rng)
    with pytest.raises(dsbd.DsbdError):
        dsbd.forest_attention_paged(dsbd.Forest(forest, "cuda"), 4, 4, 64, 0.125, t["q"], t["k_new"], t["v_new"],
                                    pg["k_pool"], pg["v_pool"], pg["table"], pg["page_off"],
                                    torch.as_tensor(poff).cuda(), poff)


def _forest_on(rng, req_beam_off, max_nodes):
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
    return out_off, out_width, out_parent, out_root, (rng.normal(size=R * width) - 9).astype(np.float32)


@pytest.mark.parametrize("dtype,Hkv,d", [(torch.bfloat16, 4, 128), (torch.float32, 2, 64)])
def test_paged_commit_over_several_steps(dtype, Hkv, d):
    """Six decode steps of cache updates on the device against the paged oracle on the host:
    tables, offsets and allocator state bit for bit; the pools through what they mean (the
    gathered caches); at the end the paged attention runs on the device's state."""
    rng = np.random.default_rng(7)
    rbo = np.array([0, 2, 3, 6, 7], np.int32)
    L = [100, 100, 63, 700, 700, 700, 64]
    poff = np.concatenate([[0], np.cumsum(L)]).astype(np.int64)
    n_pages = 60
    g = torch.Generator(device="cuda"); g.manual_seed(1)
    mk = lambda *s: torch.randn(*s, generator=g, device="cuda").to(dtype)
    kp, vp = mk(int(poff[-1]) * Hkv * d), mk(int(poff[-1]) * Hkv * d)
    hk, hv, table, page_off, free, nfree = kvp.pack_into_pages(_bits(kp), _bits(vp), poff, Hkv, d, n_pages, rng)
    dk, dv = _from_bits(hk, dtype).cuda(), _from_bits(hv, dtype).cuda()
    d_table, d_page_off = torch.as_tensor(table).cuda(), torch.as_tensor(page_off).cuda()
    d_free, d_nfree = torch.as_tensor(free).cuda(), torch.tensor([nfree], dtype=torch.int32, device="cuda")
    i32 = lambda a: torch.as_tensor(np.asarray(a, np.int32)).cuda()
    for step in range(6):
        forest = _forest_on(rng, rbo, 6)
        kn, vn = mk(forest["N"], Hkv, d), mk(forest["N"], Hkv, d)
        outs = _outputs(rng, forest, 3)
        keep_best = step == 3
        ref = kvp.kv_commit_paged(forest, *outs, _bits(kn), _bits(vn), hk, hv, table, page_off, poff, free, nfree,
                                  keep_best=keep_best)
        assert ref["error"] == 0
        res = dsbd.kv_commit_paged(dsbd.Forest(forest, "cuda"), Hkv, d, i32(outs[0]), i32(outs[1]), i32(outs[2]),
                                   i32(outs[3]), torch.as_tensor(outs[4]).cuda(), kn, vn, dk, dv, d_table,
                                   d_page_off, torch.as_tensor(poff).cuda(), poff, d_free, d_nfree,
                                   n_slots=int(outs[0][-1]), table_capacity=len(ref["new_page_table"]) + 3,
                                   keep_best=keep_best)
        torch.cuda.synchronize()
        assert int(res["status"].item()) == 0
        nb = len(ref["new_beam_slot"])
        assert np.array_equal(res["new_req_beam_off"].cpu().numpy(), ref["new_req_beam_off"])
        assert np.array_equal(res["new_prefix_off"].cpu().numpy()[:nb + 1], ref["new_prefix_off"])
        assert np.array_equal(res["new_page_off"].cpu().numpy()[:nb + 1], ref["new_page_off"])
        nt = len(ref["new_page_table"])
        assert np.array_equal(res["new_page_table"].cpu().numpy()[:nt], ref["new_page_table"])
        assert np.array_equal(res["new_beam_slot"].cpu().numpy()[:nb], ref["new_beam_slot"])
        assert int(d_nfree.item()) == ref["free_count"]
        assert np.array_equal(d_free.cpu().numpy()[:ref["free_count"]], ref["free_stack"][:ref["free_count"]])
        gk, gv = kvp.gather(_bits(dk).reshape(hk.shape), _bits(dv).reshape(hv.shape), ref["new_page_table"],
                            ref["new_page_off"], ref["new_prefix_off"])
        wk, wv = kvp.gather(ref["k_pool"], ref["v_pool"], ref["new_page_table"], ref["new_page_off"],
                            ref["new_prefix_off"])
        assert np.array_equal(gk, wk) and np.array_equal(gv, wv)
        assert torch.isfinite(dk.float()).all() and torch.isfinite(dv.float()).all()
        rbo, poff = ref["new_req_beam_off"], ref["new_prefix_off"]
        hk, hv, table, page_off = ref["k_pool"], ref["v_pool"], ref["new_page_table"], ref["new_page_off"]
        free, nfree = ref["free_stack"], ref["free_count"]
        d_table = res["new_page_table"][:nt].contiguous()
        d_page_off = res["new_page_off"][:nb + 1].contiguous()
    if dtype == torch.bfloat16:
        forest = _forest_on(rng, rbo, 6)
        Hq = 2 * Hkv
        t = dict(q=mk(forest["N"], Hq, d), k_new=mk(forest["N"], Hkv, d), v_new=mk(forest["N"], Hkv, d))
        out, st = dsbd.forest_attention_paged(dsbd.Forest(forest, "cuda"), Hq, Hkv, d, inputs.default_scale(d),
                                              t["q"], t["k_new"], t["v_new"], dk, dv, d_table, d_page_off,
                                              torch.as_tensor(poff).cuda(), poff)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        wk, wv = kvp.gather(hk, hv, table, page_off, poff)
        t["k_prefix"], t["v_prefix"] = _from_bits(wk, dtype).cuda(), _from_bits(wv, dtype).cuda()
        nodes, ref = _oracle_beams(forest, dict(Hq=Hq, Hkv=Hkv, d=d), t, poff, list(range(forest["B"])))
        attention_close(to_host_f32(out), ref, bf16=True)


def test_paged_commit_without_free_pages_changes_nothing():
    rng = np.random.default_rng(9)
    Hkv, d = 2, 64
    rbo, poff = np.array([0, 1], np.int32), np.array([0, 10], np.int64)
    kp = torch.randn(10 * Hkv * d, device="cuda")
    hk, hv, table, page_off, free, nfree = kvp.pack_into_pages(_bits(kp), _bits(kp), poff, Hkv, d, 2)
    dk, dv = _from_bits(hk, torch.float32).cuda(), _from_bits(hv, torch.float32).cuda()
    forest = _forest_on(rng, rbo, 2)
    kn = torch.randn(forest["N"], Hkv, d, device="cuda")
    i32 = lambda a: torch.as_tensor(np.asarray(a, np.int32)).cuda()
    d_free, d_nfree = torch.as_tensor(free).cuda(), torch.tensor([nfree], dtype=torch.int32, device="cuda")
    before = dk.clone()
    res = dsbd.kv_commit_paged(dsbd.Forest(forest, "cuda"), Hkv, d, i32([0, 2]), i32([2]), i32([0, 0]), i32([0, 0]),
                               None, kn, kn, dk, dv, torch.as_tensor(table).cuda(), torch.as_tensor(page_off).cuda(),
                               torch.as_tensor(poff).cuda(), poff, d_free, d_nfree, n_slots=2, table_capacity=8)
    torch.cuda.synchronize()
    assert int(res["status"].item()) == 3
    assert torch.equal(dk, before) and int(d_nfree.item()) == nfree
    assert np.array_equal(d_free.cpu().numpy(), free)


def test_paged_commit_of_several_layers_shares_the_tables():
    """Three transformer layers: one call, one plan, one set of page tables; every layer's pools
    must gather to what the oracle gives for that layer alone."""
    rng = np.random.default_rng(21)
    Hkv, d, n_layers, n_pages = 2, 128, 3, 40
    rbo = np.array([0, 2, 5], np.int32)
    L = [70, 70, 200, 200, 200]
    poff = np.concatenate([[0], np.cumsum(L)]).astype(np.int64)
    g = torch.Generator(device="cuda"); g.manual_seed(2)
    mk = lambda *s: torch.randn(*s, generator=g, device="cuda").to(torch.bfloat16)
    forest = _forest_on(rng, rbo, 5)
    outs = _outputs(rng, forest, 3)
    hosts, dks, dvs, kns, vns = [], [], [], [], []
    ids = rng.permutation(n_pages)
    for layer in range(n_layers):
        kp, vp = mk(int(poff[-1]) * Hkv * d), mk(int(poff[-1]) * Hkv * d)
        # the same page ids in every layer: seed the shuffle identically
        hk, hv, table, page_off, free, nfree = kvp.pack_into_pages(_bits(kp), _bits(vp), poff, Hkv, d, n_pages,
                                                                   np.random.default_rng(77))
        hosts.append((hk, hv))
        dks.append(_from_bits(hk, torch.bfloat16)); dvs.append(_from_bits(hv, torch.bfloat16))
        kns.append(mk(forest["N"], Hkv, d)); vns.append(mk(forest["N"], Hkv, d))
    dk, dv = torch.stack(dks).cuda(), torch.stack(dvs).cuda()
    kn, vn = torch.stack(kns), torch.stack(vns)
    i32 = lambda a: torch.as_tensor(np.asarray(a, np.int32)).cuda()
    d_free, d_nfree = torch.as_tensor(free).cuda(), torch.tensor([nfree], dtype=torch.int32, device="cuda")
    refs = [kvp.kv_commit_paged(forest, *outs, _bits(kns[l]), _bits(vns[l]), hosts[l][0], hosts[l][1], table,
                                page_off, poff, free, nfree) for l in range(n_layers)]
    assert all(r["error"] == 0 for r in refs)
    res = dsbd.kv_commit_paged(dsbd.Forest(forest, "cuda"), Hkv, d, i32(outs[0]), i32(outs[1]), i32(outs[2]),
                               i32(outs[3]), None, kn, vn, dk, dv, torch.as_tensor(table).cuda(),
                               torch.as_tensor(page_off).cuda(), torch.as_tensor(poff).cuda(), poff, d_free, d_nfree,
                               n_slots=int(outs[0][-1]), table_capacity=len(refs[0]["new_page_table"]))
    torch.cuda.synchronize()
    assert int(res["status"].item()) == 0
    nt = len(refs[0]["new_page_table"])
    for l in range(n_layers):
        ref = refs[l]
        assert np.array_equal(ref["new_page_table"], refs[0]["new_page_table"])
        assert np.array_equal(res["new_page_table"].cpu().numpy()[:nt], ref["new_page_table"])
        gk, gv = kvp.gather(_bits(dk[l]).reshape(hosts[l][0].shape), _bits(dv[l]).reshape(hosts[l][1].shape),
                            ref["new_page_table"], ref["new_page_off"], ref["new_prefix_off"])
        wk, wv = kvp.gather(ref["k_pool"], ref["v_pool"], ref["new_page_table"], ref["new_page_off"],
                            ref["new_prefix_off"])
        assert np.array_equal(gk, wk) and np.array_equal(gv, wv), l
    assert int(d_nfree.item()) == refs[0]["free_count"]
