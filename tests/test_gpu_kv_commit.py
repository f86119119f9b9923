"""GPU parity of dsbd_kv_commit against the numpy oracle: a byte-exact gather, so every output
is compared bit for bit.  Output beams are seeded synthetic ones (random widths, random parent
nodes inside the request), or the oracle's own verification results on the small config."""
import numpy as np
import pytest
import torch

import oracle
from oracle import kv_commit as kvc
import paper_2409_16560_b200 as dsbd
from paper_2409_16560_b200 import inputs

pytestmark = pytest.mark.gpu


def _bits(t):
    """Host copy of a tensor as integers of the same width (bf16 has no numpy type)."""
    t = t.detach().cpu().contiguous()
    return t.view(torch.int16 if t.element_size() == 2 else torch.int32).numpy().reshape(-1)


def _random_outputs(rng, forest, max_width, empty_every=0):
    rbo, bno = np.asarray(forest["req_beam_off"]), np.asarray(forest["beam_node_off"])
    R = int(forest["R"])
    out_off = (np.arange(R + 1) * max_width).astype(np.int32)
    out_width = rng.integers(1, max_width + 1, size=R).astype(np.int32)
    if empty_every:
        out_width[::empty_every] = 0
    slots = int(out_off[-1])
    out_parent = np.zeros(slots, np.int32)
    out_root = np.zeros(slots, np.int32)
    out_logp = (rng.normal(size=slots) * 3 - 20).astype(np.float32)
    for r in range(R):
        for k in range(max_width):                       # unused slots hold valid junk too
            b = rng.integers(rbo[r], rbo[r + 1])
            out_parent[out_off[r] + k] = rng.integers(bno[b], bno[b + 1])
            out_root[out_off[r] + k] = b
    return out_off, out_width, out_parent, out_root, out_logp


def _run_both(data, outs, keep_best, capacity=None):
    spec, forest, poff = data["spec"], data["forest"], data["prefix_off"]
    Hkv, d = spec["Hkv"], spec["d"]
    out_off, out_width, out_parent, out_root, out_logp = outs
    ref = kvc.kv_commit(forest, Hkv, d, out_off, out_width, out_parent, out_root, out_logp,
                        _bits(data["k_new"]), _bits(data["v_new"]), _bits(data["k_prefix"]),
                        _bits(data["v_prefix"]), poff, keep_best=keep_best)
    total = int(ref["new_prefix_off"][-1])
    cap = total + 7 if capacity is None else capacity
    f = dsbd.Forest(forest, "cuda")
    dv = lambda a, dt: torch.as_tensor(np.asarray(a), dtype=dt).cuda()
    canary = lambda: torch.full((cap * Hkv * d,), 7.0, dtype=data["k_new"].dtype, device="cuda")
    res = dsbd.kv_commit(f, Hkv, d, dv(out_off, torch.int32), dv(out_width, torch.int32),
                         dv(out_parent, torch.int32), dv(out_root, torch.int32), dv(out_logp, torch.float32),
                         data["k_new"], data["v_new"], data["k_prefix"], data["v_prefix"],
                         torch.as_tensor(poff).cuda(), poff, n_slots=int(out_off[-1]), dst_capacity=cap,
                         keep_best=keep_best, k_dst=canary(), v_dst=canary())
    torch.cuda.synchronize()
    return ref, res, total


def _compare(ref, res, total, spec):
    assert int(res["status"].item()) == 0
    nb = len(ref["new_beam_slot"])
    assert np.array_equal(res["new_req_beam_off"].cpu().numpy(), ref["new_req_beam_off"])
    npo = res["new_prefix_off"].cpu().numpy()
    assert np.array_equal(npo[:nb + 1], ref["new_prefix_off"])
    assert np.all(npo[nb:] == total)
    slot = res["new_beam_slot"].cpu().numpy()
    assert np.array_equal(slot[:nb], ref["new_beam_slot"]) and np.all(slot[nb:] == -1)
    n = total * spec["Hkv"] * spec["d"]
    assert np.array_equal(_bits(res["k_dst"])[:n], ref["k_cache"])
    assert np.array_equal(_bits(res["v_dst"])[:n], ref["v_cache"])
    # nothing is written past the kept caches
    assert bool((res["k_dst"][n:] == 7.0).all()) and bool((res["v_dst"][n:] == 7.0).all())


@pytest.mark.parametrize("name,kw", [("C1", {}), ("C2", {}), ("C3", {}), ("C4", {}), ("C5", dict(R=6))])
@pytest.mark.parametrize("keep_best", [False, True])
def test_configs(name, kw, keep_best):
    spec = inputs.config(name, **kw)
    data = inputs.generate(spec, "cuda", parts=("attention",))
    rng = np.random.default_rng(11)
    W = spec["W"][1] if isinstance(spec["W"], tuple) else spec["W"]
    outs = _random_outputs(rng, data["forest"], max(2, min(W, 4)), empty_every=5 if name in ("C4", "C5") else 0)
    ref, res, total = _run_both(data, outs, keep_best)
    _compare(ref, res, total, spec)


def test_outputs_of_a_real_verification_step():
    spec = inputs.config("C1")
    data = inputs.generate(spec, "cuda")
    forest, prm = data["forest"], data["params"]
    f32 = lambda t: t.detach().float().cpu().numpy()
    for step in range(5):
        v = oracle.verify_step(forest, dict(prm, step=step), f32(data["logits_p"]), f32(data["logits_q"]),
                               f32(data["root_logp"]).astype(np.float64), f32(data["root_logq"]).astype(np.float64))
        outs = (v["out_off"], v["out_width"], v["out_parent"], v["out_root_beam"], v["out_logp"].astype(np.float32))
        for keep_best in (False, True):
            ref, res, total = _run_both(data, outs, keep_best)
            _compare(ref, res, total, spec)


def test_committed_cache_feeds_the_next_attention():
    """The packed output is the layout dsbd_forest_attention reads: one-node trees on top of the
    new caches must see exactly what the oracle's attention sees on the oracle's caches."""
    spec = inputs.config("C2")
    data = inputs.generate(spec, "cuda", parts=("attention",))
    rng = np.random.default_rng(5)
    outs = _random_outputs(rng, data["forest"], 3)
    ref, res, total = _run_both(data, outs, False)
    nb = len(ref["new_beam_slot"])
    Hq, Hkv, d = spec["Hq"], spec["Hkv"], spec["d"]
    nxt = dict(R=1, B=nb, N=nb, max_depth=0, req_beam_off=np.array([0, nb], np.int32),
               beam_node_off=np.arange(nb + 1, dtype=np.int32), parent=np.full(nb, -1, np.int32),
               token=np.zeros(nb, np.int32))
    g = torch.Generator(device="cuda"); g.manual_seed(3)
    q = torch.randn(nb, Hq, d, generator=g, device="cuda").to(torch.bfloat16)
    kn = torch.randn(nb, Hkv, d, generator=g, device="cuda").to(torch.bfloat16)
    vn = torch.randn(nb, Hkv, d, generator=g, device="cuda").to(torch.bfloat16)
    npo = ref["new_prefix_off"]
    out, st = dsbd.forest_attention(dsbd.Forest(nxt, "cuda"), Hq, Hkv, d, inputs.default_scale(d), q, kn, vn,
                                    res["k_dst"], res["v_dst"], res["new_prefix_off"][:nb + 1].contiguous(), npo)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    as_f32 = lambda bits: torch.from_numpy(bits.astype(np.int16)).view(torch.bfloat16).float().numpy()
    want = oracle.forest_attention(nxt, Hq, Hkv, d, inputs.default_scale(d), q.float().cpu().numpy(),
                                   kn.float().cpu().numpy(), vn.float().cpu().numpy(),
                                   as_f32(ref["k_cache"]), as_f32(ref["v_cache"]), npo)
    err = np.abs(out.float().cpu().numpy() - want)
    assert np.all(err <= 1e-2 + 2e-2 * np.abs(want))


def test_capacity_and_bad_slots_are_reported_and_nothing_is_copied():
    spec = inputs.config("C1")
    data = inputs.generate(spec, "cuda", parts=("attention",))
    rng = np.random.default_rng(2)
    outs = _random_outputs(rng, data["forest"], 2)
    ref, res, total = _run_both(data, outs, False, capacity=None)
    _compare(ref, res, total, spec)
    # one token short
    _, res, _ = _run_both(data, outs, False, capacity=total - 1)
    assert int(res["status"].item()) == 3
    # a parent node outside the tree of the named beam
    bad = [a.copy() for a in outs]
    bad[2][0] = data["forest"]["N"] - 1
    bad[3][0] = 0
    forest, poff = data["forest"], data["prefix_off"]
    f = dsbd.Forest(forest, "cuda")
    dv = lambda a, dt: torch.as_tensor(np.asarray(a), dtype=dt).cuda()
    canary = torch.full((total * spec["Hkv"] * spec["d"],), 7.0, dtype=data["k_new"].dtype, device="cuda")
    res = dsbd.kv_commit(f, spec["Hkv"], spec["d"], dv(bad[0], torch.int32), dv(bad[1], torch.int32),
                         dv(bad[2], torch.int32), dv(bad[3], torch.int32), None, data["k_new"], data["v_new"],
                         data["k_prefix"], data["v_prefix"], torch.as_tensor(poff).cuda(), poff,
                         n_slots=int(bad[0][-1]), dst_capacity=total, k_dst=canary)
    torch.cuda.synchronize()
    assert int(res["status"].item()) == 4
    assert bool((canary == 7.0).all())
    assert int(res["new_req_beam_off"][-1].item()) == 0


def test_host_side_errors():
    spec = inputs.config("C1")
    data = inputs.generate(spec, "cuda", parts=("attention",))
    f = dsbd.Forest(data["forest"], "cuda")
    z = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(dsbd.DsbdError):           # keep_best without scores
        dsbd.kv_commit(f, spec["Hkv"], spec["d"], z, z, z, z, None, data["k_new"], data["v_new"], data["k_prefix"],
                       data["v_prefix"], torch.as_tensor(data["prefix_off"]).cuda(), data["prefix_off"],
                       n_slots=2, dst_capacity=10, keep_best=True)
    with pytest.raises(dsbd.DsbdError):           # workspace too small
        dsbd.kv_commit(f, spec["Hkv"], spec["d"], z, z, z, z, None, data["k_new"], data["v_new"], data["k_prefix"],
                       data["v_prefix"], torch.as_tensor(data["prefix_off"]).cuda(), data["prefix_off"],
                       n_slots=2, dst_capacity=10, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
