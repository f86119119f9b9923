"""GPU parity of dsbd_verify_step / dsbd_select_width against the oracle (through the C ABI)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2409_16560_b200 as dsbd
from paper_2409_16560_b200 import inputs
from parity_util import check_exempt, compare_verify, run_gpu_verify, to_host_f32

pytestmark = pytest.mark.gpu


def _oracle(forest, params, zp, zq, rp, rq, threads=8):
    return oracle.verify_step(forest, params, zp, zq, rp.astype(np.float64), rq.astype(np.float64),
                              threads=threads)


def _both(data, steps, thresh=None):
    f, prm = data["forest"], dict(data["params"])
    if thresh is not None:
        prm["thresh"] = thresh
    zp_h, zq_h = to_host_f32(data["logits_p"]), to_host_f32(data["logits_q"])
    rp_h, rq_h = to_host_f32(data["root_logp"]), to_host_f32(data["root_logq"])
    exempt = decisions = 0
    for step in steps:
        prm["step"] = step
        gpu, status = run_gpu_verify(f, prm, data["logits_p"], data["logits_q"], data["root_logp"],
                                     data["root_logq"])
        assert status == 0
        ref = _oracle(f, prm, zp_h, zq_h, rp_h, rq_h)
        e, d = compare_verify(ref, gpu, f)
        exempt += e
        decisions += d
    check_exempt(exempt, decisions)
    return exempt, decisions


@pytest.mark.parametrize("name,steps", [("C1", range(40)), ("C2", range(40)), ("C3", range(6)),
                                        ("C4", range(3)), ("C6", range(6))])
def test_configs_full_size(name, steps):
    data = inputs.generate(inputs.config(name), "cuda", parts=("verify",))
    _both(data, steps)


@pytest.mark.parametrize("thresh,wmin", [(0.9, 1), (0.3, 1), (0.7, 8)])
def test_other_width_settings(thresh, wmin):
    data = inputs.generate(inputs.config("C3", R=2, V=5000), "cuda", parts=("verify",))
    data["params"]["W_min_r"] = None
    data["params"]["W_min"] = wmin
    _both(data, range(8), thresh=thresh)


@pytest.mark.parametrize("top_k,top_p", [(0, 1.0), (10, 0.8)])
def test_c5_all_requests(top_k, top_p):
    """The large configuration at full size, as the benchmark launches it: all 64 requests of
    three decode steps against the oracle, unwarped and with the warping of the paper's
    experiments (top-k 10 / top-p 0.8 on the joints)."""
    spec = inputs.config("C5")
    data = inputs.generate(spec, "cuda", parts=("verify",), draft_top_k=top_k, draft_top_p=top_p)
    data["params"].update(top_k=top_k, top_p=top_p)
    f, prm = data["forest"], dict(data["params"])
    zp_h, zq_h = to_host_f32(data["logits_p"]), to_host_f32(data["logits_q"])
    rp_h, rq_h = to_host_f32(data["root_logp"]), to_host_f32(data["root_logq"])
    exempt = decisions = 0
    for step in range(3):
        prm["step"] = step
        gpu, status = run_gpu_verify(f, prm, data["logits_p"], data["logits_q"], data["root_logp"],
                                     data["root_logq"])
        assert status == 0
        assert np.all(gpu["req_error"] == 0)
        assert np.all((gpu["l_last"] >= 1) & (gpu["l_last"] <= f["max_depth"] + 1))
        assert np.all(gpu["out_width"] >= 1)
        ref = _oracle(f, prm, zp_h, zq_h, rp_h, rq_h, threads=16)
        e, d = compare_verify(ref, gpu, f)
        exempt += e
        decisions += d
    check_exempt(exempt, decisions)


def _random_problem(rng, R, V, gamma, max_w, stride_pad=0, ninf_frac=0.0, tree="chain"):
    widths = rng.integers(1, max_w + 1, size=R)
    spec = dict(R=R, W=(1, max_w), tree=inputs._chain(gamma) if tree == "chain" else inputs._binary(gamma),
                prefix=(1, 1))
    forest, widths, _ = inputs.build_forest(spec, rng)
    N, B = forest["N"], forest["B"]
    stride = V + stride_pad
    zp = rng.normal(0, 2.5, size=(N, stride)).astype(np.float32)
    zq = (zp + rng.normal(0, 1.0, size=(N, stride))).astype(np.float32)
    if ninf_frac > 0:
        mask = rng.uniform(size=(1, stride)) < ninf_frac      # the same vocabulary entries for p and q
        zp[np.broadcast_to(mask, zp.shape)] = -np.inf
        zq[np.broadcast_to(mask, zq.shape)] = -np.inf
    tok = np.zeros(N, np.int32)
    for n in range(N):
        p = forest["parent"][n]
        if p >= 0:
            z = zq[p, :V].astype(np.float64)
            pr = np.exp(z - z.max()); pr /= pr.sum()
            tok[n] = rng.choice(V, p=pr)
    forest["token"] = tok
    rp = rng.normal(0, 1, B).astype(np.float32)
    rq = (rp + rng.normal(0, 0.5, B)).astype(np.float32)
    prm = dict(V=V, temperature=0.9, thresh=0.6, W_min=1, W_max=max_w, W_nom=max_w, seed=5, step=0,
               W_min_r=np.minimum(2, widths).astype(np.int32))
    return forest, prm, zp, zq, rp, rq, stride


@pytest.mark.parametrize("V,pad,ninf,tree", [(1023, 0, 0.0, "chain"), (1025, 3, 0.0, "chain"),
                                             (4097, 0, 0.0, "binary"), (777, 1, 0.2, "chain"),
                                             (3000, 0, 0.3, "binary"), (5, 0, 0.0, "chain")])
def test_ragged_vocab_unaligned_rows_masked_entries(V, pad, ninf, tree):
    rng = np.random.default_rng(V)
    exempt = decisions = 0
    for trial in range(6):
        forest, prm, zp, zq, rp, rq, stride = _random_problem(rng, R=5, V=V, gamma=3, max_w=4,
                                                              stride_pad=pad, ninf_frac=ninf, tree=tree)
        prm["step"] = trial
        dz = lambda a: torch.as_tensor(a).cuda()
        gpu, status = run_gpu_verify(forest, prm, dz(zp), dz(zq), dz(rp), dz(rq), row_stride=stride)
        assert status == 0
        ref = oracle.verify_step(forest, prm, zp, zq, rp.astype(np.float64), rq.astype(np.float64),
                                 row_stride=stride)
        e, d = compare_verify(ref, gpu, forest)
        exempt += e
        decisions += d
    check_exempt(exempt, decisions)


@pytest.mark.parametrize("R,V,max_w,gamma", [(700, 300, 3, 2), (3, 2500, 64, 1), (40, 9000, 16, 3)])
def test_many_requests_and_widest_layers(R, V, max_w, gamma):
    """More requests than resident clusters (several waves, small clusters), and the limit of
    64 beams / 64 live drafts per layer."""
    rng = np.random.default_rng(R + V)
    forest, prm, zp, zq, rp, rq, stride = _random_problem(rng, R=R, V=V, gamma=gamma, max_w=max_w)
    if max_w == 64:
        prm["W_min_r"] = None
        prm["W_min"] = 1
    dz = lambda a: torch.as_tensor(a).cuda()
    exempt = decisions = 0
    for step in range(2):
        prm["step"] = step
        gpu, status = run_gpu_verify(forest, prm, dz(zp), dz(zq), dz(rp), dz(rq))
        assert status == 0
        ref = oracle.verify_step(forest, prm, zp, zq, rp.astype(np.float64), rq.astype(np.float64), threads=8)
        e, d = compare_verify(ref, gpu, forest)
        exempt += e
        decisions += d
    check_exempt(exempt, decisions)


def test_peaky_distributions_use_the_exact_fallback():
    """When the histogram bin that a residual threshold falls into holds a heavy cell its
    bracket is too wide, and that residual mass is recomputed exactly by a pass over the rows.
    The path must be exercised and stay in parity."""
    rng = np.random.default_rng(11)
    exempt = decisions = fallbacks = respass = 0
    for trial in range(3):
        # a small vocabulary: every cell is heavy compared with the bracket tolerance, so any
        # threshold that shares its bin with a cell needs the exact evaluation
        forest, prm, zp, zq, rp, rq, stride = _random_problem(rng, R=200, V=64, gamma=3, max_w=6)
        prm["step"] = trial
        dz = lambda a: torch.as_tensor(a).cuda()
        gpu, status = run_gpu_verify(forest, prm, dz(zp), dz(zq), dz(rp), dz(rq))
        assert status == 0
        ref = oracle.verify_step(forest, prm, zp, zq, rp.astype(np.float64), rq.astype(np.float64))
        e, d = compare_verify(ref, gpu, forest)
        exempt += e; decisions += d
        st = gpu["req_stats"].reshape(-1, 8)
        assert np.array_equal(st[:, 0], np.minimum(ref["l_last"], forest["max_depth"]))   # layers verified
        assert st[:, 1].sum() == (ref["trace_kind"] == oracle.TR_ACCEPT).sum()            # accept tests
        acc = ref["trace_kind"] == oracle.TR_ACCEPT
        near_ref = int((np.abs(ref["trace_u"][acc] - np.minimum(ref["trace_a"][acc], 1.0)) < 1e-5).sum())
        assert abs(int(st[:, 4].sum()) - near_ref) <= 1                                    # near ties (the band's edge may differ)
        fallbacks += int(st[:, 2].sum()); respass += int(st[:, 3].sum())
    check_exempt(exempt, decisions)
    assert fallbacks > 0


def test_flat_tail_of_tiny_cells():
    """Rows whose vocabulary is a few heavy tokens plus a flat tail of about 10^5 cells of
    probability 1e-9 .. 1e-8 each (a per-cell mass near 2^-31): the tail as a whole carries
    1e-4 .. 1e-3 of the mass, far more than the 1e-5 tie band, so a histogram that rounded such
    cells to a coarse fixed-point unit would bias every residual mass.  Statuses, widths and
    tokens must still match the oracle."""
    rng = np.random.default_rng(21)
    V, R = 120000, 6
    forest, prm, _, _, rp, rq, stride = _random_problem(rng, R=R, V=64, gamma=3, max_w=4)
    N = forest["N"]
    zp = (-5.0 + 0.4 * rng.standard_normal((N, V))).astype(np.float32)
    heavy = rng.integers(0, V, size=(N, 40))
    for n in range(N):
        zp[n, heavy[n]] = rng.normal(11.0, 1.5, size=40)
    zq = (zp + 0.5 * rng.standard_normal((N, V))).astype(np.float32)
    tok = np.zeros(N, np.int32)
    for n in range(N):
        par = forest["parent"][n]
        if par >= 0:
            tok[n] = heavy[par, rng.integers(0, 40)]
    forest["token"] = tok
    prm = dict(prm, V=V, temperature=1.0)
    dz = lambda a: torch.as_tensor(a).cuda()
    exempt = decisions = 0
    for step in range(4):
        prm["step"] = step
        gpu, status = run_gpu_verify(forest, prm, dz(zp), dz(zq), dz(rp), dz(rq))
        assert status == 0
        ref = oracle.verify_step(forest, prm, zp, zq, rp.astype(np.float64), rq.astype(np.float64), threads=8)
        e, d = compare_verify(ref, gpu, forest)
        exempt += e; decisions += d
    check_exempt(exempt, decisions)
    # the tail is real mass: about 120000 cells of e^-5 against heavy cells of about e^11
    tail = np.exp(zp[0].astype(np.float64)); tail[heavy[0]] = 0.0
    assert tail.sum() / np.exp(zp[0].astype(np.float64)).sum() > 2e-5


def test_proportional_rows_overflow_is_detected():
    """Both models give the same next-token distribution in every row, so all cells of a row have
    the same ratio p_beam / q_beam (the ratio of the two beam weights) and land in one histogram
    bin: more mass than one 32-bit word of the histogram can hold.  The kernel must notice the
    wrapped word and compute that layer's residual masses by exact passes instead."""
    rng = np.random.default_rng(22)
    V = 100000
    forest, prm, _, _, rp, rq, stride = _random_problem(rng, R=4, V=64, gamma=2, max_w=4)
    N = forest["N"]
    zp = rng.normal(0.0, 1.0, size=(N, V)).astype(np.float32)
    zq = zp.copy()
    tok = np.zeros(N, np.int32)
    for n in range(N):
        if forest["parent"][n] >= 0:
            tok[n] = rng.integers(0, V)
    forest["token"] = tok
    rq = (rp + rng.normal(0, 1.0, len(rp))).astype(np.float32)       # beam weights differ between the models
    prm = dict(prm, V=V, temperature=1.0, thresh=0.3)
    dz = lambda a: torch.as_tensor(a).cuda()
    exempt = decisions = exact = wrapped = 0
    for step in range(3):
        prm["step"] = step
        gpu, status = run_gpu_verify(forest, prm, dz(zp), dz(zq), dz(rp), dz(rq))
        assert status == 0
        ref = oracle.verify_step(forest, prm, zp, zq, rp.astype(np.float64), rq.astype(np.float64), threads=8)
        e, d = compare_verify(ref, gpu, forest)
        exempt += e; decisions += d
        st = gpu["req_stats"].reshape(-1, 8)
        exact += int(st[:, 2].sum())
        wrapped += int(st[:, 6].sum())
    check_exempt(exempt, decisions)
    assert exact > 0 and wrapped > 0


@pytest.mark.parametrize("name,steps", [("C1", range(30)), ("C2", range(30)), ("C3", range(4)), ("C4", range(3)),
                                        ("C6", range(4))])
def test_configs_with_the_papers_warping(name, steps):
    """top-k 10 / top-p 0.8 on the joint distributions, the setting of the paper's experiments."""
    data = inputs.generate(inputs.config(name), "cuda", parts=("verify",), draft_top_k=10, draft_top_p=0.8)
    data["params"].update(top_k=10, top_p=0.8)
    _both(data, steps)


@pytest.mark.parametrize("top_k,top_p", [(1, 1.0), (3, 0.5), (64, 1.0), (64, 0.95), (7, 0.05)])
def test_warping_edge_settings(top_k, top_p):
    rng = np.random.default_rng(top_k)
    exempt = decisions = 0
    for trial in range(4):
        forest, prm, zp, zq, rp, rq, stride = _random_problem(rng, R=6, V=2100, gamma=3, max_w=5,
                                                              tree="binary" if trial % 2 else "chain")
        # make some drafts land inside the warped support: the best tokens of the small model
        best = np.argsort(-zq[:, :2100], axis=1)[:, :3]
        for n in range(forest["N"]):
            if forest["parent"][n] >= 0 and rng.uniform() < 0.7:
                forest["token"][n] = best[forest["parent"][n], rng.integers(0, 3)]
        prm.update(top_k=top_k, top_p=top_p, step=trial)
        dz = lambda a: torch.as_tensor(a).cuda()
        gpu, status = run_gpu_verify(forest, prm, dz(zp), dz(zq), dz(rp), dz(rq))
        # drafts outside the support of the warped q_beam (events of probability zero for a real
        # drafter) are accepted when p' has mass there and rejected otherwise; a rejection that
        # leaves no residual mass keeps p' -- neither side may report an error
        assert status == 0
        ref = oracle.verify_step(forest, prm, zp, zq, rp.astype(np.float64), rq.astype(np.float64))
        assert not ref["error"].any()
        e, d = compare_verify(ref, gpu, forest)
        exempt += e; decisions += d
    check_exempt(exempt, decisions)


def test_roots_only_forest_goes_straight_to_the_extra_layer():
    rng = np.random.default_rng(3)
    V, B = 2000, 3
    forest = dict(R=1, B=B, N=B, max_depth=0, req_beam_off=np.array([0, B], np.int32),
                  beam_node_off=np.arange(B + 1, dtype=np.int32), parent=np.full(B, -1, np.int32),
                  token=np.zeros(B, np.int32))
    zp = rng.normal(0, 2, size=(B, V)).astype(np.float32)
    zq = rng.normal(0, 2, size=(B, V)).astype(np.float32)
    rp = rng.normal(0, 1, B).astype(np.float32)
    prm = dict(V=V, thresh=0.7, W_min=1, W_max=4, W_nom=4, seed=9)
    exempt = decisions = 0
    for step in range(20):
        prm["step"] = step
        dz = lambda a: torch.as_tensor(a).cuda()
        gpu, status = run_gpu_verify(forest, prm, dz(zp), dz(zq), dz(rp), dz(rp))
        assert status == 0 and gpu["l_last"][0] == 1 and gpu["out_width"][0] == 4
        ref = oracle.verify_step(forest, prm, zp, zq, rp.astype(np.float64), rp.astype(np.float64))
        e, d = compare_verify(ref, gpu, forest)
        exempt += e; decisions += d
    check_exempt(exempt, decisions)


def test_draft_rank_order_and_equal_models():
    rng = np.random.default_rng(4)
    forest, prm, zp, zq, rp, rq, stride = _random_problem(rng, R=3, V=500, gamma=3, max_w=4, tree="binary")
    # a draw order that disagrees with the node numbering
    forest["draft_rank"] = rng.permutation(forest["N"]).astype(np.int32)
    dz = lambda a: torch.as_tensor(a).cuda()
    gpu, status = run_gpu_verify(forest, prm, dz(zp), dz(zq), dz(rp), dz(rq))
    ref = oracle.verify_step(forest, prm, zp, zq, rp.astype(np.float64), rq.astype(np.float64))
    assert status == 0
    compare_verify(ref, gpu, forest)
    # p == q: every draft up to the width is accepted
    prm2 = dict(prm, W_min_r=None, W_min=1, W_max=64, W_nom=2)
    gpu, status = run_gpu_verify(forest, prm2, dz(zp), dz(zp), dz(rp), dz(rp))
    ref = oracle.verify_step(forest, prm2, zp, zp, rp.astype(np.float64), rp.astype(np.float64))
    assert status == 0 and np.all(gpu["l_last"] == forest["max_depth"] + 1)
    compare_verify(ref, gpu, forest)
    assert not np.any(gpu["node_status"] == dsbd.binding.NODE_REJECTED)


def test_bad_token_is_reported_not_trapped():
    rng = np.random.default_rng(6)
    forest, prm, zp, zq, rp, rq, stride = _random_problem(rng, R=2, V=300, gamma=2, max_w=2)
    forest["token"][forest["N"] - 1] = 300
    dz = lambda a: torch.as_tensor(a).cuda()
    gpu, status = run_gpu_verify(forest, prm, dz(zp), dz(zq), dz(rp), dz(rq))
    assert status == 1          # DSBD_DEV_BAD_TOKEN


def test_host_side_errors():
    rng = np.random.default_rng(7)
    forest, prm, zp, zq, rp, rq, stride = _random_problem(rng, R=1, V=64, gamma=1, max_w=2)
    f = dsbd.Forest(forest, "cuda")
    out = dsbd.alloc_verify_out(f, oracle.default_out_off(forest, prm), "cuda")
    dz = lambda a: torch.as_tensor(a).cuda()
    prm_dev = dict(prm, W_min_r=None)
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(dsbd.DsbdError) as e:
        dsbd.verify_step(f, prm_dev, dz(zp), dz(zq), dz(rp), dz(rq), out, workspace=small)
    assert e.value.code == -3
    with pytest.raises(dsbd.DsbdError) as e:
        dsbd.verify_step(f, dict(prm_dev, temperature=0.0), dz(zp), dz(zq), dz(rp), dz(rq), out)
    assert e.value.code == -1


def test_width_parameters_are_validated():
    """A zero-initialised W_max / W_nom, or a cap below the minimum width, is refused on the host;
    per-request widths, which only the device sees, are reported per request and the request
    is not verified."""
    rng = np.random.default_rng(12)
    forest, prm, zp, zq, rp, rq, stride = _random_problem(rng, R=3, V=200, gamma=2, max_w=3)
    f = dsbd.Forest(forest, "cuda")
    out = dsbd.alloc_verify_out(f, oracle.default_out_off(forest, prm), "cuda")
    dz = lambda a: torch.as_tensor(a).cuda()
    base = dict(prm, W_min_r=None, W_min=2, W_max=3, W_nom=3)
    for bad in (dict(W_max=0), dict(W_nom=0), dict(W_min=0), dict(W_min=3, W_max=2)):
        with pytest.raises(dsbd.DsbdError) as e:
            dsbd.verify_step(f, dict(base, **bad), dz(zp), dz(zq), dz(rp), dz(rq), out)
        assert e.value.code == -1, bad
    wmax_r = torch.tensor([3, 0, 3], dtype=torch.int32, device="cuda")
    status = dsbd.verify_step(f, dict(base, W_max_r=wmax_r), dz(zp), dz(zq), dz(rp), dz(rq), out)
    torch.cuda.synchronize()
    assert int(status.item()) == 6                     # DSBD_DEV_BAD_PARAM
    assert out["req_error"].cpu().tolist() == [0, 6, 0]
    assert "width" in dsbd.status_string(6)


def test_select_width_rejects_a_malformed_live_list():
    """Node ids outside the forest and offsets beyond the list are reported, never used as
    addresses; well-formed requests of the same call still get their width."""
    rng = np.random.default_rng(13)
    forest, prm, zp, zq, rp, rq, stride = _random_problem(rng, R=3, V=700, gamma=2, max_w=4)
    prm = dict(prm, W_min_r=None)
    rbo, bno = forest["req_beam_off"], forest["beam_node_off"]
    live = [bno[rbo[r]:rbo[r + 1]].copy() for r in range(forest["R"])]
    live_off = np.concatenate([[0], np.cumsum([len(x) for x in live])]).astype(np.int32)
    m = np.array([len(x) for x in live], np.int32)
    sp = rng.normal(0, 1, forest["N"]).astype(np.float32)
    f = dsbd.Forest(forest, "cuda")
    dz = lambda a: torch.as_tensor(a).cuda()
    good = np.concatenate(live).astype(np.int32)
    w_ref, _, _ = oracle.select_width(forest, prm, zp, zq, sp.astype(np.float64), sp.astype(np.float64),
                                      live_off, good, m)
    for bad_id in (forest["N"], -1, 1 << 30):
        nodes = good.copy()
        nodes[live_off[1]] = bad_id                    # first live parent of request 1
        width, _, _, status = dsbd.select_width(f, prm, dz(zp), dz(zq), dz(sp), dz(sp), dz(live_off),
                                                dz(nodes), dz(m), out_stride=8)
        torch.cuda.synchronize()
        assert int(status.item()) == 4                 # DSBD_DEV_BAD_FOREST
        w = width.cpu().numpy()
        assert w[0] == w_ref[0] and w[2] == w_ref[2]
    off = live_off.copy()
    off[-1] = 1 << 20                                  # a list far longer than the forest
    _, _, _, status = dsbd.select_width(f, prm, dz(zp), dz(zq), dz(sp), dz(sp), dz(off), dz(good), dz(m),
                                        out_stride=8)
    torch.cuda.synchronize()
    assert int(status.item()) == 4


@pytest.mark.parametrize("top_k,top_p", [(0, 1.0), (10, 0.8), (40, 1.0)])
def test_select_width_matches_oracle(top_k, top_p):
    rng = np.random.default_rng(8)
    forest, prm, zp, zq, rp, rq, stride = _random_problem(rng, R=4, V=3000, gamma=2, max_w=5)
    prm = dict(prm, W_min_r=None, top_k=top_k, top_p=top_p)
    rbo, bno = forest["req_beam_off"], forest["beam_node_off"]
    live = [bno[rbo[r]:rbo[r + 1]] for r in range(forest["R"])]      # the roots
    live_off = np.concatenate([[0], np.cumsum([len(x) for x in live])]).astype(np.int32)
    live_nodes = np.concatenate(live).astype(np.int32)
    m = np.array([len(x) for x in live], np.int32)
    sp = rng.normal(0, 1, forest["N"]).astype(np.float32)
    sq = rng.normal(0, 1, forest["N"]).astype(np.float32)
    f = dsbd.Forest(forest, "cuda")
    dz = lambda a: torch.as_tensor(a).cuda()
    width, alpha, tail, status = dsbd.select_width(f, prm, dz(zp), dz(zq), dz(sp), dz(sq), dz(live_off),
                                                   dz(live_nodes), dz(m), out_stride=8)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    w_ref, a_ref, t_ref = oracle.select_width(forest, prm, zp, zq, sp.astype(np.float64),
                                              sq.astype(np.float64), live_off, live_nodes, m)
    assert np.array_equal(width.cpu().numpy(), w_ref)
    for r in range(forest["R"]):
        assert np.abs(alpha[r, :m[r]].cpu().numpy() - a_ref[r, :m[r]]).max() < 2e-5
        assert np.abs(tail[r, :m[r] + 1].cpu().numpy() - t_ref[r, :m[r] + 1]).max() < 2e-5
