"""Three consecutive decode steps, every stage on the device and, independently, in the oracles:
draft stage (gamma sampling steps) -> forest assembly -> forest attention over paged caches ->
verification -> paged cache update -> the kept beams are the next step's input beams.  The
device chain feeds on its own results and the oracle chain on its own; they are compared after
every stage (the stand-in models are seeded random tensors, the same bytes on both sides)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import forest_build as ofb
from oracle import kv_paged as kvp
import paper_2409_16560_b200 as dsbd
from paper_2409_16560_b200 import inputs
from parity_util import attention_close, compare_verify, check_exempt

pytestmark = pytest.mark.gpu

V, GAMMA, W_S, HQ, HKV, D = 2000, 3, 4, 4, 2, 128


def _bits(t):
    return t.detach().cpu().contiguous().view(torch.int16).numpy().reshape(-1)


def test_three_decode_steps():
    g = torch.Generator(device="cuda"); g.manual_seed(5)
    rng = np.random.default_rng(5)
    bf = lambda *s: torch.randn(*s, generator=g, device="cuda").to(torch.bfloat16)
    f32 = lambda *s: torch.randn(*s, generator=g, device="cuda")
    h = lambda t: t.detach().float().cpu().numpy()
    i32 = lambda a: torch.as_tensor(np.ascontiguousarray(a, dtype=np.int32)).cuda()
    # ---- initial state: 3 requests with 2, 1, 3 beams
    rbo = np.array([0, 2, 3, 6], np.int32)
    L = np.array([100, 100, 63, 130, 130, 130])
    poff = np.concatenate([[0], np.cumsum(L)]).astype(np.int64)
    kp, vp = bf(int(poff[-1]) * HKV * D), bf(int(poff[-1]) * HKV * D)
    hk, hv, table, page_off, free, nfree = kvp.pack_into_pages(_bits(kp), _bits(vp), poff, HKV, D, 48, rng)
    dk = torch.from_numpy(hk).view(torch.bfloat16).cuda()
    dv = torch.from_numpy(hv).view(torch.bfloat16).cuda()
    d_table, d_page_off = torch.as_tensor(table).cuda(), torch.as_tensor(page_off).cuda()
    d_free, d_nfree = torch.as_tensor(free).cuda(), torch.tensor([nfree], dtype=torch.int32, device="cuda")
    sp = f32(6) - 3
    sq = sp + 0.3 * f32(6)
    o_sp, o_sq = h(sp).astype(np.float64), h(sq).astype(np.float64)
    exempt = decisions = 0
    for step in range(3):
        R, B = len(rbo) - 1, int(rbo[-1])
        dprm = dict(V=V, temperature=0.9, seed=21, step=step)
        # ---- draft stage
        cur_off, cur_off_dev, cur_sq, o_cur_sq = rbo, i32(rbo), sq, o_sq
        draws_p, draws_t, o_draws_p, o_draws_t, rows_q = [], [], [], [], []
        out_off = (W_S * np.arange(R + 1)).astype(np.int32)
        for l in range(1, GAMMA + 1):
            zq = 2.0 * f32(int(cur_off[-1]), V)
            rows_q.append(zq)
            d = dsbd.draft_layer(cur_off_dev, cur_off, dprm, l, W_S, zq, cur_sq, i32(out_off), W_S * R)
            o = oracle.draft_layer(cur_off, dprm, l, W_S, h(zq), o_cur_sq, out_off=out_off)
            torch.cuda.synchronize()
            assert int(d["status"].item()) == 0 and not o["error"].any()
            assert np.array_equal(d["out_parent"].cpu().numpy(), o["out_parent"]), (step, l)
            assert np.array_equal(d["out_token"].cpu().numpy(), o["out_token"]), (step, l)
            assert np.allclose(h(d["out_logq"]), o["out_logq"], atol=1e-4)
            draws_p.append(d["out_parent"]); draws_t.append(d["out_token"])
            o_draws_p.append(o["out_parent"]); o_draws_t.append(o["out_token"])
            cur_off, cur_off_dev, cur_sq, o_cur_sq = out_off, i32(out_off), d["out_logq"], o["out_logq"]
        rows_q.append(2.0 * f32(W_S * R, V))                    # rows of the last layer's beams
        # ---- forest assembly
        f, node_of_draw, st = dsbd.forest_build(i32(rbo), rbo, GAMMA, W_S, torch.stack(draws_p), torch.stack(draws_t))
        of = ofb.forest_build(rbo, GAMMA, W_S, np.stack(o_draws_p), np.stack(o_draws_t))
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        for k in ("beam_node_off", "parent", "token", "draft_rank"):
            assert np.array_equal(f.dev[k].cpu().numpy(), of[k]), (step, k)
        assert np.array_equal(node_of_draw.cpu().numpy(), of["node_of_draw"])
        N = f.N
        # ---- the models' rows in node order
        zq_nodes = torch.empty(N, V, device="cuda")
        zq_nodes[torch.as_tensor(of["beam_node_off"][:-1]).long().cuda()] = rows_q[0]
        for l in range(GAMMA):
            zq_nodes[node_of_draw[l].long()] = rows_q[l + 1]
        zp_nodes = zq_nodes + 0.7 * f32(N, V)
        q, kn, vn = bf(N, HQ, D), bf(N, HKV, D), bf(N, HKV, D)
        # ---- attention over the paged caches
        scale = inputs.default_scale(D)
        out, st = dsbd.forest_attention_paged(f, HQ, HKV, D, scale, q, kn, vn, dk, dv, d_table, d_page_off,
                                              torch.as_tensor(poff).cuda(), poff)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        gk, gv = kvp.gather(hk, hv, table, page_off, poff)
        as_f = lambda bits: torch.from_numpy(bits).view(torch.bfloat16).float().numpy()
        ref = oracle.forest_attention(of, HQ, HKV, D, scale, h(q), h(kn), h(vn), as_f(gk), as_f(gv), poff)
        attention_close(h(out), ref, bf16=True)
        # ---- verification
        vprm = dict(V=V, temperature=0.9, thresh=0.6, W_min=1, W_max=3, W_nom=3, seed=33, step=step)
        oo = dsbd.default_out_off(of, vprm)
        vout = dsbd.alloc_verify_out(f, oo, "cuda")
        st = dsbd.verify_step(f, vprm, zp_nodes, zq_nodes, sp, sq, vout)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        gpu = {k: v.cpu().numpy() for k, v in vout.items()}
        gpu["layer_width"] = gpu["layer_width"].reshape(R, GAMMA + 1)
        ov = oracle.verify_step(of, vprm, h(zp_nodes), h(zq_nodes), o_sp, o_sq)
        e, dcs = compare_verify(ov, gpu, of)
        exempt += e; decisions += dcs
        assert not any(e.values())                           # the chains must stay in lockstep
        # ---- cache update, paged
        n_slots = int(oo[-1])
        oc = kvp.kv_commit_paged(of, ov["out_off"], ov["out_width"], ov["out_parent"], ov["out_root_beam"],
                                 ov["out_logp"], _bits(kn), _bits(vn), hk, hv, table, page_off, poff, free, nfree)
        assert oc["error"] == 0
        res = dsbd.kv_commit_paged(f, HKV, D, i32(oo), vout["out_width"], vout["out_parent"], vout["out_root_beam"],
                                   vout["out_logp"], kn, vn, dk, dv, d_table, d_page_off, torch.as_tensor(poff).cuda(),
                                   poff, d_free, d_nfree, n_slots=n_slots, table_capacity=len(oc["new_page_table"]) + 4)
        torch.cuda.synchronize()
        assert int(res["status"].item()) == 0
        nb, nt = len(oc["new_beam_slot"]), len(oc["new_page_table"])
        assert np.array_equal(res["new_req_beam_off"].cpu().numpy(), oc["new_req_beam_off"])
        assert np.array_equal(res["new_prefix_off"].cpu().numpy()[:nb + 1], oc["new_prefix_off"])
        assert np.array_equal(res["new_page_table"].cpu().numpy()[:nt], oc["new_page_table"])
        assert np.array_equal(res["new_beam_slot"].cpu().numpy()[:nb], oc["new_beam_slot"])
        a_k, a_v = kvp.gather(_bits(dk).reshape(hk.shape), _bits(dv).reshape(hv.shape), oc["new_page_table"],
                              oc["new_page_off"], oc["new_prefix_off"])
        b_k, b_v = kvp.gather(oc["k_pool"], oc["v_pool"], oc["new_page_table"], oc["new_page_off"],
                              oc["new_prefix_off"])
        assert np.array_equal(a_k, b_k) and np.array_equal(a_v, b_v)
        # ---- the kept beams are the next step's input beams
        slots = res["new_beam_slot"][:nb].long()
        sp, sq = vout["out_logp"][slots].contiguous(), vout["out_logq"][slots].contiguous()
        o_sp, o_sq = ov["out_logp"][oc["new_beam_slot"]], ov["out_logq"][oc["new_beam_slot"]]
        rbo, poff = oc["new_req_beam_off"], oc["new_prefix_off"]
        hk, hv, table, page_off = oc["k_pool"], oc["v_pool"], oc["new_page_table"], oc["new_page_off"]
        free, nfree = oc["free_stack"], oc["free_count"]
        d_table, d_page_off = res["new_page_table"][:nt].contiguous(), res["new_page_off"][:nb + 1].contiguous()
        assert (np.diff(rbo) >= 1).all()
    check_exempt(exempt, decisions)
