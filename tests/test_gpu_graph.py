"""The entry points neither allocate nor synchronise, so a whole decode step -- attention,
verification, cache update -- can be captured into one CUDA graph and replayed; the replay must
reproduce the eager results bit for bit, also after the inputs changed in place."""
import numpy as np
import pytest
import torch

import paper_2409_16560_b200 as dsbd
from paper_2409_16560_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["C2", "C3"])
def test_step_replays_from_a_cuda_graph(name):
    spec = inputs.config(name)
    data = inputs.generate(spec, "cuda")
    forest, prm, poff = data["forest"], dict(data["params"]), data["prefix_off"]
    f = dsbd.Forest(forest, "cuda")
    prm_dev = dict(prm, W_min_r=torch.as_tensor(prm["W_min_r"]).cuda())
    out_off = dsbd.default_out_off(forest, prm)
    n_slots = int(out_off[-1])
    scale = inputs.default_scale(spec["d"])
    poff_dev = torch.as_tensor(poff).cuda()
    out_off_dev = torch.as_tensor(np.asarray(out_off, np.int32)).cuda()
    cap = int(poff[-1]) + n_slots * (forest["max_depth"] + 1) * 2 + int(np.diff(poff).max()) * n_slots

    def buffers():
        return dict(attn=torch.empty_like(data["q"]), vout=dsbd.alloc_verify_out(f, out_off, "cuda"),
                    ws_a=torch.empty(max(dsbd.forest_attention_workspace(f, spec["Hq"], spec["Hkv"], spec["d"],
                                                                         data["q"].dtype, scale, poff), 256),
                                     dtype=torch.uint8, device="cuda"),
                    ws_v=torch.empty(dsbd.verify_workspace(f, prm_dev), dtype=torch.uint8, device="cuda"),
                    status=torch.zeros(1, dtype=torch.int32, device="cuda"), commit=None)

    def step(b, stream):
        dsbd.forest_attention(f, spec["Hq"], spec["Hkv"], spec["d"], scale, data["q"], data["k_new"], data["v_new"],
                              data["k_prefix"], data["v_prefix"], poff_dev, poff, out=b["attn"], workspace=b["ws_a"],
                              status=b["status"], stream=stream)
        dsbd.verify_step(f, prm_dev, data["logits_p"], data["logits_q"], data["root_logp"], data["root_logq"],
                         b["vout"], workspace=b["ws_v"], status=b["status"], stream=stream)
        v = b["vout"]
        c = b["commit"]
        b["commit"] = dsbd.kv_commit(f, spec["Hkv"], spec["d"], out_off_dev, v["out_width"], v["out_parent"],
                                     v["out_root_beam"], v["out_logp"], data["k_new"], data["v_new"],
                                     data["k_prefix"], data["v_prefix"], poff_dev, poff, n_slots=n_slots,
                                     dst_capacity=cap, k_dst=c["k_dst"] if c else None,
                                     v_dst=c["v_dst"] if c else None, workspace=c["workspace"] if c else None,
                                     status=b["status"], stream=stream, out=c)

    eager, graphed = buffers(), buffers()
    step(eager, torch.cuda.current_stream())
    torch.cuda.synchronize()
    # allocate the graphed step's commit buffers outside the capture, then capture
    step(graphed, torch.cuda.current_stream())
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            step(graphed, side)
    torch.cuda.synchronize()

    def same():
        assert int(eager["status"].item()) == 0 and int(graphed["status"].item()) == 0
        assert torch.equal(eager["attn"], graphed["attn"])
        for k in ("l_last", "out_width", "out_parent", "out_token", "out_source", "node_status", "layer_width",
                  "out_logp"):
            assert torch.equal(eager["vout"][k], graphed["vout"][k]), k
        n = int(eager["commit"]["new_prefix_off"][-1].item()) * spec["Hkv"] * spec["d"]
        assert torch.equal(eager["commit"]["new_prefix_off"], graphed["commit"]["new_prefix_off"])
        assert torch.equal(eager["commit"]["k_dst"][:n], graphed["commit"]["k_dst"][:n])

    for trial in range(3):
        # new contents in the same buffers: the graph reads them at replay time
        data["logits_q"].add_(0.25 * torch.randn_like(data["logits_q"][:1]))
        data["q"].mul_(0.9)
        for b in (eager, graphed):
            for k in ("attn",):
                b[k].zero_()
        g.replay()
        step(eager, torch.cuda.current_stream())
        torch.cuda.synchronize()
        same()
