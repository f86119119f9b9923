"""Benchmark of the DSBD hot path: one step = forest attention + verification step over one
batch of synthetic input (configuration C5 by default: 64 requests x 8 beams x depth-8 chain
drafts = 4608 forest nodes, 32 query / 8 KV heads x 128, bf16 KV prefix 4096 per beam, fp32
logits over a 128256-token vocabulary).

  python bench.py --gpus N --steps K --warmup W            the CUDA library
  python bench.py --impl reference --steps K --warmup W    the CPU oracle on a bounded sample

Prints ONE JSON line.  `value` = forest nodes verified per second with every input resident in
HBM; `e2e` = the same through the C-ABI call with host buffers (pinned host -> device copies
of the step's inputs and a device -> host read of its results inside the timed region).
Multi-GPU: requests are independent, so each rank runs its own batch (weak scaling), with no
data-path collective; time is the max over ranks.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "verified forest nodes/sec per decode step"
UNIT = "nodes/s"

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) on the full C5 workload,
# from ncu captures of the same kernels on 16 of the 64 requests, scaled by 64/16 (the traffic is
# proportional to the number of requests).  verify_step_total = the dense pass plus the
# per-request kernel, which re-reads the live rows.
NCU_TRAFFIC_BYTES = {"C5": {"forest_attention": 8.665e9, "verify_dense_pass": 4.748e9,
                            "verify_step_total": 4.748e9 + 0.740e9}}


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.QUERY, "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        rows = [l for (t, l) in self.lines if t0 <= t <= t1] or [l for (_, l) in self.lines]
        for line in rows:
            p = [x.strip() for x in line.split(",")]
            if len(p) < 9:
                continue
            try:
                sm.append(float(p[1])); mx.append(float(p[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def rank_spec(spec, rank):
    """Requests are independent, so a multi-GPU run gives every rank its own batch of the same
    shape (weak scaling, no collective on the data path): same configuration, different seed."""
    out = dict(spec)
    out["seed"] = spec["seed"] + 1000 * rank
    return out


def max_over_ranks(ms, world, device):
    """Step time of the job = the slowest rank's device time."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(nodes_per_rank, world, ms_per_step):
    """Whole-job throughput: nodes verified by all ranks per second."""
    return nodes_per_rank * world / (ms_per_step * 1e-3)


def _cpu_baseline(data_host, spec, threads, budget_s=20.0, gpu=None):
    """The oracle, as it stands, on a bounded sample of the workload: verification of a few
    requests and attention of a few trees; returns nodes/s of the whole step extrapolated
    from per-node times, and a description of the sample.  With `gpu` (the library's outputs for
    the same inputs and Philox step, as numpy arrays) the sampled requests and trees are also
    compared and the counts returned as the second value."""
    import oracle
    forest = data_host["forest"]
    rbo, bno = forest["req_beam_off"], forest["beam_node_off"]
    par = {"verify_requests": 0, "verify_decisions": 0, "verify_mismatching_requests": 0,
           "attention_trees": 0, "attention_max_abs_err": 0.0}
    # verification: one request at a time until half of the budget is used
    n_ver, t_ver, reqs = 0, 0.0, 0
    for r in range(forest["R"]):
        sub = data_host["verify_sub"](r)
        t0 = time.perf_counter()
        ref = oracle.verify_step(*sub, trace=False, threads=threads)
        t_ver += time.perf_counter() - t0
        n_ver += sub[0]["N"]
        reqs += 1
        if gpu is not None:
            n0, n1 = int(bno[rbo[r]]), int(bno[rbo[r + 1]])
            g0, w = int(gpu["out_off"][r]), int(ref["out_width"][0])
            st_ref, st_gpu = ref["node_status"], gpu["node_status"][n0:n1]
            same = (int(ref["l_last"][0]) == int(gpu["l_last"][r]) and w == int(gpu["out_width"][r])
                    and np.array_equal(ref["layer_width"][0], gpu["layer_width"][r])
                    and np.array_equal(st_ref, st_gpu)
                    and np.array_equal(ref["out_token"][:w], gpu["out_token"][g0:g0 + w])
                    and np.array_equal(ref["out_source"][:w], gpu["out_source"][g0:g0 + w])
                    and np.array_equal(ref["out_parent"][:w] + n0, gpu["out_parent"][g0:g0 + w]))
            par["verify_requests"] += 1
            # decisions: accept tests (nodes accepted or rejected below the roots) and output beams drawn
            tested = np.isin(st_ref, (1, 2)) & (sub[0]["parent"] >= 0)
            par["verify_decisions"] += int(tested.sum()) + int((ref["out_source"][:w] != 0).sum())
            par["verify_mismatching_requests"] += 0 if same else 1
        if t_ver > budget_s / 2 or reqs >= data_host["max_reqs"]:
            break
    n_att, t_att, beams = 0, 0.0, 0
    for b in range(forest["B"]):
        sub = data_host["attn_sub"](b)
        t0 = time.perf_counter()
        ref = oracle.forest_attention(*sub, threads=threads)
        t_att += time.perf_counter() - t0
        n_att += sub[0]["N"]
        beams += 1
        if gpu is not None:
            n0, n1 = int(bno[b]), int(bno[b + 1])
            par["attention_trees"] += 1
            par["attention_max_abs_err"] = max(par["attention_max_abs_err"],
                                               float(np.abs(ref - gpu["attn_out"][n0:n1]).max()))
        if t_att > budget_s / 2 or beams >= data_host["max_beams"]:
            break
    per_node = t_ver / n_ver + t_att / n_att
    res = {"value": 1.0 / per_node, "unit": UNIT, "cores": threads, "kind": "oracle",
           "sample": "%d of %d requests verified (%.1f s), attention of %d of %d trees (%.1f s); "
                     "nodes/s = 1 / (verify s/node + attention s/node)" % (
                         reqs, forest["R"], t_ver, beams, forest["B"], t_att)}
    return (res, par) if gpu is not None else res


def _host_views(data, spec):
    """Closures that cut per-request / per-tree oracle inputs out of the device tensors."""
    import torch
    forest, prm, poff = data["forest"], data["params"], data["prefix_off"]
    rbo, bno = forest["req_beam_off"], forest["beam_node_off"]
    Hkv, d = spec["Hkv"], spec["d"]
    h = lambda x: x.detach().float().cpu().numpy()

    def sub_tree_forest(b_lo, b_hi):
        n0, n1 = int(bno[b_lo]), int(bno[b_hi])
        par = forest["parent"][n0:n1]
        return dict(R=1, B=b_hi - b_lo, N=n1 - n0, max_depth=forest["max_depth"],
                    req_beam_off=np.array([0, b_hi - b_lo], np.int32),
                    beam_node_off=(bno[b_lo:b_hi + 1] - n0).astype(np.int32),
                    parent=np.where(par >= 0, par - n0, -1).astype(np.int32),
                    token=forest["token"][n0:n1].astype(np.int32)), n0, n1

    def verify_sub(r):
        f, n0, n1 = sub_tree_forest(int(rbo[r]), int(rbo[r + 1]))
        p = dict(prm, W_min_r=np.asarray(prm["W_min_r"])[r:r + 1], req_id=np.array([r], np.int32))
        return (f, p, h(data["logits_p"][n0:n1]), h(data["logits_q"][n0:n1]),
                h(data["root_logp"][rbo[r]:rbo[r + 1]]).astype(np.float64),
                h(data["root_logq"][rbo[r]:rbo[r + 1]]).astype(np.float64))

    def attn_sub(b):
        f, n0, n1 = sub_tree_forest(b, b + 1)
        s, e = int(poff[b]) * Hkv * d, int(poff[b + 1]) * Hkv * d
        return (f, spec["Hq"], Hkv, d, 1.0 / np.sqrt(d), h(data["q"][n0:n1]), h(data["k_new"][n0:n1]),
                h(data["v_new"][n0:n1]), h(data["k_prefix"][s:e]), h(data["v_prefix"][s:e]),
                np.array([0, poff[b + 1] - poff[b]], np.int64))

    return dict(forest=forest, verify_sub=verify_sub, attn_sub=attn_sub, max_reqs=48, max_beams=256)


def run_reference(args):
    """--impl reference: the oracle on the host cores, each step a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    from paper_2409_16560_b200 import inputs
    spec = inputs.config(args.workload)
    # a slice of the workload is enough for the sample: fewer requests, same shapes
    small = dict(spec, R=min(spec["R"], 2))
    data = inputs.generate(small, "cpu", draft_top_k=args.top_k, draft_top_p=args.top_p)
    data["params"].update(top_k=args.top_k, top_p=args.top_p)
    views = _host_views(data, small)
    views["max_reqs"], views["max_beams"] = 1, 1
    threads = os.cpu_count() or 1
    for _ in range(args.warmup):
        _cpu_baseline(views, small, threads, budget_s=1e9)
    t0 = time.perf_counter()
    vals = [_cpu_baseline(views, small, threads, budget_s=1e9) for _ in range(args.steps)]
    dt = time.perf_counter() - t0
    value = float(np.mean([v["value"] for v in vals]))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / max(args.steps, 1),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": args.workload, "sample": vals[-1]["sample"]},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": vals[-1]["sample"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def _side_workload(dsbd, inputs, dev, name, steps, warmup, top_k=0, top_p=1.0, parts=("attention", "verify")):
    """Attention and verification of another workload, timed like the main one (per-part CUDA
    events on the launching stream, L2 flushed between steps when the inputs would fit it);
    returns {part: {"bytes", "ms", "gbs"}}."""
    import torch
    spec = inputs.config(name)
    data = inputs.generate(spec, dev, parts=parts, draft_top_k=top_k, draft_top_p=top_p)
    forest, poff = data["forest"], data["prefix_off"]
    f = dsbd.Forest(forest, dev)
    stream = torch.cuda.current_stream()
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    calls, nbytes = {}, {}
    if "attention" in parts:
        scale = inputs.default_scale(spec["d"])
        poff_dev = torch.as_tensor(poff).to(dev)
        out = torch.empty_like(data["q"])
        ws = torch.empty(max(dsbd.forest_attention_workspace(f, spec["Hq"], spec["Hkv"], spec["d"], data["q"].dtype,
                                                             scale, poff), 256), dtype=torch.uint8, device=dev)
        calls["forest_attention"] = lambda step: dsbd.forest_attention(
            f, spec["Hq"], spec["Hkv"], spec["d"], scale, data["q"], data["k_new"], data["v_new"], data["k_prefix"],
            data["v_prefix"], poff_dev, poff, out=out, workspace=ws, status=status, stream=stream)
        nbytes["forest_attention"] = inputs.attention_bytes(spec, forest, poff)
    if "verify" in parts:
        prm = dict(data["params"], top_k=top_k, top_p=top_p)
        prm_dev = dict(prm, W_min_r=torch.as_tensor(prm["W_min_r"]).to(dev))
        vout = dsbd.alloc_verify_out(f, dsbd.default_out_off(forest, prm), dev)
        ws_v = torch.empty(max(dsbd.verify_workspace(f, prm_dev), 256), dtype=torch.uint8, device=dev)

        def verify(step):
            prm_dev["step"] = step
            dsbd.verify_step(f, prm_dev, data["logits_p"], data["logits_q"], data["root_logp"], data["root_logq"],
                             vout, workspace=ws_v, status=status, stream=stream)
        calls["verify_step_total"] = verify
        nbytes["verify_step_total"] = inputs.verify_bytes(spec, forest)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if sum(nbytes.values()) < 4 * (126 << 20) else None
    times = {k: [] for k in calls}
    for s_ in range(warmup + steps):
        evs = {}
        for k, fn in calls.items():
            if flush is not None:
                flush.zero_()
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record(stream); fn(s_); e1.record(stream)
            evs[k] = (e0, e1)
        if s_ >= warmup:
            for k, (e0, e1) in evs.items():
                times[k].append((e0, e1))
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "device status %d on %s" % (int(status.item()), name)
    res = {}
    for k in calls:
        ms = float(np.median([a.elapsed_time(b) for a, b in times[k]]))
        res[k] = {"bytes": nbytes[k], "ms": ms, "gbs": nbytes[k] / ms * 1e-6}
    return res


PHASE_NAMES = {1: "start", 2: "prologue / previous layer's completion", 3: "layer set-up", 4: "histogram pass",
               5: "merge across the cluster", 6: "image into shared memory", 7: "suffix sums", 8: "residual chain",
               9: "width and accept loop", 10: "residual pass for a completion draw", 11: "completion draws",
               12: "extra layer and final writes"}


def run_verify_phases(args):
    """--verify-phases: where the time of the per-request verification kernel goes.  Runs the
    verification of the workload on a build of the library that stamps %globaltimer at the phase
    boundaries (DSBD_PHASE_TIMING; slower than the product build, so the shares count, not the
    absolute times) and prints one JSON line with the time line of the slowest request, the mean
    per phase over all requests and the end time by number of layers verified."""
    import torch
    import paper_2409_16560_b200 as dsbd
    from paper_2409_16560_b200 import binding, inputs
    from paper_2409_16560_b200 import build as cuda_build
    binding.use_library(cuda_build.build_phase_timing())
    dev = torch.device("cuda", 0)
    spec = inputs.config(args.workload)
    if args.requests > 0:
        spec["R"] = args.requests
    data = inputs.generate(spec, dev, parts=("verify",), draft_top_k=args.top_k, draft_top_p=args.top_p)
    forest, prm = data["forest"], dict(data["params"], top_k=args.top_k, top_p=args.top_p)
    f = dsbd.Forest(forest, dev)
    R = f.R
    prm_dev = dict(prm, W_min_r=torch.as_tensor(prm["W_min_r"]).to(dev))
    vout = dsbd.alloc_verify_out(f, dsbd.default_out_off(forest, prm), dev)
    ws = torch.zeros(dsbd.verify_workspace(f, prm_dev), dtype=torch.uint8, device=dev)
    stamps = ws[-R * 256 * 8:]                        # the stamps live behind the workspace proper
    for step in range(args.warmup + 1):
        stamps.zero_()
        prm_dev["step"] = step
        dsbd.verify_step(f, prm_dev, data["logits_p"], data["logits_q"], data["root_logp"], data["root_logq"], vout,
                         workspace=ws)
        torch.cuda.synchronize()
    dbg = stamps.view(torch.int64).cpu().numpy().reshape(R, 256)
    t0 = min(int(dbg[r, 0]) & 0xFFFFFFFFFFFF for r in range(R))
    lines, ends, per_phase = [], [], {}
    for r in range(R):
        prev, line = None, []
        for v in dbg[r]:
            if v == 0:
                break
            slot, t = int(v) >> 48, int(v) & 0xFFFFFFFFFFFF
            if prev is not None:
                line.append((slot, (t - prev) / 1e3))
                per_phase.setdefault(slot, []).append((t - prev) / 1e3)
            prev = t
        lines.append(line)
        ends.append((prev - t0) / 1e3)
    l_last = vout["l_last"].cpu().numpy()
    slow = int(np.argmax(ends))
    out = {"verify_phases": {
        "workload": args.workload, "requests": R, "top_k": args.top_k, "top_p": args.top_p, "unit": "us",
        "kernel_span": max(ends),
        "end_by_l_last": {int(k): round(float(np.mean([e for e, l in zip(ends, l_last) if l == k])), 1)
                          for k in sorted(set(l_last.tolist()))},
        "requests_by_l_last": {int(k): int((l_last == k).sum()) for k in sorted(set(l_last.tolist()))},
        "mean_per_phase": {PHASE_NAMES[k]: round(float(np.mean(v)), 1) for k, v in sorted(per_phase.items())},
        "slowest_request": {"request": slow, "l_last": int(l_last[slow]),
                            "time_line": [[PHASE_NAMES[s_], round(d, 1)] for s_, d in lines[slow]]}}}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="dsbd", choices=["dsbd", "reference"])
    ap.add_argument("--workload", default="C5")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--pipeline-steps", type=int, default=0,
                    help="also time whole decode steps (draft stage, forest assembly, paged attention, "
                         "verification, paged cache update) and report them under 'pipeline'")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--top-k", type=int, default=0, help="warp the joint distributions: top-k (0 = off)")
    ap.add_argument("--top-p", type=float, default=1.0, help="and top-p (needs --top-k); the paper uses 10 / 0.8")
    ap.add_argument("--requests", type=int, default=0,
                    help="override the number of requests of the workload (profiling on a smaller case)")
    ap.add_argument("--no-side-workloads", action="store_true",
                    help="skip the extra figures under 'kernels' (C4, C6, the paper's warping on C5, "
                         "several attention layers in one call)")
    ap.add_argument("--verify-phases", action="store_true",
                    help="print the phase time line of the per-request verification kernel (a timing "
                         "build of the library) instead of the benchmark line")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.verify_phases:
        return run_verify_phases(args)

    import torch
    import torch.distributed as dist
    import paper_2409_16560_b200 as dsbd
    from paper_2409_16560_b200 import inputs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    dsbd.load()

    spec = inputs.config(args.workload)
    if args.requests > 0:
        spec["R"] = args.requests
    spec = rank_spec(spec, rank)                         # every rank verifies its own requests
    data = inputs.generate(spec, dev, draft_top_k=args.top_k, draft_top_p=args.top_p)
    data["params"].update(top_k=args.top_k, top_p=args.top_p)
    forest, prm, poff = data["forest"], dict(data["params"]), data["prefix_off"]
    prm.update(top_k=args.top_k, top_p=args.top_p)
    f = dsbd.Forest(forest, dev)
    prm_dev = dict(prm, W_min_r=torch.as_tensor(prm["W_min_r"]).to(dev))
    out_off = dsbd.default_out_off(forest, prm)
    vout = dsbd.alloc_verify_out(f, out_off, dev)
    poff_dev = torch.as_tensor(poff).to(dev)
    scale = inputs.default_scale(spec["d"])
    attn_out = torch.empty_like(data["q"])
    ws_a = torch.empty(max(dsbd.forest_attention_workspace(f, spec["Hq"], spec["Hkv"], spec["d"],
                                                           data["q"].dtype, scale, poff), 256),
                       dtype=torch.uint8, device=dev)
    ws_v = torch.empty(max(dsbd.verify_workspace(f, prm_dev), 256), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    lse_p = torch.empty(f.N, dtype=torch.float32, device=dev)
    lse_q = torch.empty(f.N, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()

    def attention():
        dsbd.forest_attention(f, spec["Hq"], spec["Hkv"], spec["d"], scale, data["q"], data["k_new"],
                              data["v_new"], data["k_prefix"], data["v_prefix"], poff_dev, poff,
                              out=attn_out, workspace=ws_a, status=status, stream=stream)

    def verify(step):
        prm_dev["step"] = step
        dsbd.verify_step(f, prm_dev, data["logits_p"], data["logits_q"], data["root_logp"],
                         data["root_logq"], vout, workspace=ws_v, status=status, stream=stream)

    def one_step(step):
        attention()
        verify(step)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for s in range(args.warmup):
        one_step(s)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4 * args.steps + 1)]
    # workloads whose inputs would sit in the 126 MB L2 get it flushed between steps (a 256 MB
    # write outside the per-step events; the step time is then the sum of the per-step times)
    step_bytes = inputs.attention_bytes(spec, forest, poff) + inputs.verify_bytes(spec, forest)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if step_bytes < 4 * (126 << 20) else None
    t_wall0 = time.time()
    barrier()
    ev[0].record(stream)
    e_attn, e_ver = [], []
    for s in range(args.steps):
        a0 = torch.cuda.Event(enable_timing=True); a1 = torch.cuda.Event(enable_timing=True)
        a2 = torch.cuda.Event(enable_timing=True)
        if flush is not None:
            flush.zero_()
        a0.record(stream)
        attention()
        a1.record(stream)
        verify(args.warmup + s)
        a2.record(stream)
        e_attn.append((a0, a1)); e_ver.append((a1, a2))
    ev[1].record(stream)
    barrier()
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    t_attn = [a.elapsed_time(b) for a, b in e_attn]
    t_ver = [a.elapsed_time(b) for a, b in e_ver]
    total_local = ev[0].elapsed_time(ev[1]) if flush is None else float(np.sum(t_attn) + np.sum(t_ver))
    total_ms = max_over_ranks(total_local, world, dev)
    attn_ms, ver_ms = float(np.median(t_attn)), float(np.median(t_ver))
    assert int(status.item()) == 0, "device status %d" % int(status.item())
    st = vout["req_stats"].cpu().numpy().reshape(-1, 8).astype(float)
    verify_stats = {"layers_per_request": float(st[:, 0].mean()), "accept_tests_per_request": float(st[:, 1].mean()),
                    "exact_recomputations_per_request": float(st[:, 2].mean()),
                    "extra_completion_passes_per_request": float(st[:, 3].mean()),
                    "near_tie_accept_tests": int(st[:, 4].sum()), "consulted_row_pairs_per_request": float(st[:, 5].mean()),
                    "overflowed_histograms": int(st[:, 6].sum()),
                    "output_beams_per_request": float(vout["out_width"].float().mean().item())}

    # the dense logits pass alone (the kernel the verify roofline is quoted on)
    torch.cuda.synchronize()
    d0 = torch.cuda.Event(enable_timing=True); d1 = torch.cuda.Event(enable_timing=True)
    for _ in range(3):
        dsbd.node_stats(f, prm_dev, data["logits_p"], data["logits_q"], lse_p, lse_q, workspace=ws_v, stream=stream)
    n_dense = max(args.steps, 5)
    d0.record(stream)
    for _ in range(n_dense):
        dsbd.node_stats(f, prm_dev, data["logits_p"], data["logits_q"], lse_p, lse_q, workspace=ws_v, stream=stream)
    d1.record(stream)
    torch.cuda.synchronize()
    dense_ms = d0.elapsed_time(d1) / n_dense

    # the same step replayed from a CUDA graph (launch overhead removed; the decode-step counter is
    # a call argument and therefore frozen into the graph, so this is a latency figure only)
    graph_ms = None
    try:
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            stream_saved, stream = stream, side
            with torch.cuda.graph(g, stream=side):
                one_step(args.warmup)
            stream = stream_saved
        torch.cuda.synchronize()
        for _ in range(3):
            g.replay()
        r0 = torch.cuda.Event(enable_timing=True); r1 = torch.cuda.Event(enable_timing=True)
        r0.record()
        for _ in range(args.steps):
            g.replay()
        r1.record()
        torch.cuda.synchronize()
        graph_ms = r0.elapsed_time(r1) / args.steps
        del g
    except Exception as e:                                   # a figure beside the metric: never fatal
        print("graph replay skipped: %r" % (e,), file=sys.stderr)
        stream = torch.cuda.current_stream()
    assert int(status.item()) == 0, "device status %d" % int(status.item())

    # the KV-cache update of the step's output beams (reported beside the step, not part of it)
    esz = data["k_new"].element_size()
    n_slots = int(out_off[-1])
    ow = vout["out_width"].cpu().numpy().astype(np.int64)
    L_req = np.diff(poff)[np.asarray(forest["req_beam_off"][:-1])]          # beams of a request share a length
    cap = int((ow * (L_req + forest["max_depth"] + 1)).sum()) + 1
    out_off_dev = torch.as_tensor(np.asarray(out_off, dtype=np.int32)).to(dev)
    k_dst = torch.empty(cap * spec["Hkv"] * spec["d"], dtype=data["k_new"].dtype, device=dev)
    v_dst = torch.empty_like(k_dst)
    commit = None

    def kv_commit():
        return dsbd.kv_commit(f, spec["Hkv"], spec["d"], out_off_dev, vout["out_width"], vout["out_parent"],
                              vout["out_root_beam"], vout["out_logp"], data["k_new"], data["v_new"],
                              data["k_prefix"], data["v_prefix"], poff_dev, poff, n_slots=n_slots,
                              dst_capacity=cap, k_dst=k_dst, v_dst=v_dst,
                              workspace=commit["workspace"] if commit else None, status=status, stream=stream,
                              out=commit)
    for _ in range(3):
        commit = kv_commit()
    c0 = torch.cuda.Event(enable_timing=True); c1 = torch.cuda.Event(enable_timing=True)
    n_commit = max(args.steps // 4, 5)
    c0.record(stream)
    for _ in range(n_commit):
        kv_commit()
    c1.record(stream)
    torch.cuda.synchronize()
    commit_ms = c0.elapsed_time(c1) / n_commit
    commit_tokens = int(commit["new_prefix_off"][-1].item())
    commit_bytes = commit_tokens * spec["Hkv"] * spec["d"] * esz * 2 * 2      # K and V, read and write
    assert int(status.item()) == 0, "device status %d" % int(status.item())
    del k_dst, v_dst

    # the paged form of the caches: the same attention through page tables, and the cache update
    # that copies no prefix (bf16, d = 128 only)
    paged_ms = paged_commit_ms = layers_ms = None
    n_lay = 0
    if data["k_new"].dtype == torch.bfloat16 and spec["d"] == 128:
        pg = inputs.paginate(data["k_prefix"], data["v_prefix"], poff, spec["Hkv"], spec["d"],
                             extra_pages=2 * n_slots + 64, seed=int(spec["seed"]))
        attn_out_pg = torch.empty_like(attn_out)

        def attention_paged():
            dsbd.forest_attention_paged(f, spec["Hq"], spec["Hkv"], spec["d"], scale, data["q"], data["k_new"],
                                        data["v_new"], pg["k_pool"], pg["v_pool"], pg["page_table"],
                                        pg["page_off"], poff_dev, poff, out=attn_out_pg, workspace=ws_a,
                                        status=status, stream=stream)
        for _ in range(3):
            attention_paged()
        p0 = torch.cuda.Event(enable_timing=True); p1 = torch.cuda.Event(enable_timing=True)
        n_pg = max(args.steps // 2, 5)
        p0.record(stream)
        for _ in range(n_pg):
            attention_paged()
        p1.record(stream)
        torch.cuda.synchronize()
        paged_ms = p0.elapsed_time(p1) / n_pg
        assert torch.equal(attn_out_pg, attn_out), "paged and packed attention differ"
        # the attention of four transformer layers in one call: four copies of the pools, the new
        # keys/values and the queries stand for the four layers' own tensors
        layers_ms, n_lay = None, 4
        pool_bytes = pg["k_pool"].numel() * pg["k_pool"].element_size()
        if not args.no_side_workloads and 2 * n_lay * pool_bytes < 60e9:
            rep = lambda x: x.unsqueeze(0).repeat(n_lay, *([1] * x.dim()))
            kpl, vpl = rep(pg["k_pool"]), rep(pg["v_pool"])
            ql, knl, vnl = rep(data["q"]), rep(data["k_new"]), rep(data["v_new"])
            outl = torch.empty_like(ql)
            ws_l = None

            def attention_layers():
                return dsbd.forest_attention_paged(f, spec["Hq"], spec["Hkv"], spec["d"], scale, ql, knl, vnl, kpl,
                                                   vpl, pg["page_table"], pg["page_off"], poff_dev, poff, out=outl,
                                                   workspace=ws_l, status=status, stream=stream)
            for _ in range(2):
                attention_layers()
            l0 = torch.cuda.Event(enable_timing=True); l1 = torch.cuda.Event(enable_timing=True)
            n_l = max(args.steps // 4, 3)
            l0.record(stream)
            for _ in range(n_l):
                attention_layers()
            l1.record(stream)
            torch.cuda.synchronize()
            layers_ms = l0.elapsed_time(l1) / n_l
            assert all(torch.equal(outl[i], attn_out) for i in range(n_lay)), "layers differ from the single call"
            del kpl, vpl, ql, knl, vnl, outl
        table_cap = int(pg["page_table"].numel()) + 2 * n_slots
        free0, count0 = pg["free_stack"].clone(), pg["free_count"].clone()
        pc = None

        def commit_paged():
            # every call starts from the same allocator state (two small device copies)
            pg["free_stack"].copy_(free0); pg["free_count"].copy_(count0)
            return dsbd.kv_commit_paged(f, spec["Hkv"], spec["d"], out_off_dev, vout["out_width"], vout["out_parent"],
                                        vout["out_root_beam"], vout["out_logp"], data["k_new"], data["v_new"],
                                        pg["k_pool"], pg["v_pool"], pg["page_table"], pg["page_off"], poff_dev, poff,
                                        pg["free_stack"], pg["free_count"], n_slots=n_slots,
                                        table_capacity=table_cap, workspace=pc["workspace"] if pc else None,
                                        status=status, stream=stream, out=pc)
        for _ in range(3):
            pc = commit_paged()
        q0 = torch.cuda.Event(enable_timing=True); q1 = torch.cuda.Event(enable_timing=True)
        q0.record(stream)
        for _ in range(n_commit):
            commit_paged()
        q1.record(stream)
        torch.cuda.synchronize()
        paged_commit_ms = q0.elapsed_time(q1) / n_commit
        assert int(status.item()) == 0, "device status %d" % int(status.item())
        del pg, attn_out_pg

    # ---- whole decode steps: draft stage -> forest -> paged attention -> verification -> cache update
    pipeline = None
    if args.pipeline_steps > 0 and data["k_new"].dtype == torch.bfloat16 and spec["d"] == 128:
        gamma, B = int(forest["max_depth"]), f.B
        W_S = max(1, (f.N - B) // max(gamma * f.R, 1))                # the configuration's nodes per layer
        rbo_h = np.asarray(forest["req_beam_off"], dtype=np.int32)
        rbo_d = torch.as_tensor(rbo_h).to(dev)
        lay_off_h = (W_S * np.arange(f.R + 1)).astype(np.int32)
        lay_off_d = torch.as_tensor(lay_off_h).to(dev)
        ppg = inputs.paginate(data["k_prefix"], data["v_prefix"], poff, spec["Hkv"], spec["d"],
                              extra_pages=2 * n_slots + 64, seed=int(spec["seed"]))
        free0, count0 = ppg["free_stack"].clone(), ppg["free_count"].clone()
        need_rows = B + (gamma - 1) * f.R * W_S
        assert need_rows <= f.N, "not enough logits rows to stand for the draft stage"
        pout = dsbd.alloc_verify_out(f, out_off, dev)
        # attention workspace for whatever forest the draft stage samples: sized by the bound
        bound = dsbd.Forest.from_device(f.R, B, f.N, gamma, f.dev, max_tree_nodes=min(1 + gamma * W_S, 128),
                                        max_req_beams=f.max_req_beams, max_layer_nodes=W_S)
        ws_pipe = torch.empty(max(dsbd.forest_attention_workspace(bound, spec["Hq"], spec["Hkv"], spec["d"],
                                                                  data["q"].dtype, scale, poff), 256),
                              dtype=torch.uint8, device=dev)
        st = {"draft": [None] * gamma, "commit": None}
        names = ["draft", "forest", "attention", "verify", "commit"]

        def pipeline_step(step, ev):
            ev[0].record(stream)
            cur_off_h, cur_off_d, cur_s, row0 = rbo_h, rbo_d, data["root_logq"], 0
            dp, dt = [], []
            for l in range(gamma):
                n_cur = int(cur_off_h[-1])
                d = dsbd.draft_layer(cur_off_d, cur_off_h, dict(prm, step=step), l + 1, W_S,
                                     data["logits_q"][row0:row0 + n_cur], cur_s, lay_off_d, f.R * W_S,
                                     workspace=st["draft"][l]["workspace"] if st["draft"][l] else None,
                                     status=status, stream=stream, out=st["draft"][l])
                st["draft"][l] = d
                dp.append(d["out_parent"]); dt.append(d["out_token"])
                row0 += n_cur
                cur_off_h, cur_off_d, cur_s = lay_off_h, lay_off_d, d["out_logq"]
            ev[1].record(stream)
            bf, _, _ = dsbd.forest_build(rbo_d, rbo_h, gamma, W_S, torch.stack(dp), torch.stack(dt), status=status,
                                         stream=stream, exact=True)
            ev[2].record(stream)
            dsbd.forest_attention_paged(bf, spec["Hq"], spec["Hkv"], spec["d"], scale, data["q"], data["k_new"],
                                        data["v_new"], ppg["k_pool"], ppg["v_pool"], ppg["page_table"],
                                        ppg["page_off"], poff_dev, poff, out=attn_out, workspace=ws_pipe,
                                        status=status, stream=stream)
            ev[3].record(stream)
            dsbd.verify_step(bf, dict(prm_dev, step=step), data["logits_p"], data["logits_q"], data["root_logp"],
                             data["root_logq"], pout, workspace=ws_v, status=status, stream=stream)
            ev[4].record(stream)
            ppg["free_stack"].copy_(free0); ppg["free_count"].copy_(count0)
            st["commit"] = dsbd.kv_commit_paged(
                bf, spec["Hkv"], spec["d"], out_off_dev, pout["out_width"], pout["out_parent"], pout["out_root_beam"],
                pout["out_logp"], data["k_new"], data["v_new"], ppg["k_pool"], ppg["v_pool"], ppg["page_table"],
                ppg["page_off"], poff_dev, poff, ppg["free_stack"], ppg["free_count"], n_slots=n_slots,
                table_capacity=int(ppg["page_table"].numel()) + 2 * n_slots,
                workspace=st["commit"]["workspace"] if st["commit"] else None, status=status, stream=stream,
                out=st["commit"])
            ev[5].record(stream)
            return bf

        mk = lambda: [torch.cuda.Event(enable_timing=True) for _ in range(6)]
        for s_ in range(3):
            bf_last = pipeline_step(s_, mk())
        torch.cuda.synchronize()
        evs = []
        for s_ in range(args.pipeline_steps):
            e = mk(); pipeline_step(3 + s_, e); evs.append(e)
        torch.cuda.synchronize()
        assert int(status.item()) == 0, "device status %d" % int(status.item())
        parts = {n: float(np.median([e[i].elapsed_time(e[i + 1]) for e in evs])) for i, n in enumerate(names)}
        total = float(np.median([e[0].elapsed_time(e[5]) for e in evs]))
        pipeline = {"ms_per_step": total, "nodes_per_s": f.N / total * 1e3, "parts_ms": parts, "gamma": gamma,
                    "W_S": W_S, "largest_tree": bf_last.max_tree_nodes, "steps": args.pipeline_steps,
                    "note": "every step starts from the same beams and caches; the forest is the one the draft "
                            "stage samples (ragged trees), the models' rows are the synthetic tensors"}
        del ppg

    # one draft-stage sampling step of the same shape (W_S = beams of the request), reported
    # beside the step: the small model's logits of the first B rows stand for a draft layer
    rbo_host = np.asarray(forest["req_beam_off"], dtype=np.int32)
    W_S_r = torch.as_tensor(np.diff(rbo_host).astype(np.int32)).to(dev)
    rbo_dev = torch.as_tensor(rbo_host).to(dev)
    zq_rows = data["logits_q"][:f.B]
    draft = None

    def draft_layer():
        return dsbd.draft_layer(rbo_dev, rbo_host, prm, 1, W_S_r, zq_rows, data["root_logq"], rbo_dev, f.B,
                                workspace=draft["workspace"] if draft else None, status=status, stream=stream,
                                out=draft)
    for _ in range(3):
        draft = draft_layer()
    g0 = torch.cuda.Event(enable_timing=True); g1 = torch.cuda.Event(enable_timing=True)
    n_draft = max(args.steps, 5)
    g0.record(stream)
    for _ in range(n_draft):
        draft_layer()
    g1.record(stream)
    torch.cuda.synchronize()
    draft_ms = g0.elapsed_time(g1) / n_draft
    draft_bytes = 4 * f.B * spec["V"]
    assert int(status.item()) == 0, "device status %d" % int(status.item())

    # end to end through the C ABI with host buffers
    e2e = None
    if args.e2e_steps > 0:
        names = ["q", "k_new", "v_new", "k_prefix", "v_prefix", "logits_p", "logits_q", "root_logp", "root_logq"]
        host = {k: data[k].cpu().pin_memory() for k in names}
        host_forest = {k: torch.from_numpy(np.ascontiguousarray(forest[k], dtype=np.int32)).pin_memory()
                       for k in ("req_beam_off", "beam_node_off", "parent", "token")}
        h2d = sum(v.numel() * v.element_size() for v in host.values()) + \
            sum(v.numel() * v.element_size() for v in host_forest.values())
        res_keys = ["l_last", "out_width", "out_parent", "out_node", "out_root_beam", "out_token", "out_logp",
                    "out_logq", "out_source", "node_status", "layer_width"]
        host_res = {k: torch.empty_like(vout[k], device="cpu").pin_memory() for k in res_keys}
        host_attn = torch.empty_like(attn_out, device="cpu").pin_memory()
        d2h = sum(v.numel() * v.element_size() for v in host_res.values()) + host_attn.numel() * host_attn.element_size()

        def e2e_step(step):
            for k in names:
                data[k].copy_(host[k], non_blocking=True)
            for k, v in host_forest.items():
                f.dev[k].copy_(v, non_blocking=True)
            one_step(step)
            host_attn.copy_(attn_out, non_blocking=True)
            for k in res_keys:
                host_res[k].copy_(vout[k], non_blocking=True)

        e2e_step(0)
        barrier()
        s0 = torch.cuda.Event(enable_timing=True); s1 = torch.cuda.Event(enable_timing=True)
        s0.record(stream)
        for s in range(args.e2e_steps):
            e2e_step(s + 1)
        s1.record(stream)
        barrier()
        te = max_over_ranks(s0.elapsed_time(s1), world, dev)
        e2e = {"value": job_value(f.N, world, te / args.e2e_steps), "unit": UNIT,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": args.e2e_steps}
        del host

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = _peaks()
    a_bytes = inputs.attention_bytes(spec, forest, poff)
    v_bytes = inputs.verify_bytes(spec, forest)
    kernels = {
        "forest_attention": {"bytes": a_bytes, "ms": attn_ms, "gbs": a_bytes / attn_ms * 1e-6},
        "verify_dense_pass": {"bytes": v_bytes, "ms": dense_ms, "gbs": v_bytes / dense_ms * 1e-6},
        "verify_step_total": {"bytes": v_bytes, "ms": ver_ms, "gbs": v_bytes / ver_ms * 1e-6},
        "kv_commit": {"bytes": commit_bytes, "ms": commit_ms, "gbs": commit_bytes / commit_ms * 1e-6},
        "draft_layer": {"bytes": draft_bytes, "ms": draft_ms, "gbs": draft_bytes / draft_ms * 1e-6},
    }
    if paged_ms is not None:
        kernels["forest_attention_paged"] = {"bytes": a_bytes, "ms": paged_ms, "gbs": a_bytes / paged_ms * 1e-6}
        # the paged update moves only partial pages and paths; the same kept-cache bytes as
        # kv_commit are the work it replaces, so no bandwidth figure is given
        kernels["kv_commit_paged"] = {"bytes": 0, "ms": paged_commit_ms, "gbs": 0.0}
    if layers_ms is not None:
        kernels["forest_attention_paged_%dlayers" % n_lay] = {"bytes": n_lay * a_bytes, "ms": layers_ms,
                                                               "gbs": n_lay * a_bytes / layers_ms * 1e-6}
    for k in kernels.values():
        k["frac_of_%s_peak" % peak_kind] = k["gbs"] / peak
        k["frac_of_8TBs_nominal"] = k["gbs"] / 8000.0
    # The step has two parts, both bound by HBM: the attention kernel (the longest kernel of the
    # step) and the verification (dense pass + per-request kernel).  The headline entry is the
    # part with the LOWER fraction of peak, so a part that misses its target shows on the line;
    # both are listed under "parts".
    def part(name):
        return {"kernel": name, "bound": "hbm", "achieved": kernels[name]["gbs"], "peak": peak,
                "peak_kind": peak_kind, "unit": "GB/s", "frac": kernels[name]["gbs"] / peak,
                "frac_of_8TBs_nominal": kernels[name]["gbs"] / 8000.0,
                "traffic": NCU_TRAFFIC_BYTES.get(args.workload, {}).get(name) if args.requests <= 0 else None,
                "algorithmic_bytes": kernels[name]["bytes"], "ms": kernels[name]["ms"]}
    parts_rl = [part("forest_attention"), part("verify_step_total"), part("verify_dense_pass")]
    roofline = dict(min(parts_rl[:2], key=lambda x: x["frac"]))
    roofline["parts"] = parts_rl
    if roofline["frac"] > 1.0:
        roofline["note"] = "above 1: the peak is a read+write copy, a read-only stream runs faster"

    if not args.no_side_workloads and world == 1 and args.requests <= 0:
        side_steps, side_warm = max(5, min(args.steps, 30)), 3
        torch.cuda.empty_cache()
        for wname in ("C4", "C6"):
            if wname != args.workload:
                for k, v in _side_workload(dsbd, inputs, dev, wname, side_steps, side_warm).items():
                    kernels["%s.%s" % (wname, k)] = v
        if args.top_k == 0:
            w = _side_workload(dsbd, inputs, dev, args.workload, side_steps, side_warm, top_k=10, top_p=0.8,
                               parts=("verify",))
            kernels["%s.verify_step_total_topk10_topp0.8" % args.workload] = w["verify_step_total"]
        for name, k in kernels.items():
            if "." in name:
                k["frac_of_%s_peak" % peak_kind] = k["gbs"] / peak
                k["frac_of_8TBs_nominal"] = k["gbs"] / 8000.0

    cpu, parity = None, None
    if not args.no_cpu_baseline:
        # the library's results at the Philox step of the inputs' parameters, for the comparison with
        # the oracle's sample (what the oracle computes on the way is compared, nothing is added to it)
        attention()
        verify(int(prm.get("step", 0)))
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        gpu_res = {k: vout[k].cpu().numpy() for k in ("l_last", "out_width", "layer_width", "node_status",
                                                      "out_token", "out_source", "out_parent")}
        gpu_res["layer_width"] = gpu_res["layer_width"].reshape(f.R, -1)
        gpu_res["out_off"] = np.asarray(out_off)
        gpu_res["attn_out"] = attn_out.float().cpu().numpy()
        cpu, parity = _cpu_baseline(_host_views(data, spec), spec, os.cpu_count() or 1, gpu=gpu_res)
        parity["note"] = ("the oracle's sample of the cpu_baseline leg against this run's outputs; a mismatching "
                          "request is one whose layer widths, node statuses or output beams differ in any entry")

    # kernels of this library per step: the attention kernel (plus its plan / combine kernels when
    # the launch shape uses them), the dense logits pass and the per-request verification kernel
    launches_per_step = dsbd.forest_attention_launches(f, spec["Hq"], spec["Hkv"], spec["d"], data["q"].dtype,
                                                       scale, poff) + 2
    ms_per_step = total_ms / args.steps
    line = {"metric": METRIC, "value": job_value(f.N, world, ms_per_step), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16 attention / f32 logits", "data": "synthetic",
            "config": {"workload": args.workload, "requests": f.R, "beams": f.B, "nodes": f.N,
                       "heads": "%dq/%dkv x %d" % (spec["Hq"], spec["Hkv"], spec["d"]), "vocab": spec["V"],
                       "prefix": list(spec["prefix"]), "temperature": spec["temperature"],
                       "thresh": prm["thresh"], "top_k": args.top_k, "top_p": args.top_p, "l2": ("inputs (%.1f GB) far exceed the 126 MB L2; no flush" % ((a_bytes + v_bytes) * 1e-9)) if flush is None
                       else "inputs (%.0f MB) would fit the 126 MB L2: flushed by a 256 MB write between steps" % (
                           (a_bytes + v_bytes) * 1e-6),
                       "parallelism": "replicas x%d" % world},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline, "kernels": kernels, "graph_replay_ms_per_step": graph_ms, "pipeline": pipeline,
            "verify_stats_last_step": verify_stats, "cpu_baseline": cpu, "parity": parity}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
