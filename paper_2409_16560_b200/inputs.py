"""Seeded synthetic inputs for the five benchmark configurations.

This module holds input generation only -- forest topologies, random tensors, draft tokens --
and none of the method's arithmetic; both the CUDA library's harness and the tests' oracle
read the bytes it produces.  The shapes stand in for the 7B/8B-class target models the
method was evaluated with (32 heads x 128, vocabulary 32000; 32 query / 8 KV heads x 128,
vocabulary 128256); logits are Gaussian with a Zipf-shaped bias, the small model's logits are
the large model's plus noise, and every draft token is drawn from the small model's
next-token distribution at its parent.
"""
import math

import numpy as np
import torch

# name -> specification.  "tree": local parent array of one draft tree (root first).
def _chain(depth):
    return [-1] + list(range(depth))


def _binary(depth):
    n = 2 ** (depth + 1) - 1
    return [-1] + [(i - 1) // 2 for i in range(1, n)]


def _wide_tree():
    # level sizes 1,2,4,4,4,4,1: branching 2 at the first two levels, then four chains of which
    # only the first reaches depth 6
    par = [-1, 0, 0, 1, 1, 2, 2]
    par += [3, 4, 5, 6]          # depth 3: nodes 7..10
    par += [7, 8, 9, 10]         # depth 4: 11..14
    par += [11, 12, 13, 14]      # depth 5: 15..18
    par += [15]                  # depth 6: 19
    return par


CONFIGS = {
    "C1": dict(R=1, W=2, tree=_binary(3), Hq=4, Hkv=4, d=64, dtype="f32", prefix=(64, 64), V=1000,
               sigma_p=2.0, zipf=False, sigma_n=0.5, temperature=1.0, seed=0),
    "C2": dict(R=1, W=4, tree=_chain(4), Hq=32, Hkv=32, d=128, dtype="bf16", prefix=(512, 512),
               V=32000, sigma_p=3.0, zipf=True, sigma_n=1.0, temperature=1.0, seed=0),
    "C3": dict(R=4, W=8, tree=_wide_tree(), Hq=32, Hkv=32, d=128, dtype="bf16", prefix=(2048, 2048),
               V=32000, sigma_p=3.0, zipf=True, sigma_n=1.0, temperature=1.0, seed=0),
    "C4": dict(R=16, W=(1, 8), tree=_chain(5), Hq=32, Hkv=8, d=128, dtype="bf16", prefix=(1024, 4096),
               V=128256, sigma_p=3.0, zipf=True, sigma_n=1.0, temperature=1.0, seed=0),
    "C5": dict(R=64, W=8, tree=_chain(8), Hq=32, Hkv=8, d=128, dtype="bf16", prefix=(4096, 4096),
               V=128256, sigma_p=3.0, zipf=True, sigma_n=1.0, temperature=0.8, seed=7),
    # a sixth shape beside the five benchmark configurations: 40 heads of 128 without grouping and
    # a 32000-token vocabulary, the dimensions of the 13B model of the paper's experiments; the
    # batch, widths, depth and prefix length are this build's choice
    "C6": dict(R=8, W=4, tree=_chain(5), Hq=40, Hkv=40, d=128, dtype="bf16", prefix=(2048, 2048),
               V=32000, sigma_p=3.0, zipf=True, sigma_n=1.0, temperature=1.0, seed=0),
}


def config(name, **overrides):
    spec = dict(CONFIGS[name])
    spec.update(overrides)
    spec["name"] = name
    return spec


def build_forest(spec, rng):
    """Forest arrays (numpy) of a configuration: per-request widths, trees, prefix lengths."""
    R = spec["R"]
    W = spec["W"]
    widths = (rng.integers(W[0], W[1] + 1, size=R) if isinstance(W, tuple) else np.full(R, W)).astype(np.int64)
    lo, hi = spec["prefix"]
    L_req = rng.integers(lo, hi + 1, size=R) if hi > lo else np.full(R, lo)
    tree = np.asarray(spec["tree"], dtype=np.int64)
    n_tree = len(tree)
    B = int(widths.sum())
    N = B * n_tree
    base = np.arange(B)[:, None] * n_tree
    parent = np.where(tree[None, :] >= 0, tree[None, :] + base, -1).reshape(-1).astype(np.int32)
    depth = np.zeros(n_tree, np.int64)
    for i, p in enumerate(tree):
        depth[i] = 0 if p < 0 else depth[p] + 1
    forest = dict(R=R, B=B, N=N, max_depth=int(depth.max()),
                  req_beam_off=np.concatenate([[0], np.cumsum(widths)]).astype(np.int32),
                  beam_node_off=(np.arange(B + 1) * n_tree).astype(np.int32),
                  parent=parent, token=np.zeros(N, np.int32))
    L_beam = np.repeat(L_req, widths).astype(np.int64)
    prefix_off = np.concatenate([[0], np.cumsum(L_beam)]).astype(np.int64)
    return forest, widths, prefix_off


def generate(spec, device, parts=("attention", "verify"), draft_top_k=0, draft_top_p=1.0):
    """All tensors of one decode step on `device`, from one seeded torch generator.

    draft_top_k / draft_top_p: when set, every draft token is drawn by ordinary per-row top-k /
    top-p sampling from the small model's next-token distribution (the usual sampler of a
    draft model run with warping), so the drafts are high-probability tokens.

    Returns a dict: forest (numpy arrays), widths, prefix_off (numpy int64), params (python
    scalars + per-request width arrays as numpy), and the torch tensors q, k_new, v_new,
    k_prefix, v_prefix, logits_p, logits_q, root_logp, root_logq."""
    seed = int(spec["seed"])
    rng = np.random.default_rng(seed)
    forest, widths, prefix_off = build_forest(spec, rng)
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    N, B = forest["N"], forest["B"]
    Hq, Hkv, d, V = spec["Hq"], spec["Hkv"], spec["d"], spec["V"]
    dtype = torch.bfloat16 if spec["dtype"] == "bf16" else torch.float32
    out = dict(spec=spec, forest=forest, widths=widths, prefix_off=prefix_off)

    def randn(*shape, dt=torch.float32):
        return torch.randn(*shape, generator=gen, device=device, dtype=torch.float32).to(dt)

    if "attention" in parts:
        out["q"] = randn(N, Hq, d, dt=dtype)
        out["k_new"] = randn(N, Hkv, d, dt=dtype)
        out["v_new"] = randn(N, Hkv, d, dt=dtype)
        total = int(prefix_off[-1])
        kp = torch.empty(total * Hkv * d, dtype=dtype, device=device)
        vp = torch.empty(total * Hkv * d, dtype=dtype, device=device)
        chunk = 1 << 24
        for t in (kp, vp):
            for s in range(0, t.numel(), chunk):
                e = min(s + chunk, t.numel())
                t[s:e] = randn(e - s, dt=dtype)
        out["k_prefix"], out["v_prefix"] = kp, vp

    if "verify" in parts:
        tau = float(spec["temperature"])
        if spec["zipf"]:
            perm = torch.randperm(V, generator=gen, device=device)
            bias = -torch.log1p(perm.to(torch.float32))
        else:
            bias = torch.zeros(V, device=device)
        zp = torch.empty(N, V, dtype=torch.float32, device=device)
        zq = torch.empty(N, V, dtype=torch.float32, device=device)
        rows = max(1, (1 << 24) // V)
        for s in range(0, N, rows):
            e = min(s + rows, N)
            zp[s:e] = randn(e - s, V) * spec["sigma_p"] + bias
            zq[s:e] = zp[s:e] + randn(e - s, V) * spec["sigma_n"]
        out["logits_p"], out["logits_q"] = zp, zq
        out["root_logp"] = randn(B)
        out["root_logq"] = out["root_logp"] + 0.5 * randn(B)
        # draft tokens: node n's token ~ softmax(z_q[parent(n)] / tau)
        parent = torch.from_numpy(forest["parent"]).to(device)
        nonroot = torch.nonzero(parent >= 0).squeeze(1)
        token = torch.zeros(N, dtype=torch.int64, device=device)
        for s in range(0, nonroot.numel(), rows):
            idx = nonroot[s:s + rows]
            probs = torch.softmax(zq[parent[idx].long()] / tau, dim=1)
            if draft_top_k > 0:
                top, ids = torch.topk(probs, min(int(draft_top_k), V), dim=1)
                if 0.0 < draft_top_p < 1.0:
                    top = top / top.sum(1, keepdim=True)
                    before = torch.cumsum(top, 1) - top
                    top = torch.where(before < draft_top_p, top, torch.zeros_like(top))
                pick = torch.multinomial(top, 1, generator=gen)
                token[idx] = ids.gather(1, pick).squeeze(1)
            else:
                token[idx] = torch.multinomial(probs, 1, generator=gen).squeeze(1)
        forest["token"] = token.to(torch.int32).cpu().numpy()
        W_cfg = spec["W"][1] if isinstance(spec["W"], tuple) else spec["W"]
        out["params"] = dict(V=V, temperature=tau, thresh=0.7, W_min=1, W_max=W_cfg, W_nom=W_cfg,
                             W_min_r=np.minimum(2, widths).astype(np.int32),
                             seed=seed, step=0)
    return out


PAGE_TOKENS = 64


def paginate(k_prefix, v_prefix, prefix_off, Hkv, d, extra_pages, seed=0):
    """The packed caches cut into pages of 64 tokens with shuffled page ids (layout change only).
    Returns dict(k_pool, v_pool [n_pages, Hkv, 64, d], page_table int32, page_off int64 [B+1],
    free_stack int32 [n_pages], free_count int32 [1]); rows past a cache's length are zero."""
    dev = k_prefix.device
    L = np.diff(np.asarray(prefix_off))
    need = [int(-(-int(l) // PAGE_TOKENS)) for l in L]
    total = int(sum(need))
    n_pages = total + int(extra_pages)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    ids = torch.randperm(n_pages, generator=gen)
    k_pool = torch.zeros(n_pages, Hkv, PAGE_TOKENS, d, dtype=k_prefix.dtype, device=dev)
    v_pool = torch.zeros_like(k_pool)
    page_off = np.concatenate([[0], np.cumsum(need)]).astype(np.int64)
    for b, l in enumerate(L):
        l = int(l)
        if l == 0:
            continue
        base = int(prefix_off[b]) * Hkv * d
        pages = ids[int(page_off[b]):int(page_off[b + 1])].to(dev)
        for src, pool in ((k_prefix, k_pool), (v_prefix, v_pool)):
            x = src[base:base + Hkv * l * d].view(Hkv, l, d)
            pad = need[b] * PAGE_TOKENS - l
            if pad:
                x = torch.cat([x, torch.zeros(Hkv, pad, d, dtype=x.dtype, device=dev)], dim=1)
            pool[pages] = x.view(Hkv, need[b], PAGE_TOKENS, d).permute(1, 0, 2, 3)
    free = torch.sort(ids[total:]).values.to(torch.int32)
    free_stack = torch.zeros(n_pages, dtype=torch.int32)
    free_stack[:free.numel()] = free
    return dict(k_pool=k_pool, v_pool=v_pool, page_table=ids[:total].to(torch.int32).to(dev),
                page_off=torch.as_tensor(page_off).to(dev), free_stack=free_stack.to(dev),
                free_count=torch.tensor([free.numel()], dtype=torch.int32, device=dev))


def attention_bytes(spec, forest, prefix_off):
    """Algorithmic HBM bytes of one forest-attention launch: the KV prefix of every beam once
    (K and V), plus Q, O and the new K/V of every node."""
    esz = 2 if spec["dtype"] == "bf16" else 4
    kv = int(prefix_off[-1]) * spec["Hkv"] * spec["d"] * 2 * esz
    qo = forest["N"] * (2 * spec["Hq"] + 2 * spec["Hkv"]) * spec["d"] * esz
    return kv + qo


def verify_bytes(spec, forest):
    """Algorithmic HBM bytes of one verification step: every logits row of both models once."""
    return 8 * forest["N"] * spec["V"]


def default_scale(d):
    return 1.0 / math.sqrt(d)
