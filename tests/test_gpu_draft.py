"""GPU parity of dsbd_draft_layer against the oracle: the beam each draw extends and its token
are compared bit for bit (a draw whose uniform lies within 1e-6 of a boundary of its cell's CDF
interval may differ and is counted in the "draw" class of the parity helper), the new
cumulative score within 1e-4 + 1e-5 |oracle|."""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2409_16560_b200 as dsbd
import parity_util

pytestmark = pytest.mark.gpu


def _problem(rng, beams_per_req, V, sigma=3.0, zipf=True, stride=None):
    rbo = np.concatenate([[0], np.cumsum(beams_per_req)]).astype(np.int32)
    n = int(rbo[-1])
    bias = -np.log1p(rng.permutation(V)) if zipf else np.zeros(V)
    z = (rng.normal(0, sigma, size=(n, V)) + bias).astype(np.float32)
    s = rng.normal(-5, 1.5, size=n).astype(np.float32)
    return rbo, z, s


def _both(rbo, z, s, prm, layer, W_S, out_off=None, stride=None):
    R = len(rbo) - 1
    W_r = np.full(R, W_S, np.int32) if np.isscalar(W_S) else np.asarray(W_S, np.int32)
    if out_off is None:
        out_off = np.concatenate([[0], np.cumsum(W_r)]).astype(np.int32)
    ref = oracle.draft_layer(rbo, prm, layer, W_r, z, s.astype(np.float64), out_off=out_off)
    zd = torch.as_tensor(z).cuda()
    if stride is not None:
        buf = torch.zeros(z.shape[0], stride, device="cuda")
        buf[:, :z.shape[1]] = zd
        zd = buf                      # padded rows; the call gets row_stride
    gpu = dsbd.draft_layer(torch.as_tensor(rbo).cuda(), rbo, prm, layer,
                           W_S if np.isscalar(W_S) else torch.as_tensor(W_r).cuda(), zd,
                           torch.as_tensor(s).cuda(), torch.as_tensor(np.asarray(out_off, np.int32)).cuda(),
                           int(out_off[-1]), row_stride=stride)
    torch.cuda.synchronize()
    return ref, {k: v.cpu().numpy() for k, v in gpu.items() if k != "workspace"}, W_r, out_off


def _compare(ref, gpu, W_r, out_off):
    exempt = draws = 0
    assert np.array_equal(ref["error"], gpu["req_error"])
    for r in range(len(W_r)):
        if ref["error"][r]:
            continue
        for k in range(W_r[r]):
            s = out_off[r] + k
            draws += 1
            same = ref["out_parent"][s] == gpu["out_parent"][s] and ref["out_token"][s] == gpu["out_token"][s]
            if not same:
                u = oracle.uniform(ref_prm["seed"], ref_prm["step"], r, (1 << 29) + ref_layer, 3, k)
                near = min(abs(u - ref["cdf_lo"][s]), abs(ref["cdf_hi"][s] - u)) < parity_util.DRAW_BAND
                assert near, (r, k, ref["out_parent"][s], gpu["out_parent"][s], ref["out_token"][s], gpu["out_token"][s])
                exempt += 1
                continue
            x, y = ref["out_logq"][s], gpu["out_logq"][s]
            assert abs(x - y) <= 1e-4 + 1e-5 * abs(x), (r, k, x, y)
    # a sampled token may differ only inside a tie of the cumulative distribution (fp32 cell masses
    # on the device, fp64 in the oracle); counted with the verification's draws
    parity_util.check_exempt(parity_util.Exempt(draw=exempt), draws)
    # slots past a request's W_S draws keep their initial -1
    used = np.zeros(len(gpu["out_token"]), bool)
    for r in range(len(W_r)):
        # (a request that reported an error leaves its own slot range unspecified)
        used[out_off[r]:(out_off[r + 1] if ref["error"][r] else out_off[r] + W_r[r])] = True
    assert (gpu["out_token"][~used] == -1).all() and (gpu["out_parent"][~used] == -1).all()
    return draws


ref_prm, ref_layer = {}, 0


def _case(rng, beams, V, W_S, layer, stride=None, **kw):
    global ref_prm, ref_layer
    rbo, z, s = _problem(rng, beams, V)
    prm = dict(V=V, temperature=kw.pop("temperature", 1.0), seed=kw.pop("seed", 7), step=kw.pop("step", 0), **kw)
    ref_prm, ref_layer = prm, layer
    ref, gpu, W_r, out_off = _both(rbo, z, s, prm, layer, W_S, stride=stride)
    assert int(gpu["status"][0]) == 0
    return _compare(ref, gpu, W_r, out_off)


@pytest.mark.parametrize("V", [1000, 32000, 128256])
@pytest.mark.parametrize("top_k,top_p", [(0, 1.0), (10, 0.8)])
def test_first_and_later_layers(V, top_k, top_p):
    rng = np.random.default_rng(V + top_k)
    R = 6 if V > 100000 else 12
    # first draft layer: the input beams (ragged counts); later layers: W_S beams per request
    assert _case(rng, rng.integers(1, 9, size=R), V, 12, 1, top_k=top_k, top_p=top_p, temperature=0.8) == 12 * R
    assert _case(rng, np.full(R, 12), V, 12, 3, top_k=top_k, top_p=top_p, step=5) == 12 * R


def test_per_request_widths_ragged_vocab_and_row_stride():
    rng = np.random.default_rng(4)
    W = rng.integers(0, 17, size=9)
    _case(rng, rng.integers(1, 6, size=9), 5003, W, 2, stride=5008)
    _case(rng, rng.integers(1, 6, size=9), 2100, W, 2, stride=2101, top_k=64, top_p=0.95)


def test_many_draws_follow_the_stream():
    rng = np.random.default_rng(5)
    for step in range(20):
        _case(rng, [4, 2, 7], 3000, 64, 1, step=step)


def test_the_largest_live_set():
    rng = np.random.default_rng(8)
    _case(rng, [64, 1, 64], 4096, 64, 5)
    _case(rng, [64, 64], 1500, 64, 2, top_k=64, top_p=0.9)


def test_capacity_error_is_per_request():
    rng = np.random.default_rng(6)
    rbo, z, s = _problem(rng, [2, 3], 1000)
    prm = dict(V=1000, seed=1)
    global ref_prm, ref_layer
    ref_prm, ref_layer = dict(prm, step=0), 1
    ref, gpu, W_r, out_off = _both(rbo, z, s, prm, 1, 4, out_off=np.array([0, 3, 7], np.int32))
    assert list(ref["error"]) == [3, 0] and int(gpu["status"][0]) == 3
    _compare(ref, gpu, W_r, out_off)


def test_host_side_errors():
    z = torch.zeros(2, 100, device="cuda")
    s = torch.zeros(2, device="cuda")
    off = torch.tensor([0, 2], dtype=torch.int32, device="cuda")
    with pytest.raises(dsbd.DsbdError):        # top-p without top-k
        dsbd.draft_layer(off, [0, 2], dict(V=100, top_p=0.5), 1, 2, z, s, off, 2)
    with pytest.raises(dsbd.DsbdError):        # more beams in a request than the kernel's live limit
        dsbd.draft_layer(torch.tensor([0, 70], dtype=torch.int32, device="cuda"), [0, 70], dict(V=100), 1, 2,
                         torch.zeros(70, 100, device="cuda"), torch.zeros(70, device="cuda"), off, 2)
