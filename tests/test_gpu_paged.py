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


@pytest.mark.parametrize("name,kw,n_beams", [("C2", {}, None), ("C3", {}, 3), ("C4", {}, 4), ("C5", dict(R=3), 2)])
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


def test_unsupported_shapes_are_refused():
    rng = np.random.default_rng(0)
    forest, spec, t, poff = _custom(rng, [[-1, 0]], [100], 4, 4, 64, torch.float32)
    pg = _paged(t, poff, 4, 64, 1, rng)
    with pytest.raises(dsbd.DsbdError):
        dsbd.forest_attention_paged(dsbd.Forest(forest, "cuda"), 4, 4, 64, 0.125, t["q"], t["k_new"], t["v_new"],
                                    pg["k_pool"], pg["v_pool"], pg["table"], pg["page_off"],
                                    torch.as_tensor(poff).cuda(), poff)
