"""A bounded wait of the tensor-core attention kernel that runs out.

Every mbarrier wait of that kernel gives up after a limit, records DSBD_DEV_TIMEOUT, lets the
copies in flight land, frees its tensor memory and returns.  The product library offers no way
to make a wait run out, so this test builds a second library from the same sources with
DSBD_TEST_WAIT_TIMEOUT: the limit drops to about a millisecond and the copy producer of one CTA
leaves out one tile, whose barrier is then never completed.  Nothing faults and nothing hangs:
the call returns with the status set, the other CTAs finish their work, and the next launch
of the product library on the same context matches the oracle."""
import ctypes as C

import numpy as np
import pytest
import torch

import paper_2409_16560_b200 as dsbd
from paper_2409_16560_b200 import binding as bd
from paper_2409_16560_b200 import build as cuda_build
from paper_2409_16560_b200 import inputs
from parity_util import attention_close, to_host_f32
from test_gpu_attention import _custom, _gpu, _oracle_beams

pytestmark = pytest.mark.gpu

DEV_TIMEOUT = 5


def test_a_wait_that_runs_out_sets_the_status_and_leaves_the_context_usable():
    lib = C.CDLL(cuda_build.build_wait_test())
    lib.dsbd_forest_attention_workspace.restype = C.c_size_t
    lib.dsbd_forest_attention_workspace.argtypes = [C.c_void_p, C.c_void_p]
    lib.dsbd_forest_attention.restype = C.c_int
    lib.dsbd_forest_attention.argtypes = [C.c_void_p] * 10 + [C.c_size_t, C.c_void_p, C.c_void_p]

    rng = np.random.default_rng(31)
    rand_tree = lambda n: [-1] + [int(rng.integers(0, i)) for i in range(1, n)]
    trees = [rand_tree(9), rand_tree(5), rand_tree(12), rand_tree(3)]
    L = [700, 300, 1000, 200]                              # every unit has several tiles
    forest, spec, t, poff = _custom(rng, trees, L, 8, 2, 128, torch.bfloat16)
    f = dsbd.Forest(forest, "cuda")
    fs = f.struct()
    desc = bd._attn_desc(8, 2, 128, torch.bfloat16, inputs.default_scale(128), poff)
    poff_dev = torch.as_tensor(poff).cuda()
    out = torch.zeros_like(t["q"])
    need = int(lib.dsbd_forest_attention_workspace(C.addressof(fs), C.addressof(desc)))
    ws = torch.zeros(max(need, 256), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rc = lib.dsbd_forest_attention(C.addressof(fs), C.addressof(desc), t["q"].data_ptr(), t["k_new"].data_ptr(),
                                   t["v_new"].data_ptr(), t["k_prefix"].data_ptr(), t["v_prefix"].data_ptr(),
                                   poff_dev.data_ptr(), out.data_ptr(), ws.data_ptr(), ws.numel(), status.data_ptr(),
                                   torch.cuda.current_stream().cuda_stream)
    assert rc == 0
    torch.cuda.synchronize()                               # returns: the wait was bounded
    assert int(status.item()) == DEV_TIMEOUT
    assert "wait" in dsbd.status_string(DEV_TIMEOUT)
    # the CTAs whose tiles all arrived did their work: the last tree's rows are right
    nodes, ref = _oracle_beams(forest, spec, t, poff, list(range(len(trees))))
    bno = forest["beam_node_off"]
    last = slice(int(bno[-2]), int(bno[-1]))
    attention_close(to_host_f32(out[last]), ref[last], bf16=True)
    # the context is intact (tensor memory freed, no copy left in flight): the product library's
    # next launch on the same device gives the full, correct result
    good = _gpu(forest, spec, t, poff)
    attention_close(to_host_f32(good), ref, bf16=True)
