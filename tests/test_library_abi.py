"""The C-ABI library builds for sm_100a, loads, and exports every symbol include/dsbd.h declares
(no compute calls: this runs without a GPU)."""
import ctypes
import os
import re

import paper_2409_16560_b200 as dsbd
from paper_2409_16560_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "dsbd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dsbd_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    lib = dsbd.load()
    names = _declared()
    assert set(binding.EXPORTS) <= set(names)
    for n in names:
        assert hasattr(lib, n), n
        assert isinstance(getattr(lib, n), ctypes._CFuncPtr)


def test_status_strings_and_workspace_queries_without_a_device():
    assert dsbd.status_string(0) == "ok"
    assert "workspace" in dsbd.status_string(-3)
    lib = dsbd.load()
    f = binding.ForestT()
    p = binding.VerifyParamsT()
    assert lib.dsbd_verify_workspace(ctypes.addressof(f), ctypes.addressof(p)) == 0   # invalid -> 0


def test_no_cpu_fallback():
    import numpy as np
    import pytest
    import torch
    arrays = dict(R=1, B=1, N=1, max_depth=0, req_beam_off=[0, 1], beam_node_off=[0, 1], parent=[-1], token=[0])
    f = dsbd.Forest(arrays, "cpu")
    z = torch.zeros(1, 8)
    out = dsbd.alloc_verify_out(f, np.array([0, 1]), "cpu")
    with pytest.raises(RuntimeError):
        dsbd.verify_step(f, dict(V=8), z, z, torch.zeros(1), torch.zeros(1), out)


def test_header_is_plain_c(tmp_path):
    """include/dsbd.h is a C header: a C99 compiler accepts it with warnings as errors."""
    import shutil
    import subprocess
    import pytest
    if shutil.which("gcc") is None:
        pytest.skip("no C compiler")
    src = tmp_path / "use_header.c"
    src.write_text('#include "dsbd.h"\n'
                   "int main(void) { dsbd_forest_t f; dsbd_verify_params_t p; dsbd_commit_params_t c;\n"
                   "  (void)f; (void)p; (void)c; return dsbd_status_string(0) == 0; }\n")
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only",
                    "-I", os.path.join(ROOT, "include"), str(src)], check=True)


def test_forest_depths_match_a_plain_walk():
    """The binding computes node depths (they size the verification's launches) with array
    operations; a plain walk over the parent array must agree on random trees."""
    import numpy as np
    from paper_2409_16560_b200.binding import _node_depths
    rng = np.random.default_rng(0)
    for _ in range(100):
        n = int(rng.integers(1, 400))
        parent = np.array([-1] + [int(rng.integers(-1, i)) for i in range(1, n)])
        ref = np.zeros(n, np.int64)
        for i, p in enumerate(parent):
            ref[i] = 0 if p < 0 else ref[p] + 1
        assert np.array_equal(_node_depths(parent), ref)
