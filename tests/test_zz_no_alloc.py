"""The no-allocation entry point against the ordinary one.

Some callers cannot call cudaMalloc (a pool owns the device, or an allocation's implicit
synchronisation is not acceptable where they run).  monarch_attn_fwd_noalloc serves them with
scratch that is part of the library image.  This file is collected last on purpose: if it fails,
a run that stops at the first failure has already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import __graft_entry__ as entry
from paper_2505_18698_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    entry.build()
    return binding.load_library()


@pytest.mark.parametrize("dtype,tol", [("f32", 1e-6), ("bf16", 1e-2)])
def test_noalloc_matches_existing_entry_point_on_two_calls_in_a_row(dtype, tol):
    # two different problems back to back: the second call finds the first call's states in the
    # shared scratch and must not be disturbed by them
    cases = [dict(batch=2, heads=3, N=256, d=64, b=16, T=2, seed=3),
             dict(batch=1, heads=2, N=384, d=64, b=24, T=3, seed=4)]
    for c in cases:
        Q, K, V = wl.make_qkv(c["batch"], c["heads"], c["N"], c["d"], dtype, 4, 1.0, c["seed"])
        Qd, Kd, Vd = (binding.to_device(x, dtype) for x in (Q, K, V))
        Y = torch.empty_like(Qd)
        binding.monarch_attn_fwd_noalloc(Qd, Kd, Vd, c["b"], c["T"], Y)
        torch.cuda.synchronize()
        ref = binding.monarch_attn_fwd_ex(Qd, Kd, Vd, c["b"], c["T"], path=binding.MA_PATH_GENERIC)
        torch.cuda.synchronize()
        a = Y.float().cpu().numpy().astype(np.float64)
        r = ref.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(a).all()
        err = np.linalg.norm(a - r) / np.linalg.norm(r)
        assert err <= tol, (c, err)


def test_noalloc_rejects_what_does_not_fit():
    lib = binding.load_library()
    x = torch.zeros(16, 16, 1024, 64, device="cuda", dtype=torch.bfloat16)   # needs ~200 MB of states
    y = torch.empty_like(x)
    rc = lib.monarch_attn_fwd_noalloc(x.data_ptr(), x.data_ptr(), x.data_ptr(), y.data_ptr(),
                                      16, 16, 1024, 64, 32, 2, binding.MA_BF16, None)
    assert rc == 9
    assert "scratch" in binding.status_string(rc)
    assert lib.monarch_attn_fwd_noalloc(None, None, None, None, 1, 1, 16, 4, 4, 1, 0, None) == 1
