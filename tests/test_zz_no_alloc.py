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


def _problem(batch, heads, N, d, b, dtype, seed):
    Q, K, V = wl.make_qkv(batch, heads, N, d, dtype, 4, 1.0, seed)
    return tuple(binding.to_device(x, dtype) for x in (Q, K, V))


def test_noalloc_leaves_device_memory_as_it_found_it():
    """The property the entry point exists for: after the first call (module load, the symbol
    lookup) further calls change nothing in the device's free memory."""
    Qd, Kd, Vd = _problem(2, 3, 256, 64, 16, "f16", 5)
    Y = torch.empty_like(Qd)
    binding.monarch_attn_fwd_noalloc(Qd, Kd, Vd, 16, 2, Y)
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    for _ in range(5):
        binding.monarch_attn_fwd_noalloc(Qd, Kd, Vd, 16, 2, Y)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0


def test_noalloc_two_problems_on_one_side_stream_without_a_host_sync():
    """Stream order alone separates two calls that share the scratch."""
    p1 = _problem(2, 3, 256, 64, 16, "f32", 6)
    p2 = _problem(1, 4, 384, 64, 24, "f32", 7)
    y1, y2 = torch.empty_like(p1[0]), torch.empty_like(p2[0])
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        binding.monarch_attn_fwd_noalloc(*p1, 16, 2, y1, stream=side)
        binding.monarch_attn_fwd_noalloc(*p2, 24, 3, y2, stream=side)
    side.synchronize()
    r1 = binding.monarch_attn_fwd_ex(*p1, 16, 2, path=binding.MA_PATH_GENERIC)
    r2 = binding.monarch_attn_fwd_ex(*p2, 24, 3, path=binding.MA_PATH_GENERIC)
    torch.cuda.synchronize()
    assert torch.equal(y1, r1) and torch.equal(y2, r2)


def test_noalloc_limit_at_both_edges():
    """N = 256, d = 64: a unit needs 3 * 65536 + 2 * 1024 bytes of states, the scratch is 8 MiB with a
    256-byte status block: 42 units fit, 43 do not (and then nothing is enqueued)."""
    lib = binding.load_library()
    per_unit, limit = 3 * 4 * 256 * 64 + 2 * 4 * 256, 8 << 20
    assert 256 + 42 * per_unit <= limit < 256 + 43 * per_unit
    Qd, Kd, Vd = _problem(1, 42, 256, 64, 16, "f32", 8)
    Y = torch.empty_like(Qd)
    binding.monarch_attn_fwd_noalloc(Qd, Kd, Vd, 16, 1, Y)
    ref = binding.monarch_attn_fwd_ex(Qd, Kd, Vd, 16, 1, path=binding.MA_PATH_GENERIC)
    torch.cuda.synchronize()
    assert torch.equal(Y, ref)
    x = torch.zeros(1, 43, 256, 64, device="cuda")
    y = torch.full_like(x, 7.0)
    rc = lib.monarch_attn_fwd_noalloc(x.data_ptr(), x.data_ptr(), x.data_ptr(), y.data_ptr(),
                                      1, 43, 256, 64, 16, 1, binding.MA_F32, None)
    torch.cuda.synchronize()
    assert rc == 9 and bool((y == 7.0).all())
