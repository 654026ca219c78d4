"""The C-ABI library builds, loads, and exports every symbol the public header declares.
Host-side argument validation is exercised too (it returns before touching the GPU)."""
import ctypes

import pytest

import __graft_entry__ as entry
from paper_2505_18698_b200 import binding


@pytest.fixture(scope="module")
def lib():
    entry.build()
    return binding.load_library()


def test_header_symbols_are_exported(lib):
    names = binding.declared_symbols()
    assert {"monarch_attn_fwd", "monarch_attn_fwd_ex", "monarch_attn_workspace_bytes",
            "monarch_attn_fwd_host", "monarch_attn_device_status",
            "monarch_attn_status_string", "monarch_attn_last_launch_count",
            "monarch_attn_fwd_noalloc", "monarch_attn_set_trace_buffer"} <= set(names)
    for n in names:
        assert getattr(lib, n) is not None


def test_status_strings(lib):
    seen = {binding.status_string(c) for c in range(10)}
    assert len(seen) == 10 and binding.status_string(0) == "ok"
    assert binding.status_string(99) == "unknown status"


def test_workspace_query(lib):
    wb = lib.monarch_attn_workspace_bytes
    assert wb(1, 1, 256, 64, 16, 1, binding.MA_F32, binding.MA_PATH_GENERIC) >= 3 * 256 * 64 * 4
    assert wb(4, 16, 4096, 64, 64, 2, binding.MA_BF16, binding.MA_PATH_AUTO) > 0
    assert wb(1, 1, 256, 64, 15, 1, binding.MA_F32, 0) == 0      # N % b != 0
    assert wb(1, 1, 256, 64, 16, 0, binding.MA_F32, 0) == 0      # T < 1
    assert wb(1, 1, 256, 64, 16, 1, 7, 0) == 0                   # dtype
    assert wb(1, 1, 256, 64, 16, 1, binding.MA_F32, binding.MA_PATH_TENSOR) == 0   # fp32 has no tensor path


def test_host_side_validation_returns_before_any_launch(lib):
    f = lib.monarch_attn_fwd_ex
    p = ctypes.c_void_p
    ok = (p(4096), p(8192), p(12288), p(16384))

    def call(Q=ok[0], K=ok[1], V=ok[2], Y=ok[3], batch=1, heads=1, N=16, d=4, b=4, T=1, dtype=0,
             scale=0.5, path=0, ws=p(1 << 20), wsb=1 << 30):
        return f(Q, K, V, Y, batch, heads, N, d, b, T, dtype, scale, path, ws, wsb, None)

    assert call(Q=None) == 1
    assert call(Y=None) == 1
    assert call(N=18) == 2
    assert call(T=0) == 2
    assert call(batch=0) == 2
    assert call(dtype=5) == 3
    assert call(path=binding.MA_PATH_TENSOR) == 4
    assert call(Q=p(4100)) == 5
    assert call(Y=p(4096 + 16)) == 5        # Y overlaps Q
    assert call(ws=None) == 6
    assert call(wsb=16) == 6
    assert call(ws=p((1 << 20) + 16)) == 5
    assert lib.monarch_attn_fwd(None, None, None, None, 1, 1, 16, 4, 4, 1, 0, None) == 1


def test_binding_refuses_cpu_tensors(lib):
    import torch
    x = torch.zeros(1, 1, 16, 4)
    with pytest.raises(binding.MonarchAttnError):
        binding.monarch_attn_fwd(x, x, x, b=4, T=1)
