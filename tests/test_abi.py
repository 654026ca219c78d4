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


def test_binding_constants_match_the_header():
    import os
    import re
    here = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    text = open(os.path.join(here, "include", "monarch_attn.h")).read()
    enums = {name: int(val) for name, val in re.findall(r"\b(MA_[A-Z0-9_]+)\s*=\s*(\d+)", text)}
    assert len(enums) >= 20
    for name, val in enums.items():
        if hasattr(binding, name):
            assert getattr(binding, name) == val, name
    for name in ("MA_PATH_AUTO", "MA_PATH_GENERIC", "MA_PATH_TENSOR", "MA_PATH_TENSOR_TMEM", "MA_PATH_FUSED_SMALL",
                 "MA_PATH_TILE_MMA", "MA_F32", "MA_F16", "MA_BF16"):
        assert name in enums and hasattr(binding, name), name
    assert len({v for k, v in enums.items() if k.startswith("MA_PATH_")}) == \
        len([k for k in enums if k.startswith("MA_PATH_")])


def test_workspace_query_of_the_fused_and_tile_paths(lib):
    wb = lib.monarch_attn_workspace_bytes
    F16, BF16 = binding.MA_F16, binding.MA_BF16
    # fused per-head kernel: only a status block; shapes outside its limits are refused
    assert wb(64, 12, 210, 64, 14, 2, F16, binding.MA_PATH_FUSED_SMALL) == 256
    assert wb(1, 1, 480, 64, 24, 2, F16, binding.MA_PATH_FUSED_SMALL) == 0       # 4 tiles do not fit
    assert wb(1, 1, 480, 64, 24, 1, F16, binding.MA_PATH_FUSED_SMALL) == 256
    assert wb(1, 1, 480, 64, 12, 1, F16, binding.MA_PATH_FUSED_SMALL) == 0       # m = 40 > 32
    assert wb(1, 1, 210, 64, 14, 2, binding.MA_F32, binding.MA_PATH_FUSED_SMALL) == 0
    # tile kernels: three f16 states + c_L, two more states from the third round on
    n = 2 * 16 * 8192 * 64
    w2 = wb(2, 16, 8192, 64, 64, 2, BF16, binding.MA_PATH_TILE_MMA)
    w3 = wb(2, 16, 8192, 64, 64, 3, BF16, binding.MA_PATH_TILE_MMA)
    assert 3 * 2 * n <= w2 < 3 * 2 * n + 4 * n // 64 + 4096
    assert w3 - w2 == 2 * 2 * n
    assert wb(1, 1, 8192, 64, 32, 1, F16, binding.MA_PATH_TILE_MMA) == 0         # m = 256 > 128
    assert wb(1, 1, 2048, 136, 32, 1, F16, binding.MA_PATH_TILE_MMA) == 0        # d > 128
    # AUTO: a generic-sized workspace is never smaller than what AUTO needs for 16-bit inputs
    for (N, d, b, T) in [(210, 64, 14, 2), (8192, 64, 64, 1), (7680, 48, 128, 3), (4096, 64, 64, 2)]:
        assert 0 < wb(1, 2, N, d, b, T, F16, binding.MA_PATH_AUTO) <= wb(1, 2, N, d, b, T, F16, binding.MA_PATH_GENERIC)


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


def test_binding_rejects_an_output_tensor_that_does_not_match_the_input():
    """The kernels write Q.numel() elements of Q's dtype through Y's pointer: a smaller, differently
    typed or strided Y must be refused on the host (no GPU needed to check the rule)."""
    import torch
    Q = torch.zeros(2, 3, 16, 8)
    assert binding._out_like(None, Q).shape == Q.shape
    ok = torch.empty_like(Q)
    assert binding._out_like(ok, Q) is ok
    for bad in (torch.zeros(2, 3, 16, 4), torch.zeros(2, 3, 16, 8, dtype=torch.float16),
                torch.zeros(2, 3, 8, 16).transpose(2, 3), "not a tensor"):
        with pytest.raises(ValueError):
            binding._out_like(bad, Q)
