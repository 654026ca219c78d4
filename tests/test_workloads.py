"""Input generator and configuration registry (no arithmetic of the method here)."""
import numpy as np
import pytest

from paper_2505_18698_b200 import workloads as wl


def test_registry_matches_the_five_configs():
    w = wl.WORKLOADS
    assert [w[c].BH for c in ("C1", "C2", "C3", "C4", "C5")] == [1, 768, 192, 64, 16]
    assert [(w[c].N, w[c].b, w[c].T, w[c].dtype) for c in ("C1", "C2", "C3", "C4", "C5")] == [
        (256, 16, 1, "f32"), (256, 16, 1, "f16"), (1024, 32, 2, "bf16"),
        (4096, 64, 2, "bf16"), (16384, 128, 2, "bf16")]
    assert all(w[c].tokens == 16384 for c in ("C2", "C3", "C4", "C5"))
    assert w["C5"].algorithmic_bytes() == 134217728
    assert w["C5"].algorithmic_flops() == 38654705664
    assert w["C4"].algorithmic_flops() == 19327352832


def test_extra_workloads_are_the_short_irregular_shapes():
    e = wl.EXTRA_WORKLOADS
    assert not set(e) & set(wl.WORKLOADS)
    assert (e["S1"].N, e["S1"].b, e["S1"].m, e["S1"].T) == (210, 14, 15, 2)      # 197 tokens padded
    assert (e["S2"].N, e["S2"].b, e["S2"].m, e["S2"].T) == (384, 24, 16, 1)
    assert (e["S3"].N, e["S3"].b, e["S3"].m, e["S3"].T) == (8192, 64, 128, 1)
    assert (e["S4"].N, e["S4"].b, e["S4"].m, e["S4"].d) == (7680, 128, 60, 48)
    assert all(w.N == w.m * w.b and w.dtype in ("f16", "bf16") for w in e.values())


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
def test_inputs_are_seeded_and_representable(dtype):
    a = wl.make_qkv(2, 3, 32, 8, dtype, rank=4, s=2.0, seed=5)
    b = wl.make_qkv(2, 3, 32, 8, dtype, rank=4, s=2.0, seed=5)
    c = wl.make_qkv(2, 3, 32, 8, dtype, rank=4, s=2.0, seed=6)
    for x, y, z in zip(a, b, c):
        assert x.dtype == np.float32 and x.shape == (2, 3, 32, 8)
        assert np.array_equal(x, y) and not np.array_equal(x, z)
        assert np.array_equal(wl.round_to_dtype(x, dtype), x)
    if dtype == "bf16":
        assert np.array_equal(wl.from_bf16_bits(wl.to_bf16_bits(a[0])), a[0])


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.0 + 2**-8, 1.0 + 2**-7, 1.0 + 3 * 2**-8, -3.14159], dtype=np.float32)
    r = wl.round_to_dtype(x, "bf16")
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.0 + 2**-7 and r[3] == 1.0 + 2**-6
    assert abs(r[4] + 3.14159) < 2**-7


def test_shared_component_makes_logits_peaky():
    Q, K, _ = wl.make_qkv(1, 2, 512, 64, "bf16", rank=8, s=2.0, seed=1)
    logits = (Q[0, 0] @ K[0, 0].T) / 8.0
    assert 6.0 < logits.std() < 20.0
    Q, K, _ = wl.make_qkv(1, 1, 512, 64, "f32", seed=0)
    assert 0.8 < ((Q[0, 0] @ K[0, 0].T) / 8.0).std() < 1.2


def test_shard_units_partitions_exactly():
    for total in (1, 16, 64, 192, 768, 7):
        for ws in (1, 2, 3, 4, 8):
            spans = [wl.shard_units(total, ws, r) for r in range(ws)]
            assert spans[0][0] == 0 and spans[-1][1] == total
            assert all(spans[i][1] == spans[i + 1][0] for i in range(ws - 1))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1
