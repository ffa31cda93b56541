"""The all-cores restatement of the oracle (oracle/graddrop_oracle_par.cpp) against pins of its own
(pure-Python brute force, exact conservation) and against the numpy oracle, bit for bit."""
import struct

import numpy as np
import pytest

from oracle import graddrop_oracle as orc
from oracle import parallel as par


def f32_bits(x) -> int:
    return struct.unpack("<I", struct.pack("<f", float(x)))[0]


def brute_force_kept(v, k):
    keys = [f32_bits(x) & 0x7FFFFFFF for x in v]
    kept = []
    for i, ki in enumerate(keys):
        ahead = sum(1 for j, kj in enumerate(keys) if kj > ki or (kj == ki and j < i))
        if ahead < k:
            kept.append(i)
    return kept


def same_bits(a, b):
    return np.array_equal(np.asarray(a).view(np.uint32), np.asarray(b).view(np.uint32))


def test_library_builds_and_reports_threads():
    par.build(force=True)
    assert par.threads() >= 1


@pytest.mark.parametrize("seed", range(6))
def test_brute_force_small(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 300))
    # few distinct magnitudes and both zeros, so ties at the cut are the rule
    v = rng.choice(np.array([0.0, -0.0, 0.5, -0.5, 1.0, -2.0, 3.25], dtype=np.float32), size=n)
    r = np.full(n, -0.0, dtype=np.float32)                  # v + (-0) == v bit for bit
    drop_ppm = int(rng.choice([0, 500_000, 900_000, 990_000, 1_000_000]))
    out = par.compress(v, r, [0, n], [0, n], drop_ppm)
    k = n - (n * drop_ppm) // 1_000_000
    kept = brute_force_kept(v, k)
    assert out["idx"].tolist() == kept
    assert same_bits(out["val"], v[kept])
    expect_r = v.copy()
    expect_r[kept] = 0.0
    assert same_bits(out["residual"], expect_r)
    tau = min((f32_bits(v[i]) & 0x7FFFFFFF for i in kept), default=0xFFFFFFFF)
    assert int(out["tau"][0]) == tau
    assert out["shard_cnt_off"].tolist() == [0, k]


def test_conservation_over_steps_integer_gradients():
    # every add is exact on small integers, so nothing may be lost: sum(sent) + residual == sum(g)
    rng = np.random.default_rng(7)
    n, steps = 5000, 6
    layer_off, shard_off = [0, 1200, 1201, n], [0, 2500, n]
    r = np.zeros(n, dtype=np.float32)
    sent = np.zeros(n, dtype=np.float64)
    total = np.zeros(n, dtype=np.float64)
    for _ in range(steps):
        g = rng.integers(-1024, 1025, size=n).astype(np.float32)
        total += g
        out = par.compress(g, r, layer_off, shard_off, 950_000, scope_mode=1)
        sent[out["idx"]] += out["val"]
        r = out["residual"]
        assert out["idx"].shape[0] == sum(orc.kept_count(b - a, 950_000) for a, b in zip(layer_off, layer_off[1:]))
    assert np.array_equal(sent + r, total)


@pytest.mark.parametrize("scope_mode", [0, 1])
@pytest.mark.parametrize("value_mode", [0, 1])
def test_matches_numpy_oracle(scope_mode, value_mode):
    rng = np.random.default_rng(100 + 2 * scope_mode + value_mode)
    sizes = [70_001, 13, 4096, 250_000, 1]
    layer_off = np.concatenate([[0], np.cumsum(sizes)]).tolist()
    n = layer_off[-1]
    shard_off = [0, 100_000, 100_001, 300_000, n]
    g = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    g[rng.random(n) < 0.3] = 0.0
    g[1000:1400] = np.float32(0.25)                          # a tie group across the cut of layer 0
    r = (rng.standard_normal(n) * 1e-4).astype(np.float32)
    a = orc.compress(g, r, layer_off, shard_off, 990_000, scope_mode, value_mode)
    b = par.compress(g, r, layer_off, shard_off, 990_000, scope_mode, value_mode)
    assert np.array_equal(a["idx"], b["idx"])
    assert same_bits(a["val"], b["val"])
    assert same_bits(a["residual"], b["residual"])
    assert np.array_equal(a["tau"], b["tau"])
    assert np.array_equal(a["shard_cnt_off"], b["shard_cnt_off"])
    if value_mode == 1:
        np.testing.assert_allclose(b["means"], a["means"], rtol=1e-6, atol=0)
        # apply: the fp32 result lies within 1e-6 of the fp64 reference, relative to the summed magnitudes
        p0 = (rng.standard_normal(n) * 0.01).astype(np.float32)
        ref, bound = orc.apply_pushes(p0, 0, [a], 0.5, value_mode, layer_off)
        got = par.apply(p0.copy(), b, 0.5, value_mode, layer_off)
        assert np.all(np.abs(got.astype(np.float64) - ref) <= 1e-6 * bound + 1e-30)
    else:
        p0 = (rng.standard_normal(n) * 0.01).astype(np.float32)
        ref, bound = orc.apply_pushes(p0, 0, [a], 0.5)
        got = par.apply(p0.copy(), b, 0.5)
        assert np.all(np.abs(got.astype(np.float64) - ref) <= 1e-6 * bound + 1e-30)


def test_rejects_bad_arguments():
    g = np.zeros(8, dtype=np.float32)
    with pytest.raises(ValueError):
        par.compress(g, g, [0, 8], [0, 8], 1_000_001)
    with pytest.raises(ValueError):
        par.compress(g, g, [0, 8], [0, 8], 990_000, value_mode=3)
