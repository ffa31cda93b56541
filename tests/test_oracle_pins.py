"""Pins for the CPU oracle: every check here is independent of the oracle's own formulas.

Brute-force rank counts in pure Python, closed forms, library selection routines, exact
rational arithmetic, and the payload ratios the paper prints (tests/golden/payload_ratios.txt).
"""
import itertools
import math
import os
import struct
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import graddrop_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def f32_bits(x) -> int:
    return struct.unpack("<I", struct.pack("<f", float(x)))[0]


def brute_force_kept(v, k):
    """O(n^2): entry i is kept iff fewer than k entries precede it in (|v| desc, index asc)."""
    keys = [f32_bits(x) & 0x7FFFFFFF for x in v]
    kept = []
    for i, ki in enumerate(keys):
        ahead = 0
        for j, kj in enumerate(keys):
            if kj > ki or (kj == ki and j < i):
                ahead += 1
        if ahead < k:
            kept.append(i)
    return kept


def run_flat(v, drop_ppm, **kw):
    """GradDrop of v itself: the residual is -0.0 everywhere, the one value with x + r == x bit for bit."""
    g = np.asarray(v, dtype=np.float32)
    r = np.full_like(g, -0.0)
    n = g.shape[0]
    return orc.compress(g, r, [0, n], [0, n], drop_ppm, **kw)


# ---------------------------------------------------------------- kept-count formula
def test_kept_count_values():
    assert orc.kept_count(1 << 20, 990_000) == 10_486
    assert orc.kept_count(1 << 30, 999_000) == 1_073_742
    assert orc.kept_count(10, 990_000) == 1
    assert orc.kept_count(0, 990_000) == 0
    assert orc.kept_count(7, 0) == 7
    assert orc.kept_count(7, 1_000_000) == 0
    # the six tensors of the MNIST-shaped workload at 99 %
    sizes = [784 * 4096, 4096, 4096 * 4096, 4096, 40960, 10]
    assert [orc.kept_count(s, 990_000) for s in sizes] == [32113, 41, 167773, 41, 410, 1]
    assert orc.kept_count(sum(sizes), 990_000) == 200_377
    # equals ceil((1 - R) n) evaluated exactly
    for n in (1, 3, 99, 100, 101, 12345, 1 << 20):
        for ppm in (0, 1, 900_000, 990_000, 999_000, 999_999, 1_000_000):
            assert orc.kept_count(n, ppm) == math.ceil(Fraction(n) * (1 - Fraction(ppm, 1_000_000)))


def test_paper_payload_ratios():
    rec = {}
    with open(os.path.join(GOLDEN, "payload_ratios.txt")) as fh:
        for line in fh:
            if line.strip() and not line.startswith("#"):
                parts = line.split()
                rec[parts[0]] = parts[1]
    ratio99 = float(rec["ratio_dense_over_sparse_at_99pct"])
    min_ratio = float(rec["min_ratio_984_to_99"])
    for n in (100, 1000, 1 << 20, 137_585_000):
        out = run_flat(np.arange(1, n + 1, dtype=np.float32) if n <= 1000 else
                       np.random.default_rng(0).standard_normal(n).astype(np.float32), 990_000,
                       method="select")
        sparse_bytes = out["idx"].nbytes + out["val"].nbytes
        assert out["idx"].dtype == np.uint32 and out["val"].dtype == np.float32
        got = 4 * n / sparse_bytes
        if n % 100 == 0:
            assert got == ratio99
        else:
            assert abs(got - ratio99) / ratio99 < 1e-4
    k984 = orc.kept_count(10**6, 984_000)
    k99 = orc.kept_count(10**6, 990_000)
    assert k984 / k99 > min_ratio and k984 / k99 == pytest.approx(1.6)


# ---------------------------------------------------------------- brute force on tiny vectors
ALPHABET = [0.0, -0.0, 1.0, -1.0, 2.0, -2.0, 1e-45, -3.5]


@pytest.mark.parametrize("n", [1, 2, 3, 4])
def test_exhaustive_tiny_vectors_all_k(n):
    ppms = sorted({(d * 1_000_000) // n for d in range(n + 1)} | {1_000_000, 0, 999_999, 1})
    for v in itertools.product(ALPHABET, repeat=n):
        for ppm in ppms:
            k = n - (n * ppm) // 1_000_000
            want = brute_force_kept(v, k)
            out = run_flat(v, ppm)
            assert out["idx"].tolist() == want, (v, ppm)
            if k:
                assert int(out["tau"][0]) == min(f32_bits(v[i]) & 0x7FFFFFFF for i in want)
            else:
                assert int(out["tau"][0]) == 0xFFFFFFFF


@pytest.mark.parametrize("seed", range(6))
def test_brute_force_random_with_ties(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(5, 400))
    # few distinct magnitudes => many ties at the cut
    v = rng.choice(np.array([0.0, -0.0, 0.5, -0.5, 0.75, 3.0, -3.0, 1e-40], dtype=np.float32), size=n)
    for ppm in (0, 500_000, 900_000, 990_000, 1_000_000):
        for method in ("sort", "select"):
            out = run_flat(v, ppm, method=method)
            assert out["idx"].tolist() == brute_force_kept(v.tolist(), orc.kept_count(n, ppm))


def test_brute_force_per_layer_and_shards():
    rng = np.random.default_rng(11)
    sizes = [10, 0, 37, 1, 128, 5]
    layer_off = np.concatenate([[0], np.cumsum(sizes)]).tolist()
    n = layer_off[-1]
    g = rng.standard_normal(n).astype(np.float32)
    g[rng.integers(0, n, 40)] = 0.25           # ties
    r = (rng.standard_normal(n) * 0.1).astype(np.float32)
    shard_off = [0, 7, 7, 100, n]
    out = orc.compress(g, r, layer_off, shard_off, 900_000, scope_mode=orc.SCOPE_PER_LAYER)
    v = [float(np.float32(a) + np.float32(b)) for a, b in zip(g, r)]
    want = []
    for li, s in enumerate(sizes):
        lo = layer_off[li]
        k = s - (s * 900_000) // 1_000_000
        want += [lo + i for i in brute_force_kept(v[lo:lo + s], k)]
    assert out["idx"].tolist() == want
    assert out["shard_cnt_off"].tolist() == [sum(1 for i in want if i < b) for b in shard_off]
    assert [int(t) for t in out["tau"]][1] == 0xFFFFFFFF        # empty layer keeps nothing


# ---------------------------------------------------------------- invariants
def check_invariants(g, r, layer_off, shard_off, ppm, scope_mode, out):
    v = (g + r).astype(np.float32)
    keys = v.view(np.uint32) & np.uint32(0x7FFFFFFF)
    idx = out["idx"].astype(np.int64) & 0x7FFFFFFF if out["idx"].dtype == np.uint32 and "means" in out \
        else out["idx"].astype(np.int64)
    kept_mask = np.zeros(v.shape[0], dtype=bool)
    kept_mask[idx] = True
    assert np.all(np.diff(idx) > 0)                                   # strictly ascending
    # kept + residual reassemble v bit for bit
    res_bits = out["residual"].view(np.uint32)
    assert np.all(res_bits[kept_mask] == 0)
    assert np.array_equal(res_bits[~kept_mask], v.view(np.uint32)[~kept_mask])
    if "means" not in out:
        assert np.array_equal(out["val"].view(np.uint32), v.view(np.uint32)[idx])
    for si, (lo, hi) in enumerate(orc.scopes_of(layer_off, scope_mode)):
        k = (hi - lo) - ((hi - lo) * ppm) // 1_000_000
        m = kept_mask[lo:hi]
        assert int(m.sum()) == k
        if 0 < k < hi - lo:
            kk, dk = keys[lo:hi][m], keys[lo:hi][~m]
            tau = int(out["tau"][si])
            assert int(kk.min()) == tau and int(dk.max()) <= tau
            ties = np.flatnonzero(keys[lo:hi] == tau)
            kept_ties, dropped_ties = ties[m[ties]], ties[~m[ties]]
            if len(kept_ties) and len(dropped_ties):
                assert kept_ties.max() < dropped_ties.min()
    sc = out["shard_cnt_off"].astype(np.int64)
    assert np.all(np.diff(sc) >= 0) and sc[0] == 0 and sc[-1] == idx.shape[0]


@pytest.mark.parametrize("seed", range(4))
@pytest.mark.parametrize("scope_mode", [orc.SCOPE_GLOBAL, orc.SCOPE_PER_LAYER])
def test_invariants_random(seed, scope_mode):
    rng = np.random.default_rng(100 + seed)
    sizes = rng.integers(0, 5000, size=7).tolist()
    layer_off = np.concatenate([[0], np.cumsum(sizes)]).tolist()
    n = layer_off[-1]
    g = rng.laplace(0, 1e-3, n).astype(np.float32)
    g[rng.random(n) < 0.3] = 0.0
    r = np.where(rng.random(n) < 0.5, rng.laplace(0, 1e-3, n), 0).astype(np.float32)
    shard_off = [0, n // 3, n // 2, n]
    for ppm in (0, 900_000, 990_000, 999_000, 1_000_000):
        out = orc.compress(g, r, layer_off, shard_off, ppm, scope_mode=scope_mode)
        check_invariants(g, r, layer_off, shard_off, ppm, scope_mode, out)


# ---------------------------------------------------------------- closed forms
def test_closed_form_distinct_magnitudes():
    n = 1000
    rng = np.random.default_rng(5)
    m = rng.permutation(n) + 1                               # magnitudes m / 1024, all distinct
    sign = rng.choice([-1.0, 1.0], n)
    v = (sign * m / 1024.0).astype(np.float32)
    for ppm in (500_000, 900_000, 990_000, 999_000):
        k = orc.kept_count(n, ppm)
        out = run_flat(v, ppm)
        assert sorted(m[out["idx"]].tolist()) == list(range(n - k + 1, n + 1))
        assert int(out["tau"][0]) == f32_bits((n - k + 1) / 1024.0)


def test_closed_form_degenerate_inputs():
    n = 257
    for c in (0.0, -0.0, 3.25, -3.25):
        for ppm in (900_000, 990_000):
            k = orc.kept_count(n, ppm)
            out = run_flat(np.full(n, c, dtype=np.float32), ppm)
            assert out["idx"].tolist() == list(range(k))         # ties go to the lowest indices
            assert int(out["tau"][0]) == f32_bits(c) & 0x7FFFFFFF
            assert np.array_equal(out["val"].view(np.uint32), np.full(k, f32_bits(c), dtype=np.uint32))
    v = np.random.default_rng(1).standard_normal(n).astype(np.float32)
    out = run_flat(v, 0)                                         # R = 0: everything travels
    assert out["idx"].tolist() == list(range(n)) and not out["residual"].any()
    assert np.all(out["residual"].view(np.uint32) == 0)
    out = run_flat(v, 1_000_000)                                 # R = 100 %: nothing travels
    assert out["idx"].size == 0 and np.array_equal(out["residual"], v)
    # k = 1 is the lowest-index arg-max of |v|
    v[[17, 200]] = [-9.0, 9.0]
    out = run_flat(v, orc_ppm_for_k1(n))
    assert out["idx"].tolist() == [17] and out["val"].tolist() == [-9.0]


def orc_ppm_for_k1(n):
    ppm = ((n - 1) * 1_000_000 + n - 1) // n
    assert orc.kept_count(n, ppm) == 1
    return ppm


def test_signed_zero_and_subnormals_are_preserved():
    v = np.array([-0.0, 1e-45, -1e-45, 0.0, 5.0, -1e-39], dtype=np.float32)
    out = run_flat(v, 500_000)                                   # keeps 3: 5.0, -1e-39, then 1e-45 (idx 1)
    assert out["idx"].tolist() == [1, 4, 5]
    assert [f32_bits(x) for x in out["val"]] == [f32_bits(1e-45), f32_bits(5.0), f32_bits(-1e-39)]
    assert [f32_bits(x) for x in out["residual"]] == [0x80000000, 0, f32_bits(-1e-45), 0, 0, 0]


# ---------------------------------------------------------------- library selection routines
@pytest.mark.parametrize("seed", range(3))
def test_threshold_equals_library_selection(seed):
    rng = np.random.default_rng(200 + seed)
    n = 50_000 + seed * 777
    g = rng.laplace(0, 1e-3, n).astype(np.float32)
    r = rng.laplace(0, 1e-4, n).astype(np.float32)
    for ppm in (900_000, 990_000, 999_000):
        k = orc.kept_count(n, ppm)
        out = orc.compress(g, r, [0, n], [0, n], ppm)
        a = np.abs(g + r)
        tau_f = np.partition(a, n - k)[n - k]
        assert np.uint32(out["tau"][0]).view(np.float32) == tau_f
        tv = torch.kthvalue(torch.from_numpy(a), n - k + 1).values.item()
        assert np.uint32(out["tau"][0]).view(np.float32) == np.float32(tv)
        if np.unique(a).size == n:                                # tie-free: top-k set is unique
            top = torch.topk(torch.from_numpy(a), k).indices.numpy()
            assert np.array_equal(np.sort(top), out["idx"].astype(np.int64))
        mask = np.zeros(n, dtype=bool)
        mask[out["idx"]] = True
        assert np.array_equal(np.flatnonzero(mask), out["idx"].astype(np.int64))


def test_select_method_equals_sort_method():
    rng = np.random.default_rng(9)
    n = 1 << 20
    g = rng.laplace(0, 1e-3, n).astype(np.float32)
    g[rng.random(n) < 0.6] = 0.0
    r = np.zeros(n, dtype=np.float32)
    layer_off = [0, 1000, 1000, 300_000, n]
    for scope_mode in (orc.SCOPE_GLOBAL, orc.SCOPE_PER_LAYER):
        for ppm in (300_000, 990_000):                            # 30 % drop cuts inside the zero ties
            a = orc.compress(g, r, layer_off, [0, n], ppm, scope_mode=scope_mode, method="sort")
            b = orc.compress(g, r, layer_off, [0, n], ppm, scope_mode=scope_mode, method="select")
            for key in ("idx", "val", "residual", "tau", "shard_cnt_off"):
                assert np.array_equal(a[key].view(np.uint32), b[key].view(np.uint32))


# ---------------------------------------------------------------- error feedback over steps
def test_nothing_is_lost_over_steps():
    """Integer-valued gradients make every fp32 add exact: sent mass + residual == sum of gradients."""
    rng = np.random.default_rng(3)
    n, steps = 4096, 12
    layer_off, shard_off = [0, 100, n], [0, n // 2, n]
    r = orc.residual_reset(n)
    sent = np.zeros(n, dtype=np.int64)
    total = np.zeros(n, dtype=np.int64)
    for _ in range(steps):
        g = rng.integers(-1024, 1025, n).astype(np.float32)
        total += g.astype(np.int64)
        out = orc.compress(g, r, layer_off, shard_off, 990_000, scope_mode=orc.SCOPE_PER_LAYER)
        sent[out["idx"]] += out["val"].astype(np.int64)
        r = out["residual"]
    assert np.array_equal(sent + r.astype(np.int64), total)
    assert np.abs(r).max() > 1024                                 # residuals really accumulated


# ---------------------------------------------------------------- two-value quantisation
def test_two_means_closed_form_and_independent_sum():
    rng = np.random.default_rng(21)
    layer_off = [0, 300, 300, 1000]
    n = layer_off[-1]
    g = (rng.standard_normal(n) * 1e-3).astype(np.float32)
    big = rng.choice(n, 64, replace=False)
    g[big] = np.where(rng.random(64) < 0.5, 2.5, -1.5).astype(np.float32)   # kept values are exactly +2.5 / -1.5
    r = np.zeros(n, dtype=np.float32)
    out = orc.compress(g, r, layer_off, [0, 500, n], 950_000, scope_mode=orc.SCOPE_GLOBAL,
                       value_mode=orc.VALUES_TWO_MEANS)
    k = orc.kept_count(n, 950_000)
    assert k == 50
    pos = (out["idx"] & np.uint32(0x7FFFFFFF)).astype(np.int64)
    sign = out["idx"] >> np.uint32(31)
    assert set(pos.tolist()) <= set(big.tolist())
    assert np.array_equal(sign, (g[pos] < 0).astype(np.uint32))
    for li in (0, 2):
        in_l = (pos >= layer_off[li]) & (pos < layer_off[li + 1])
        for sg, c in ((0, 2.5), (1, -1.5)):
            cnt = int(np.sum(in_l & (sign == sg)))
            assert out["counts"][li, sg] == cnt
            assert out["means"][li, sg] == (np.float32(c) if cnt else np.float32(0.0))
    assert out["counts"][1].tolist() == [0, 0] and out["means"][1].tolist() == [0.0, 0.0]
    assert out["counts"].sum() == k
    # residual holds the dropped mass only (the quantisation error is not fed back)
    plain = orc.compress(g, r, layer_off, [0, 500, n], 950_000)
    assert np.array_equal(plain["residual"].view(np.uint32), out["residual"].view(np.uint32))
    assert np.array_equal(plain["idx"], pos.astype(np.uint32))

    # general values: means against exactly rounded sums (math.fsum), independent of numpy's add
    g2 = rng.laplace(0, 1e-3, n).astype(np.float32)
    out2 = orc.compress(g2, r, layer_off, [0, n], 900_000, scope_mode=orc.SCOPE_PER_LAYER,
                        value_mode=orc.VALUES_TWO_MEANS)
    pos2 = (out2["idx"] & np.uint32(0x7FFFFFFF)).astype(np.int64)
    for li in range(3):
        for sg in (0, 1):
            sel = [float(g2[p]) for p in pos2 if layer_off[li] <= p < layer_off[li + 1]
                   and (f32_bits(g2[p]) >> 31) == sg]
            want = np.float32(math.fsum(sel) / len(sel)) if sel else np.float32(0)
            assert abs(float(out2["means"][li, sg]) - float(want)) <= 1e-6 * abs(float(want))


# ---------------------------------------------------------------- server-side apply
def test_apply_against_exact_rationals():
    rng = np.random.default_rng(8)
    n, shard_start, shard_len = 600, 150, 300
    p0 = (rng.standard_normal(shard_len) * 0.01).astype(np.float32)
    pushes = []
    for w in range(3):
        g = rng.laplace(0, 1e-3, n).astype(np.float32)
        out = orc.compress(g, np.zeros(n, np.float32), [0, n], [0, n], 900_000)
        pushes.append({"idx": out["idx"], "val": out["val"]})
    alpha = 0.5
    ref, bound = orc.apply_pushes(p0, shard_start, pushes, alpha=alpha)
    exact = [Fraction(float(x)) for x in p0]
    mag = [abs(Fraction(float(x))) for x in p0]
    for push in pushes:
        for i, x in zip(push["idx"].tolist(), push["val"].tolist()):
            if shard_start <= i < shard_start + shard_len:
                exact[i - shard_start] += Fraction(alpha) * Fraction(x)
                mag[i - shard_start] += abs(Fraction(alpha) * Fraction(x))
    for j in range(shard_len):
        assert abs(Fraction(float(ref[j])) - exact[j]) <= Fraction(1, 10**14) * max(mag[j], Fraction(1, 10**30))
        assert abs(Fraction(float(bound[j])) - mag[j]) <= Fraction(1, 10**14) * max(mag[j], Fraction(1, 10**30))


def test_apply_two_means_decode():
    layer_off = [0, 4, 10]
    means = np.array([[0.5, -0.25], [2.0, -3.0]], dtype=np.float32)
    idx = np.array([1, 3 | (1 << 31), 4 | (1 << 31), 9], dtype=np.uint32)
    pos, val = orc.decode_push(idx, None, orc.VALUES_TWO_MEANS, means, layer_off)
    assert pos.tolist() == [1, 3, 4, 9] and val.tolist() == [0.5, -0.25, -3.0, 2.0]
    ref, _ = orc.apply_pushes(np.ones(6, np.float32), 4, [{"idx": idx, "means": means}],
                              value_mode=orc.VALUES_TWO_MEANS, layer_off=layer_off)
    assert ref.tolist() == [-2.0, 1.0, 1.0, 1.0, 1.0, 3.0]


# ---------------------------------------------------------------- threshold quantisation
def test_threshold_quantisation_values():
    """Every survivor stands for +-(the smallest kept magnitude of its scope), written out by hand."""
    layer_off = [0, 4, 10]
    g = np.array([0.5, -3.0, 0.25, 2.0,   -0.125, 7.0, -6.0, 0.0625, 5.0, -0.03125], dtype=np.float32)
    r = np.full(10, -0.0, dtype=np.float32)
    out = orc.compress(g, r, layer_off, [0, 10], 500_000, scope_mode=orc.SCOPE_PER_LAYER,
                       value_mode=orc.VALUES_THRESHOLD)
    # layer 0 keeps 2 of 4: -3.0, 2.0 -> t = 2.0 ; layer 1 keeps 3 of 6: 7.0, -6.0, 5.0 -> t = 5.0
    assert (out["idx"] & np.uint32(0x7FFFFFFF)).tolist() == [1, 3, 5, 6, 8]
    assert (out["idx"] >> np.uint32(31)).tolist() == [1, 0, 0, 1, 0]
    assert out["means"].tolist() == [[2.0, -2.0], [5.0, -5.0]]
    pos, val = orc.decode_push(out["idx"], None, orc.VALUES_THRESHOLD, out["means"], layer_off)
    assert val.tolist() == [-2.0, 2.0, 5.0, -5.0, 5.0]
    assert np.all(np.abs(val) <= np.abs(g[pos]))          # never larger than the value it stands for
    glob = orc.compress(g, r, layer_off, [0, 10], 500_000, scope_mode=orc.SCOPE_GLOBAL,
                        value_mode=orc.VALUES_THRESHOLD)
    assert glob["means"].tolist() == [[2.0, -2.0], [2.0, -2.0]]     # one global threshold: 7, -6, 5, -3, 2 kept
    none = orc.compress(g, r, layer_off, [0, 10], 1_000_000, value_mode=orc.VALUES_THRESHOLD)
    assert none["idx"].size == 0 and np.all(none["means"].view(np.uint32) == [[0, 0x80000000]] * 2)


# ---------------------------------------------------------------- parameter pulls as dropped deltas
def test_quantisation_error_feedback_by_hand_and_conservation():
    # kept: 4, -3, 2 (k = 3 of 10): mu+ = 3, mu- = -3; each kept slot keeps v - decoded, dropped slots keep v
    v = np.array([4.0, 0.5, -3.0, 0.25, 2.0, -0.5, 1.0, -1.0, 0.0, 0.125], dtype=np.float32)
    base = run_flat(v, 700_000, value_mode=orc.VALUES_TWO_MEANS)
    out = run_flat(v, 700_000, value_mode=orc.VALUES_TWO_MEANS, error_feedback=True)
    assert out["idx"].tolist() == base["idx"].tolist() == [0, 2 | (1 << 31), 4]
    assert out["means"].tolist() == [[3.0, -3.0]]
    assert out["residual"].tolist() == [1.0, 0.5, 0.0, 0.25, -1.0, -0.5, 1.0, -1.0, 0.0, 0.125]
    # without the option the same slots hold +0 (Algorithm 1 as printed)
    assert base["residual"].tolist() == [0.0, 0.5, 0.0, 0.25, 0.0, -0.5, 1.0, -1.0, 0.0, 0.125]
    # threshold quantiser: decoded = +-2, so 4 -> 2, -3 -> -1, and the entry at the threshold leaves +0
    thr = run_flat(v, 700_000, value_mode=orc.VALUES_THRESHOLD, error_feedback=True)
    assert thr["residual"].tolist() == [2.0, 0.5, -1.0, 0.25, 0.0, -0.5, 1.0, -1.0, 0.0, 0.125]
    # conservation: what the receiver decodes plus what stays is v (exact here: small dyadic numbers), per
    # layer and per column, over several steps with the residual carried
    rng = np.random.default_rng(11)
    layer_off, cols = [0, 64, 64 + 96], [8, 1]
    n = layer_off[-1]
    for mode in (orc.VALUES_TWO_MEANS, orc.VALUES_THRESHOLD, orc.VALUES_COLUMN_MEANS):
        r = np.zeros(n, dtype=np.float32)
        total = np.zeros(n, dtype=np.float64)
        received = np.zeros(n, dtype=np.float64)
        for _ in range(4):
            g = (rng.integers(-64, 65, size=n) * 0.25).astype(np.float32)
            total += g
            o = orc.compress(g, r, layer_off, [0, n], 750_000, orc.SCOPE_PER_LAYER, mode, layer_cols=cols,
                             error_feedback=True)
            pos, dec = orc.decode_push(o["idx"], None, mode, o["means"], layer_off, cols)
            # dyadic inputs, but a mean of them need not be: compare against the fp32 subtraction by hand
            manual = o["v"].copy()
            manual[pos] = o["v"][pos] - dec
            assert np.array_equal(manual.view(np.uint32), o["residual"].view(np.uint32))
            received[pos] += dec
            r = o["residual"]
            assert np.allclose(received + r, total, rtol=0, atol=1e-4)
    with pytest.raises(ValueError):
        run_flat(v, 700_000, error_feedback=True)


def test_delta_pull_by_hand_and_invariants():
    # by hand: delta = p - last = [0.5, -4, 0.25, 3, 0, -1]; keep 2 of 6 (drop 2/3): -4 and 3
    p = np.array([1.5, -3.0, 0.25, 5.0, 2.0, 0.0], dtype=np.float32)
    last = np.array([1.0, 1.0, 0.0, 2.0, 2.0, 1.0], dtype=np.float32)
    out = orc.compress_delta(p, last, [0, 6], [0, 3, 6], 666_667)
    assert out["idx"].tolist() == [1, 3] and out["val"].tolist() == [-4.0, 3.0]
    assert out["last_pulled"].tolist() == [1.0, -3.0, 0.0, 5.0, 2.0, 1.0]
    assert out["residual"].tolist() == [0.5, 0.0, 0.25, 0.0, 0.0, -1.0]
    assert out["shard_cnt_off"].tolist() == [0, 1, 2]

    rng = np.random.default_rng(31)
    n = 3000
    layer_off, shard_off = [0, 1000, n], [0, n]
    p = rng.integers(-500, 500, n).astype(np.float32)              # integer-valued: every fp32 op is exact
    last = np.zeros(n, dtype=np.float32)
    client = np.zeros(n, dtype=np.float32)
    for step in range(6):
        p = p + rng.integers(-50, 51, n).astype(np.float32)
        out = orc.compress_delta(p, last, layer_off, shard_off, 900_000, scope_mode=orc.SCOPE_PER_LAYER)
        v = [float(a) - float(b) for a, b in zip(p, last)]
        want = []
        for lo, hi in ((0, 1000), (1000, n)):
            want += [lo + i for i in brute_force_kept(v[lo:hi], orc.kept_count(hi - lo, 900_000))]
        assert out["idx"].tolist() == want
        client[out["idx"]] = client[out["idx"]] + out["val"]       # what the client does with the pull
        last = out["last_pulled"]
        assert np.array_equal(client.view(np.uint32), last.view(np.uint32))      # server's record == client's copy
        assert np.array_equal(p - last, out["residual"])           # nothing lost: the rest is the next delta
    out = orc.compress_delta(p, last, layer_off, shard_off, 0)     # R = 0: the client catches up completely
    assert np.array_equal(out["last_pulled"], p)


# ---------------------------------------------------------------- sampled threshold (Section 4)
def _mix32_py(x):
    x &= 0xFFFFFFFF
    x ^= x >> 16
    x = (x * 0x7FEB352D) & 0xFFFFFFFF
    x ^= x >> 15
    x = (x * 0x846CA68B) & 0xFFFFFFFF
    x ^= x >> 16
    return x


def test_sampled_positions_are_one_pair_per_stratum():
    for lo, hi, si in ((0, 10, 0), (5, 4101, 3), (100, 100 + 4097, 1), (101, 101 + 4097, 1), (0, 5_000_000, 7),
                       (17, 17 + 123_457, 2), (0, 4_097_001, 4)):
        ns = hi - lo
        pos = orc.sampled_positions(lo, hi, si)
        if ns <= 4096:
            assert pos.tolist() == list(range(lo, hi))           # small scopes: everything
            continue
        m = max(4096, -(-ns // 1000))
        m += m % 2
        assert pos.shape[0] == m
        first = lo + lo % 2
        pairs, strata = (hi - first) // 2, m // 2
        w_, rem = pairs // strata, pairs % strata
        starts = [0]
        for i in range(strata):                                 # strata of pairs laid end to end: rem wide ones first
            starts.append(starts[-1] + w_ + (1 if i < rem else 0))
        assert starts[-1] == pairs
        for i in (0, 1, strata // 2, strata - 1):               # pure-Python restatement on a few strata
            width = starts[i + 1] - starts[i]
            pair = starts[i] + (_mix32_py(i * 0x9E3779B9 + si) % width if width > 1 else 0)
            assert int(pos[2 * i]) == first + 2 * pair and int(pos[2 * i + 1]) == first + 2 * pair + 1
        assert np.all(pos[0::2] % 2 == 0)                       # both reads of a pair share an aligned 8 bytes
        assert np.all(np.diff(pos) > 0) and pos[0] >= lo and pos[-1] < hi      # distinct, ordered, in range
    assert orc.sampled_positions(3, 3 + 4096, 0).tolist() == list(range(3, 3 + 4096))


def test_sampled_positions_equal_the_stored_literals():
    """The position rule is frozen: tests/golden/sampled_positions.txt holds literal positions (sample size,
    first / middle / last eight) for five scopes, and the oracle must still produce exactly those."""
    seen = 0
    for line in open(os.path.join(GOLDEN, "sampled_positions.txt")):
        if line.startswith("#") or not line.strip():
            continue
        head, first, middle, last = [part.split() for part in line.split("|")]
        lo, hi, scope, m = (int(x) for x in head)
        pos = orc.sampled_positions(lo, hi, scope)
        assert pos.shape[0] == m
        mid = m // 2 - 4
        assert pos[:8].tolist() == [int(x) for x in first]
        assert pos[mid:mid + 8].tolist() == [int(x) for x in middle]
        assert pos[-8:].tolist() == [int(x) for x in last]
        seen += 1
    assert seen == 5


def test_sampled_positions_worked_by_hand():
    """8200 elements from index 1, scope 0: m = 4096 samples = 2048 pairs out of the 4099 pairs that start at
    even indices 2, 4, ..., 8198; 4099 = 2 * 2048 + 3, so strata 0..2 hold three pairs and the others two.
    The mix of 0 is 0 (every step of it maps 0 to 0), so stratum 0 of scope 0 contributes its first pair,
    (2, 3).  Stratum 2047, the last, holds the pairs starting at 8196 and 8198."""
    pos = orc.sampled_positions(1, 8201, 0)
    assert pos.shape[0] == 4096
    assert pos[:2].tolist() == [2, 3]
    assert pos[-2:].tolist() in ([8196, 8197], [8198, 8199])
    # stratum i >= 3 starts at pair 2 i + 3: its sample is one of two pairs
    for i in (3, 100, 2046):
        assert int(pos[2 * i]) in (2 + 2 * (2 * i + 3), 2 + 2 * (2 * i + 4))
    # every pair position is even and the index 1 (before the first even index) is never read
    assert int(pos.min()) == 2 and int(pos.max()) <= 8199


@pytest.mark.parametrize("config", [1, 2, 3, 5])
def test_sampled_threshold_kept_count_error_on_the_workloads(config):
    """Section 4 presents the sampled threshold as an approximation; this checks it as one, without the position
    formula: on the workloads' own shapes the number kept per scope stays within the sampling error of the exact
    count k.  A threshold from k_m tail samples has a relative error of about 1 / sqrt(k_m) in rank; samples are
    taken in pairs of neighbours, which in the worst case (neighbours always equal) halves the effective
    sample, so the band is 5 sqrt(2 / k_m).  Scopes sampled completely keep at least k (k plus ties)."""
    from paper_1704_05021_b200 import workloads as W
    if config == 5:
        w = W.workload(5, scale_log2=24)                     # the flat stress shape, cut to what the CPU suite can afford
    elif config == 2:
        w = W.workload(2, scope_mode=orc.SCOPE_PER_LAYER)    # six scopes from 10 to 16.8 M elements
    else:
        w = W.workload(config)
    g = W.make_gradient(w, 0, "cpu").numpy()
    r = np.zeros(w.n, np.float32)
    out = orc.compress_sampled(g, r, w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode)
    idx = out["idx"].astype(np.int64)
    for lo, hi in orc.scopes_of(w.layer_off, w.scope_mode):
        ns = hi - lo
        k = orc.kept_count(ns, w.drop_ppm)
        kept = int(np.searchsorted(idx, hi) - np.searchsorted(idx, lo))
        m = orc.sampled_positions(lo, hi, 0).shape[0]
        k_m = orc.kept_count(m, w.drop_ppm)
        if ns <= 4096:
            assert kept >= k
            continue
        band = 5.0 * math.sqrt(2.0 / k_m)
        assert abs(kept / k - 1.0) <= band, (config, lo, hi, kept, k, band)


def test_sampled_threshold_small_scope_is_exact_selection_with_all_ties():
    rng = np.random.default_rng(41)
    n = 3000                                                   # <= 4096: the sample is the whole scope
    g = rng.choice(np.array([0.0, 0.5, -0.5, 1.0, -2.0, 3.0], np.float32), n)
    r = np.full(n, -0.0, np.float32)
    for ppm in (500_000, 900_000, 990_000, 1_000_000, 0):
        out = orc.compress_sampled(g, r, [0, n], [0, n // 2, n], ppm)
        exact = orc.compress(g, r, [0, n], [0, n // 2, n], ppm)
        assert int(out["tau"][0]) == int(exact["tau"][0])
        if ppm == 1_000_000:
            assert out["idx"].size == 0
            continue
        keys = g.view(np.uint32) & np.uint32(0x7FFFFFFF)
        want = np.flatnonzero(keys >= out["tau"][0])           # the exact set plus every tie at tau
        assert np.array_equal(out["idx"].astype(np.int64), want)
        assert set(exact["idx"].tolist()) <= set(out["idx"].tolist())
        assert out["shard_cnt_off"].tolist() == [0, int((want < n // 2).sum()), want.size]


def test_sampled_threshold_keeps_about_the_requested_fraction():
    rng = np.random.default_rng(43)
    n = 4_000_000
    g = rng.laplace(0, 1e-3, n).astype(np.float32)
    r = np.zeros(n, np.float32)
    out = orc.compress_sampled(g, r, [0, n], [0, n], 990_000)
    m = 4096                                                   # ceil(n / 1000) = 4000 < 4096 (and already even)
    pos = orc.sampled_positions(0, n, 0)
    assert pos.shape[0] == m
    k_m = m - (m * 990_000) // 1_000_000
    t = sorted((f32_bits(x) & 0x7FFFFFFF for x in g[pos]), reverse=True)[k_m - 1]
    assert int(out["tau"][0]) == t
    frac = out["idx"].size / n
    assert abs(frac - 0.01) < 6 * 0.01 / math.sqrt(k_m)        # sampling error of a quantile from k_m tail samples
    assert np.array_equal(out["val"], g[out["idx"]])
    assert not out["residual"][out["idx"]].any()


# ---------------------------------------------------------------- column-wise averages (Section 5.4)
def test_column_means_by_hand_and_against_two_means():
    # one 3 x 4 matrix (row-major) followed by a vector of 4; keep 6 of 12 and 2 of 4
    m = np.array([[4.0, -1.0, 0.5, 6.0],
                  [-5.0, 0.25, 3.0, -0.125],
                  [7.0, -8.0, 0.0625, -9.0]], dtype=np.float32)
    vec = np.array([0.5, -2.0, 3.0, 0.25], dtype=np.float32)
    g = np.concatenate([m.ravel(), vec])
    r = np.full(g.shape[0], -0.0, np.float32)
    layer_off, cols = [0, 12, 16], [4, 1]
    out = orc.compress(g, r, layer_off, [0, 16], 500_000, scope_mode=orc.SCOPE_PER_LAYER,
                       value_mode=orc.VALUES_COLUMN_MEANS, layer_cols=cols)
    # matrix keeps |.| in {9, 8, 7, 6, 5, 4}: col 0: 4, -5, 7 ; col 1: -8 ; col 2: none ; col 3: 6, -9.  vector keeps 3, -2
    assert (out["idx"] & np.uint32(0x7FFFFFFF)).tolist() == [0, 3, 4, 8, 9, 11, 13, 14]
    want = [[5.5, -5.0], [0.0, -8.0], [0.0, 0.0], [6.0, -9.0], [3.0, -2.0]]
    assert out["means"].tolist() == want
    assert out["counts"].tolist() == [[2, 1], [0, 1], [0, 0], [1, 1], [1, 1]]
    pos, val = orc.decode_push(out["idx"], None, orc.VALUES_COLUMN_MEANS, out["means"], layer_off, cols)
    assert val.tolist() == [5.5, 6.0, -5.0, 5.5, -8.0, -9.0, -2.0, 3.0]
    # with one column per layer the pairs are the two-means pairs
    rng = np.random.default_rng(77)
    g2 = rng.laplace(0, 1e-3, 16).astype(np.float32)
    a = orc.compress(g2, r, layer_off, [0, 16], 500_000, value_mode=orc.VALUES_COLUMN_MEANS, layer_cols=[1, 1])
    b = orc.compress(g2, r, layer_off, [0, 16], 500_000, value_mode=orc.VALUES_TWO_MEANS)
    assert np.array_equal(a["means"], b["means"]) and np.array_equal(a["idx"], b["idx"])
    # a column mean never leaves the range of the values it stands for
    big = rng.standard_normal(40 * 25).astype(np.float32)
    o = orc.compress(big, np.full(1000, -0.0, np.float32), [0, 1000], [0, 1000], 800_000,
                     value_mode=orc.VALUES_COLUMN_MEANS, layer_cols=[25])
    pos, val = orc.decode_push(o["idx"], None, orc.VALUES_COLUMN_MEANS, o["means"], [0, 1000], [25])
    for c in range(25):
        for sg, sel in ((0, big[pos] >= 0), (1, big[pos] < 0)):
            mine = big[pos][(pos % 25 == c) & sel]
            if mine.size:
                assert mine.min() - 1e-6 <= o["means"][c, sg] <= mine.max() + 1e-6
                assert abs(float(o["means"][c, sg]) - math.fsum(float(x) for x in mine) / mine.size) <= 1e-6 * abs(float(o["means"][c, sg]))
