"""Parity of the CUDA library (through its C ABI) with the CPU oracle, element by element.

Bit-exact: thresholds, survivor indices, survivor values, residuals, shard offsets.
Within 1e-6 relative: the two means (fp64 reference sums) and the scatter-added parameters.
"""
import gc
import numpy as np
import pytest
import torch

from oracle import graddrop_oracle as orc
from paper_1704_05021_b200 import binding as B
from paper_1704_05021_b200 import workloads as W
from paper_1704_05021_b200.session import GradDropSession

pytestmark = pytest.mark.gpu

REL_TOL = 1e-6   # stated tolerance for means and applied parameters


def _np_u32(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().numpy().view(np.uint32)


def compare_step(sess: GradDropSession, exp: dict, tag: str):
    assert sess.status() == B.GD_OK, f"{tag}: device status {sess.status()}"
    k = sess.k_total
    assert exp["idx"].shape[0] == k
    got_tau = _np_u32(sess.out_tau)
    assert np.array_equal(got_tau, exp["tau"]), f"{tag}: tau {got_tau[:8]} vs {exp['tau'][:8]}"
    got_idx = _np_u32(sess.out_idx)[:k]
    if not np.array_equal(got_idx, exp["idx"]):
        bad = np.flatnonzero(got_idx != exp["idx"])
        raise AssertionError(f"{tag}: idx differs at {bad[:5]} ({bad.size} of {k}): got {got_idx[bad[:5]]} "
                             f"want {exp['idx'][bad[:5]]}")
    if sess.value_mode == B.GD_VALUES_FP32:
        got_val = _np_u32(sess.out_val)[:k]
        assert np.array_equal(got_val, exp["val"].view(np.uint32)), f"{tag}: val bits differ"
    elif sess.value_mode == B.GD_VALUES_THRESHOLD:
        assert np.array_equal(_np_u32(sess.out_means), exp["means"].view(np.uint32)), f"{tag}: +-tau pairs differ"
    else:
        got_means = sess.out_means.cpu().numpy().astype(np.float64)
        ref = np.where(exp["counts"] > 0, exp["sums"] / np.maximum(exp["counts"], 1), 0.0)
        assert np.all(np.abs(got_means - ref) <= REL_TOL * np.abs(ref)), f"{tag}: means {got_means} vs {ref}"
    got_res = _np_u32(sess.residual)
    if not np.array_equal(got_res, exp["residual"].view(np.uint32)):
        bad = np.flatnonzero(got_res != exp["residual"].view(np.uint32))
        raise AssertionError(f"{tag}: residual differs at {bad[:5]} ({bad.size} places)")
    assert np.array_equal(_np_u32(sess.out_shard_cnt_off), exp["shard_cnt_off"]), f"{tag}: shard offsets"


def check_apply(sess: GradDropSession, exp: dict, p_before: np.ndarray, params: torch.Tensor, alpha: float, tag: str):
    push = {"idx": exp["idx"], "val": exp.get("val"), "means": exp.get("means")}
    cols = sess.layer_cols
    got = params.cpu().numpy()
    for j in range(sess.n_shards):
        lo, hi = sess.shard_off[j], sess.shard_off[j + 1]
        ref, bound = orc.apply_pushes(p_before[lo:hi], lo, [push], alpha=alpha, value_mode=sess.value_mode,
                                      layer_off=sess.layer_off, layer_cols=cols)
        err = np.abs(got[lo:hi].astype(np.float64) - ref)
        assert np.all(err <= REL_TOL * bound + 1e-45), f"{tag}: shard {j} max err {err.max()}"
        if alpha == 1.0 and sess.value_mode == B.GD_VALUES_FP32:     # one push, alpha 1: exactly fl32(p + v)
            want = p_before[lo:hi].copy()
            sel = (exp["idx"] >= lo) & (exp["idx"] < hi)
            want[exp["idx"][sel].astype(np.int64) - lo] += exp["val"][sel]
            assert np.array_equal(got[lo:hi].view(np.uint32), want.view(np.uint32)), f"{tag}: shard {j} not exact"


def run_steps(w, device, steps, flags=0, method="sort", grads=None, alpha=1.0, with_apply=True, expect_dense=None,
              layer_cols=None):
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, flags, device,
                           layer_cols=layer_cols)
    r_host = orc.residual_reset(w.n)
    params = W.make_params(w, device) if with_apply else None
    views = sess.shard_views(params) if with_apply else None
    for step in range(steps):
        g = grads[step].to(device) if grads is not None else W.make_gradient(w, step, device)
        g_host = g.cpu().numpy()
        exp = orc.compress(g_host, r_host, w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode,
                           method=method, layer_cols=layer_cols,
                           error_feedback=bool(flags & B.GD_FLAG_QUANT_ERROR_FEEDBACK))
        g_before = g.clone()
        sess.compress(g)
        tag = f"{w.name} step {step} flags {flags}"
        compare_step(sess, exp, tag)
        assert torch.equal(g, g_before), f"{tag}: gradient was modified"
        if expect_dense is not None:
            st = sess.stats()
            assert (st["n_scopes_dense"] > 0) == expect_dense, f"{tag}: stats {st}"
        if with_apply:
            p_before = params.cpu().numpy().copy()
            sess.apply(views, alpha)
            torch.cuda.synchronize()
            check_apply(sess, exp, p_before, params, alpha, tag)
        r_host = exp["residual"]
    return sess


# ---------------------------------------------------------------- workload 1: 2^20 flat, 5 steps
@pytest.mark.parametrize("flags", [0, B.GD_FLAG_NO_PREDICTION, B.GD_FLAG_PREDICT_ALWAYS,
                                   B.GD_FLAG_PREDICT_ALWAYS | B.GD_FLAG_PLAIN_RADIX])
def test_config1_five_steps(cuda_device, flags):
    """Short enough for the one-launch dense kernel, which is the default here; with GD_FLAG_PREDICT_ALWAYS through the
    sample, the fused pass and the lists."""
    run_steps(W.workload(1), cuda_device, 5, flags=flags, expect_dense=not flags & B.GD_FLAG_PREDICT_ALWAYS)


@pytest.mark.parametrize("flags", [0, B.GD_FLAG_NO_PREDICTION])
def test_config1_shape_at_2_19(cuda_device, flags):
    """Half the length of workload 1: short enough to be selected densely whatever the flags (three passes out of L2)."""
    run_steps(W.workload(1, scale_log2=19), cuda_device, 3, flags=flags, expect_dense=True)


@pytest.mark.parametrize("flags", [0, B.GD_FLAG_NO_PREDICTION, B.GD_FLAG_NO_EARLY_ZERO, B.GD_FLAG_PLAIN_RADIX])
def test_config1_shape_at_2_23(cuda_device, flags):
    """The same distribution just above the length where the prediction is switched on."""
    run_steps(W.workload(1, scale_log2=23), cuda_device, 3, flags=flags, method="select",
              expect_dense=bool(flags & B.GD_FLAG_NO_PREDICTION))


# ---------------------------------------------------------------- edge sizes and drop ratios
@pytest.mark.parametrize("flags", [0, B.GD_FLAG_NO_PREDICTION])
def test_edge_sizes(cuda_device, flags):
    rng = np.random.default_rng(42)
    for n in (1, 2, 3, 31, 32, 33, 255, 4095, 4096, 4097, 8191, 12289, 70001):
        for ppm in (0, 500_000, 990_000, 999_999, 1_000_000):
            w = W.small_layered(1, [n], ppm, B.GD_SCOPE_GLOBAL, B.GD_VALUES_FP32, 1)
            g = torch.from_numpy(rng.laplace(0, 1e-3, n).astype(np.float32))
            g2 = torch.from_numpy(rng.laplace(0, 1e-3, n).astype(np.float32))
            run_steps(w, cuda_device, 2, flags=flags, grads=[g, g2])


def test_empty_gradient(cuda_device):
    w = W.small_layered(2, [0, 0], 990_000, B.GD_SCOPE_PER_LAYER, B.GD_VALUES_FP32, 2)
    run_steps(w, cuda_device, 1, grads=[torch.empty(0)], with_apply=False)


@pytest.mark.parametrize("flags", [0, B.GD_FLAG_NO_PREDICTION])
@pytest.mark.parametrize("scope_mode", [B.GD_SCOPE_GLOBAL, B.GD_SCOPE_PER_LAYER])
@pytest.mark.parametrize("value_mode", [B.GD_VALUES_FP32, B.GD_VALUES_TWO_MEANS, B.GD_VALUES_THRESHOLD])
def test_ragged_layers(cuda_device, flags, scope_mode, value_mode):
    sizes = [10, 0, 37, 1, 4096 + 5, 5, 100_003, 3, 8192, 2]      # unaligned starts, tiny and empty layers
    rng = np.random.default_rng(7)
    for ppm, shards in ((990_000, 3), (900_000, 1), (0, 4), (1_000_000, 2)):
        w = W.small_layered(len(sizes), sizes, ppm, scope_mode, value_mode, shards)
        grads = [torch.from_numpy((rng.standard_normal(w.n) * 10.0 ** rng.integers(-4, 0, w.n)).astype(np.float32))
                 for _ in range(3)]
        run_steps(w, cuda_device, 3, flags=flags, grads=grads, alpha=0.5 if ppm == 900_000 else 1.0)


# ---------------------------------------------------------------- ties
@pytest.mark.parametrize("flags", [0, B.GD_FLAG_NO_PREDICTION])
def test_heavy_ties(cuda_device, flags):
    rng = np.random.default_rng(13)
    n = 300_007
    cases = {
        "all_zero": np.zeros(n, np.float32),
        "all_equal": np.full(n, -2.5, np.float32),
        "few_levels": rng.choice(np.array([0.0, -0.0, 0.5, -0.5, 0.75, 3.0, -3.0, 1e-40], np.float32), n),
        "outliers_at_one_value": np.where(rng.random(n) < 0.01, np.float32(0.2) * rng.choice([-1, 1], n),
                                          rng.standard_normal(n) * 1e-2).astype(np.float32),
        "mostly_zero": np.where(rng.random(n) < 0.004, rng.standard_normal(n), 0).astype(np.float32),
    }
    for name, g in cases.items():
        for scope_mode in (B.GD_SCOPE_GLOBAL, B.GD_SCOPE_PER_LAYER):
            w = W.small_layered(3, [100_000, 7, n - 100_007], 990_000, scope_mode, B.GD_VALUES_FP32, 2)
            w.name = name
            run_steps(w, cuda_device, 2, flags=flags, grads=[torch.from_numpy(g), torch.from_numpy(g)])


@pytest.mark.parametrize("flags", [0, B.GD_FLAG_NO_EARLY_ZERO, B.GD_FLAG_PLAIN_RADIX])
def test_ties_and_dense_runs_on_the_predicted_path(cuda_device, flags):
    """Vectors long enough for the prediction (above 2^21 elements), shaped to reach every branch behind it:
    lists that overflow (the scope is then selected densely, after the slots cleared early got v back), warps
    whose stash overflows (runs of candidates), estimates of tau above and below the real one, ties at the cut."""
    rng = np.random.default_rng(17)
    n = (1 << 22) + 12_345
    one_up = np.frombuffer(np.uint32(0x3F800001).tobytes(), dtype=np.float32)[0]       # just above a bucket edge
    base = (rng.laplace(0, 1e-3, n)).astype(np.float32)
    cases = {}
    g = base.copy(); g[rng.random(n) < 0.4] = one_up; cases["many_ties_above_a_bucket_edge"] = g
    g = base.copy(); g[1_000_000:1_005_000] = 0.5; g[3_000_000:3_002_000] = -0.75; cases["runs_of_kept_entries"] = g
    g = base.copy(); g[500_000:540_000] = np.float32(6.5e-3) * rng.choice([-1, 1], 40_000).astype(np.float32)
    cases["run_of_ties_around_the_cut"] = g                      # about k entries share one magnitude near tau
    g = np.where(rng.random(n) < 0.012, rng.standard_normal(n), 0.0).astype(np.float32)
    cases["mostly_zero_just_above_k_nonzeros"] = g
    g = np.where(rng.random(n) < 0.008, rng.standard_normal(n), 0.0).astype(np.float32)
    cases["mostly_zero_fewer_nonzeros_than_k"] = g
    cases["all_equal"] = np.full(n, -2.5, np.float32)
    g = base.copy(); g[::3] *= 40.0; cases["a_third_forty_times_larger"] = g
    for name, g in cases.items():
        for scope_mode in (B.GD_SCOPE_GLOBAL, B.GD_SCOPE_PER_LAYER):
            w = W.small_layered(3, [1_500_000, 7, n - 1_500_007], 990_000, scope_mode, B.GD_VALUES_FP32, 2)
            w.name = name
            run_steps(w, cuda_device, 2, flags=flags, grads=[torch.from_numpy(g), torch.from_numpy(-g)])


def test_signed_zero_and_subnormals(cuda_device):
    n = 5000
    rng = np.random.default_rng(3)
    g = (rng.standard_normal(n) * 1e-41).astype(np.float32)          # all subnormal
    g[::7] = -0.0
    g[5::11] = 0.0
    w = W.small_layered(1, [n], 900_000, B.GD_SCOPE_GLOBAL, B.GD_VALUES_FP32, 1)
    run_steps(w, cuda_device, 3, grads=[torch.from_numpy(g), torch.from_numpy(-g), torch.from_numpy(g)])


@pytest.mark.parametrize("flags", [0, B.GD_FLAG_NO_PREDICTION])
def test_infinities_are_the_largest_magnitudes(cuda_device, flags):
    """+-inf order above every finite value by bit pattern and add deterministically, so parity stays bit-exact
    (the infinities leave the residual when they are sent, so no inf - inf arises)."""
    n = (1 << 22) + 77
    rng = np.random.default_rng(21)
    g = rng.laplace(0, 1e-3, n).astype(np.float32)
    pos = rng.choice(n, size=300, replace=False)
    g[pos[:150]] = np.inf
    g[pos[150:]] = -np.inf
    g[-1] = np.float32(3.4028235e38)                                     # the largest finite value
    w = W.small_layered(1, [n], 999_000, B.GD_SCOPE_GLOBAL, B.GD_VALUES_FP32, 2)
    run_steps(w, cuda_device, 2, flags=flags, grads=[torch.from_numpy(g), torch.from_numpy(g)], with_apply=False)


@pytest.mark.parametrize("flags", [0, B.GD_FLAG_NO_PREDICTION])
def test_nan_inputs_are_sent_not_stuck(cuda_device, flags):
    """NaNs are outside the bit-exact contract (the payload of NaN + x differs between processors), but they
    must behave: every NaN has a larger key than any number, so all of them are sent (there are fewer than k),
    the numbers that fill the rest of the quota are the oracle's, and the call ends with status ok."""
    n = (1 << 22) + 5
    rng = np.random.default_rng(22)
    g = rng.laplace(0, 1e-3, n).astype(np.float32)
    nan_pos = np.sort(rng.choice(n, size=200, replace=False))
    g[nan_pos] = np.nan
    w = W.small_layered(1, [n], 999_000, B.GD_SCOPE_GLOBAL, B.GD_VALUES_FP32, 2)
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, flags, cuda_device)
    sess.compress(torch.from_numpy(g).to(cuda_device))
    assert sess.status() == B.GD_OK
    exp = orc.compress(g, orc.residual_reset(n), w.layer_off, w.shard_off, w.drop_ppm)
    k = sess.k_total
    got_idx = _np_u32(sess.out_idx)[:k]
    got_val = sess.out_val.cpu().numpy()[:k]
    assert np.array_equal(got_idx, exp["idx"])                           # same positions: NaNs first in rank, then numbers
    assert np.array_equal(np.flatnonzero(np.isnan(got_val)), np.flatnonzero(np.isin(got_idx, nan_pos)))
    finite = ~np.isnan(got_val)
    assert np.array_equal(got_val[finite].view(np.uint32), exp["val"][finite].view(np.uint32))
    res = sess.residual.cpu().numpy()
    assert not np.isnan(res).any()
    assert np.array_equal(res.view(np.uint32), exp["residual"].view(np.uint32))
    assert int(_np_u32(sess.out_tau)[0]) == int(exp["tau"][0])


def test_integer_gradients_conserve_mass(cuda_device):
    """Error feedback loses nothing: sent mass + residual == sum of the gradients, exactly."""
    n, steps = 1 << 18, 8
    w = W.small_layered(2, [1000, n - 1000], 990_000, B.GD_SCOPE_PER_LAYER, B.GD_VALUES_FP32, 4)
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, 0, cuda_device)
    gen = torch.Generator(device=cuda_device).manual_seed(5)
    total = torch.zeros(n, dtype=torch.int64, device=cuda_device)
    params = torch.zeros(n, dtype=torch.float32, device=cuda_device)
    views = sess.shard_views(params)
    for _ in range(steps):
        g = torch.randint(-1024, 1025, (n,), generator=gen, device=cuda_device).to(torch.float32)
        total += g.to(torch.int64)
        sess.compress(g)
        sess.apply(views)
    assert sess.status() == B.GD_OK
    assert torch.equal(params.to(torch.int64) + sess.residual.to(torch.int64), total)


# ---------------------------------------------------------------- workloads 2, 3, 4 (shapes of the paper's models)
@pytest.mark.parametrize("scope_mode", [B.GD_SCOPE_GLOBAL, B.GD_SCOPE_PER_LAYER])
def test_config2_mnist_shaped(cuda_device, scope_mode):
    # the workload's 20 steps with either scope, error feedback carried, every step compared with the oracle
    run_steps(W.workload(2, scope_mode=scope_mode), cuda_device, 20, method="select", expect_dense=False)


def test_config3_threshold_quantisation(cuda_device):
    w = W.workload(4)
    w.value_mode = B.GD_VALUES_THRESHOLD
    run_steps(w, cuda_device, 1, method="select")


def test_bounded_wait_gives_up_and_context_survives(cuda_device):
    """A wait on a tile that nothing publishes runs out of polls, one on an mbarrier at which nothing arrives runs out
    of time; both report a timeout, and the next calls (short and long vectors) work."""
    ws = torch.zeros(4096, dtype=torch.uint8, device=cuda_device)
    B.gd_selftest_bounded_wait(ws, spin_limit=2000)
    st = B.gd_get_stats(ws)
    assert st["status"] == B.GD_ERR_DEVICE_TIMEOUT
    assert st["n_scopes"] == 1            # the first wait gave up
    assert st["n_scopes_predicted"] == 1  # the tile behind it aborted instead of waiting
    assert st["n_kept"] == 1              # the wait on an mbarrier at which nothing arrives gave up too
    run_steps(W.workload(1), cuda_device, 1)
    w = W.small_layered(2, [2_000_000, 900_001], 990_000, B.GD_SCOPE_PER_LAYER, B.GD_VALUES_FP32, 2)
    run_steps(w, cuda_device, 1, grads=[torch.randn(w.n, generator=torch.Generator().manual_seed(3)) * 1e-3])


def test_config2_no_prediction(cuda_device):
    run_steps(W.workload(2, scope_mode=B.GD_SCOPE_PER_LAYER), cuda_device, 1, flags=B.GD_FLAG_NO_PREDICTION,
              method="select", expect_dense=True)


def test_config3_and_config4_twenty_steps(cuda_device):
    """The NMT-shaped workloads at their full length: 20 steps, residual carried, every step compared with the oracle.

    Workload 4 is workload 3 with two-value quantisation, so both run on the same gradients, each with a
    session (and residual) of its own.  The oracle is called once per step, in two-means mode: what it returns
    for the selection (positions, values, residual, thresholds, shard offsets) does not depend on the value
    mode, so the fp32 expectation is the same record with the sign bits taken off the packed positions.
    """
    w3, w4 = W.workload(3), W.workload(4)
    assert w3.layer_off == w4.layer_off and w3.shard_off == w4.shard_off and w3.drop_ppm == w4.drop_ppm
    s3 = GradDropSession(w3.layer_off, w3.shard_off, w3.drop_ppm, w3.scope_mode, w3.value_mode, 0, cuda_device)
    s4 = GradDropSession(w4.layer_off, w4.shard_off, w4.drop_ppm, w4.scope_mode, w4.value_mode, 0, cuda_device)
    p3, p4 = W.make_params(w3, cuda_device), W.make_params(w4, cuda_device)
    v3, v4 = s3.shard_views(p3), s4.shard_views(p4)
    r_host = orc.residual_reset(w3.n)
    for step in range(20):
        g = W.make_gradient(w3, step, cuda_device)
        exp4 = orc.compress(g.cpu().numpy(), r_host, w4.layer_off, w4.shard_off, w4.drop_ppm, w4.scope_mode,
                            w4.value_mode, method="select")
        exp3 = dict(exp4)
        exp3["idx"] = exp4["idx"] & np.uint32(0x7FFFFFFF)
        s3.compress(g)
        s4.compress(g)
        compare_step(s3, exp3, f"workload 3 step {step}")
        compare_step(s4, exp4, f"workload 4 step {step}")
        for st in (s3.stats(), s4.stats()):
            assert st["n_scopes_dense"] == 0, st
        for sess, exp, params, views in ((s3, exp3, p3, v3), (s4, exp4, p4, v4)):
            p_before = params.cpu().numpy().copy()
            sess.apply(views)
            torch.cuda.synchronize()
            check_apply(sess, exp, p_before, params, 1.0, f"workload {3 if sess is s3 else 4} step {step}")
        r_host = exp4["residual"]


def test_config4_matches_config3_sets(cuda_device):
    w3, w4 = W.workload(3), W.workload(4)
    s3 = GradDropSession(w3.layer_off, w3.shard_off, w3.drop_ppm, w3.scope_mode, w3.value_mode, 0, cuda_device)
    s4 = GradDropSession(w4.layer_off, w4.shard_off, w4.drop_ppm, w4.scope_mode, w4.value_mode, 0, cuda_device)
    g = W.make_gradient(w3, 0, cuda_device)
    s3.compress(g)
    s4.compress(g)
    assert s3.status() == B.GD_OK and s4.status() == B.GD_OK
    k = s3.k_total
    assert torch.equal(s3.out_idx[:k], s4.out_idx[:k] & 0x7FFFFFFF)
    assert torch.equal(s3.out_tau, s4.out_tau)
    assert torch.equal(s3.residual.view(torch.int32), s4.residual.view(torch.int32))


# ---------------------------------------------------------------- workload 5 at reduced and at full scale
def test_config5_reduced_scale(cuda_device):
    run_steps(W.workload(5, scale_log2=24), cuda_device, 2, method="select", expect_dense=False)


def test_determinism_two_runs(cuda_device):
    w = W.workload(5, scale_log2=22)
    outs = []
    for _ in range(2):
        sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, 0, cuda_device)
        for step in range(2):
            sess.compress(W.make_gradient(w, step, cuda_device))
        outs.append((sess.out_idx.clone(), sess.out_val.clone(), sess.residual.clone()))
    for a, b in zip(*outs):
        assert torch.equal(a.view(torch.int32), b.view(torch.int32))


def test_config5_full_scale_properties(cuda_device):
    """2^30 elements in the launch configuration the benchmark times.

    The workload's 10 steps with the residual carried.  Every step is checked through the properties that
    define the result at any size: the threshold is the k-th largest key (fewer than k keys above it, at
    least k at or above it), every key above it is kept, the ties kept are the lowest-index ones, positions
    ascend, values and residual reassemble v bit for bit, shard offsets and the applied parameters follow.
    Together these fix the result uniquely, so the check is as strong as a comparison with the sorted
    definition.  On the first and the last step the threshold is also compared with a host-side selection
    of the k-th largest of the 2^30 keys (a library routine, not the CUDA path).
    """
    free, _total = torch.cuda.mem_get_info()
    if free < 40 * (1 << 30):
        pytest.skip("needs 40 GiB of free device memory")
    w = W.workload(5)
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, 0, cuda_device)
    params = torch.zeros(w.n, dtype=torch.float32, device=cuda_device)
    views = sess.shard_views(params)
    steps = 10
    for step in range(steps):
        g = W.make_gradient(w, step, cuda_device)
        v = g + sess.residual                       # the same single fp32 add, by the tensor library
        sess.compress(g)
        assert sess.status() == B.GD_OK
        st = sess.stats()
        assert st["n_scopes_dense"] == 0, st
        k = sess.k_total
        idx = sess.out_idx[:k].to(torch.int64) & 0xFFFFFFFF
        val = sess.out_val[:k]
        tau = int(_np_u32(sess.out_tau)[0])
        keys = v.view(torch.int32) & 0x7FFFFFFF
        if step in (0, steps - 1):                  # threshold against a host selection of the k-th largest key
            keys_host = keys.cpu().numpy().view(np.uint32)
            kth = np.partition(keys_host, w.n - k)[w.n - k]
            assert int(kth) == tau
            del keys_host
        n_gt = int((keys > tau).sum().item())
        n_eq = int((keys == tau).sum().item())
        assert n_gt < k <= n_gt + n_eq
        assert bool((idx[1:] > idx[:-1]).all())
        assert torch.equal(val.view(torch.int32), v[idx].view(torch.int32))
        kept_keys = keys[idx]
        assert int((kept_keys > tau).sum().item()) == n_gt          # every key above tau is kept
        assert int(kept_keys.min().item()) == tau
        ties = torch.nonzero(keys == tau).flatten()
        assert torch.equal(ties[: k - n_gt], idx[kept_keys == tau])  # the lowest-index ties
        expect_res = v.clone()
        expect_res[idx] = 0.0
        assert torch.equal(sess.residual.view(torch.int32), expect_res.view(torch.int32))
        bounds = torch.tensor(w.shard_off, device=cuda_device)
        assert torch.equal(torch.searchsorted(idx, bounds).to(torch.int32), sess.out_shard_cnt_off)
        p_before = params.clone()
        sess.apply(views)
        p_before[idx] += val
        assert torch.equal(params.view(torch.int32), p_before.view(torch.int32))
        del v, keys, expect_res, p_before, g


@pytest.mark.parametrize("value_mode", [B.GD_VALUES_FP32, B.GD_VALUES_TWO_MEANS])
def test_many_layers_and_shards(cuda_device, value_mode):
    """More layers and shards than fit a kernel argument: the tables go through the workspace instead."""
    rng = np.random.default_rng(99)
    sizes = [int(x) for x in rng.integers(0, 9000, size=70)]
    sizes[5] = 0
    sizes[17] = 70_000
    for scope_mode in (B.GD_SCOPE_GLOBAL, B.GD_SCOPE_PER_LAYER):
        w = W.small_layered(len(sizes), sizes, 980_000, scope_mode, value_mode, 40)
        grads = [torch.from_numpy(rng.laplace(0, 1e-3, w.n).astype(np.float32)) for _ in range(2)]
        run_steps(w, cuda_device, 2, grads=grads)


@pytest.mark.parametrize("value_mode", [B.GD_VALUES_FP32, B.GD_VALUES_TWO_MEANS])
@pytest.mark.parametrize("scope_mode", [B.GD_SCOPE_GLOBAL, B.GD_SCOPE_PER_LAYER])
def test_many_layers_on_the_predicted_path(cuda_device, scope_mode, value_mode):
    """A model with a hundred and twenty tensors, long enough (about 12 M elements) to take the predicted path:
    more scopes than the kernels keep in shared memory, tables too large for a kernel argument, layers that are
    empty, tiny, unaligned, all zero, or sampled completely."""
    rng = np.random.default_rng(1234)
    sizes = [int(x) for x in rng.integers(1, 200_000, size=120)]
    sizes[3], sizes[4], sizes[50], sizes[77], sizes[119] = 0, 1, 7, 1_000_003, 33
    w = W.small_layered(len(sizes), sizes, 990_000, scope_mode, value_mode, 5)
    assert w.n > (1 << 21)
    grads = []
    for _ in range(2):
        g = rng.laplace(0, 1e-3, w.n).astype(np.float32)
        g[w.layer_off[10]:w.layer_off[11]] = 0.0                          # an all-zero layer: every entry ties
        lo, hi = w.layer_off[20], w.layer_off[21]
        g[lo:hi] = np.where(rng.random(hi - lo) < 0.002, g[lo:hi], 0.0)    # fewer non-zeros than k
        grads.append(torch.from_numpy(g))
    sess = run_steps(w, cuda_device, 2, grads=grads)
    st = sess.stats()
    assert st["n_scopes_predicted"] >= 1


# ---------------------------------------------------------------- guard words around every buffer
@pytest.mark.parametrize("case", ["predicted_fp32", "predicted_two_means", "dense_fp32", "dense_one_launch", "sampled",
                                  "many_scopes"])
def test_nothing_is_written_outside_the_buffers(cuda_device, case):
    """Every buffer the library writes (residual, outputs, workspace, parameters) sits between guard words; the guards
    must be intact after compress + apply and the outputs must equal the oracle's.  Buffers have exactly the sizes the
    sizing calls return."""
    rng = np.random.default_rng(5150)
    G = 1024                                                       # guard elements on either side
    value_mode, flags, scope = B.GD_VALUES_FP32, 0, B.GD_SCOPE_PER_LAYER
    sizes = [1_300_000, 9, 4097, 1_000_003]                        # short enough for the one-launch dense kernel ...
    if case == "predicted_fp32":
        flags = B.GD_FLAG_PREDICT_ALWAYS                            # ... so the predicted path is asked for
    elif case == "predicted_two_means":
        value_mode, flags = B.GD_VALUES_TWO_MEANS, B.GD_FLAG_PREDICT_ALWAYS
    elif case == "dense_fp32":
        sizes = [200_001, 9, 4097]
    elif case == "sampled":
        flags = B.GD_FLAG_SAMPLED_THRESHOLD
    elif case == "many_scopes":
        sizes = [1_200_000] + [int(x) for x in rng.integers(1, 5000, size=45)] + [900_001]
    w = W.small_layered(len(sizes), sizes, 990_000, scope, value_mode, 3)
    n = w.n
    sampled = bool(flags & B.GD_FLAG_SAMPLED_THRESHOLD)
    k_cap = (B.gd_sampled_capacity(w.layer_off, scope, w.drop_ppm) if sampled
             else B.gd_total_kept(w.layer_off, scope, w.drop_ppm))
    n_scopes = len(sizes)
    ws_bytes = B.gd_workspace_bytes(w.layer_off, w.n_shards, scope, w.drop_ppm, None)
    aws_bytes = B.gd_apply_workspace_bytes(w.n_shards, len(sizes))

    def padded(count, dtype, fill):
        t = torch.full((count + 2 * G,), fill, dtype=dtype, device=cuda_device)
        return t, t[G:G + count]

    def intact(t, count, fill):
        ref = torch.full((G,), fill, dtype=t.dtype, device=t.device)
        return torch.equal(t[:G], ref) and torch.equal(t[G + count:], ref)

    res_t, res = padded(n, torch.float32, 7.0)
    res.zero_()
    par_t, par = padded(n, torch.float32, 7.0)
    par.zero_()
    idx_t, idx = padded(max(k_cap, 1), torch.int32, 0x5A5A5A5A)
    val_t, val = padded(max(k_cap, 1), torch.float32, 7.0)
    off_t, off = padded(w.n_shards + 1, torch.int32, 0x5A5A5A5A)
    tau_t, tau = padded(n_scopes, torch.int32, 0x5A5A5A5A)
    mean_t, mean = padded(2 * len(sizes), torch.float32, 7.0)
    ws_t, ws = padded(ws_bytes, torch.uint8, 0x5A)
    aws_t, aws = padded(aws_bytes, torch.uint8, 0x5A)
    g_host = rng.laplace(0, 1e-3, n).astype(np.float32)
    grad = torch.from_numpy(g_host).to(cuda_device)
    call = B.CompressCall(grad, res, w.layer_off, w.shard_off, w.drop_ppm, scope, value_mode, idx, val, off, tau,
                          mean.view(-1, 2), ws, flags=flags)
    B.gd_compress(call)
    assert B.gd_status(ws) == B.GD_OK
    st = B.gd_get_stats(ws)
    if case.startswith("predicted"):
        assert st["n_scopes_predicted"] >= 2 and st["n_scopes_dense"] == 0, st
    elif case.startswith("dense"):
        assert st["n_scopes_dense"] == len(sizes) and st["n_candidates"] == 0, st   # the one-launch kernel: no lists
    views = [par[w.shard_off[j]:w.shard_off[j + 1]] for j in range(w.n_shards)]
    push = {"idx": idx, "val": None if value_mode != B.GD_VALUES_FP32 else val, "shard_cnt_off": off,
            "means": mean.view(-1, 2) if value_mode != B.GD_VALUES_FP32 else None}
    acall = B.ApplyCall(views, w.shard_off, [push], value_mode, 1.0, aws, layer_off=w.layer_off)
    B.gd_decompress_apply(acall)
    torch.cuda.synchronize()
    for name, t, count, fill in (("residual", res_t, n, 7.0), ("params", par_t, n, 7.0),
                                 ("out_idx", idx_t, max(k_cap, 1), 0x5A5A5A5A), ("out_val", val_t, max(k_cap, 1), 7.0),
                                 ("out_shard_cnt_off", off_t, w.n_shards + 1, 0x5A5A5A5A),
                                 ("out_tau", tau_t, n_scopes, 0x5A5A5A5A), ("out_means", mean_t, 2 * len(sizes), 7.0),
                                 ("workspace", ws_t, ws_bytes, 0x5A), ("apply workspace", aws_t, aws_bytes, 0x5A)):
        assert intact(t, count, fill), f"{case}: guard words around {name} were overwritten"
    r0 = orc.residual_reset(n)
    if sampled:
        exp = orc.compress_sampled(g_host, r0, w.layer_off, w.shard_off, w.drop_ppm, scope)
    else:
        exp = orc.compress(g_host, r0, w.layer_off, w.shard_off, w.drop_ppm, scope, value_mode)
    K = exp["idx"].shape[0]
    assert np.array_equal(_np_u32(idx)[:K], exp["idx"])
    assert np.array_equal(_np_u32(res), exp["residual"].view(np.uint32))
    assert np.array_equal(_np_u32(tau), exp["tau"])
    if value_mode == B.GD_VALUES_FP32:
        sent = np.zeros(n, np.float32)
        sent[exp["idx"]] = exp["val"]
        assert np.array_equal(_np_u32(par), sent.view(np.uint32))


# ---------------------------------------------------------------- other drop ratios (Section 5.1: 90 %, 99 %, 99.9 %)
@pytest.mark.parametrize("drop_ppm", [900_000, 999_000])
@pytest.mark.parametrize("config", [2, 3])
def test_drop_ratio_sweep(cuda_device, config, drop_ppm):
    """The paper's other two drop ratios on the MNIST- and NMT-shaped sets (at 90 % the push is 10x larger,
    most warps of the fused pass overflow their stash, and the apply matters)."""
    w = W.workload(config, scope_mode=B.GD_SCOPE_PER_LAYER)
    w.drop_ppm = drop_ppm
    run_steps(w, cuda_device, 2, method="select")


def test_more_kept_than_nonzero(cuda_device):
    """Row-sparse layers whose non-zero entries number fewer than k: the threshold is 0 and the lowest-index
    zeros fill the quota (the NMT embeddings at a 90 % drop ratio)."""
    rng = np.random.default_rng(5)
    sizes = [200_000, 64, 300_001]
    grads = []
    for _ in range(2):
        g = np.zeros(sum(sizes), np.float32)
        rows = rng.choice(sizes[0] // 500, 12, replace=False)
        for r_ in rows:
            g[r_ * 500:(r_ + 1) * 500] = rng.standard_normal(500) * 1e-3
        g[sizes[0] + sizes[1]:] = np.where(rng.random(sizes[2]) < 0.03, rng.standard_normal(sizes[2]), 0)
        grads.append(torch.from_numpy(g))
    for scope_mode in (B.GD_SCOPE_PER_LAYER, B.GD_SCOPE_GLOBAL):
        w = W.small_layered(3, sizes, 900_000, scope_mode, B.GD_VALUES_FP32, 3)
        sess = run_steps(w, cuda_device, 2, grads=grads)
        assert sess.stats()["n_scopes_dense"] >= 1


# ---------------------------------------------------------------- several workers pushing into one server shard
@pytest.mark.parametrize("apply_flags", [0, B.GD_APPLY_ATOMIC], ids=["ordered", "atomic"])
@pytest.mark.parametrize("value_mode", [B.GD_VALUES_FP32, B.GD_VALUES_TWO_MEANS])
def test_three_workers_push_into_each_server(cuda_device, value_mode, apply_flags):
    """Section 3: every server owns 1/N of the parameters and receives one piece from every worker.  Three
    workers compress their own gradients; each of the 4 servers applies the three pieces of its shard in
    one call (pushes collide on many indices), either one after another or - GD_APPLY_ATOMIC - in one launch
    with atomic updates; the fp64 reference admits any order."""
    rng = np.random.default_rng(17)
    sizes = [30_000, 11, 50_001]
    w = W.small_layered(3, sizes, 950_000, B.GD_SCOPE_PER_LAYER, value_mode, 4)
    workers, expected = [], []
    for _ in range(3):
        sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, 0, cuda_device)
        g = rng.laplace(0, 1e-3, w.n).astype(np.float32)
        g[rng.integers(0, w.n, 2000)] *= 50.0                      # shared hot spots are unlikely; force some
        g[:500] += 0.5
        exp = orc.compress(g, orc.residual_reset(w.n), w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode)
        sess.compress(torch.from_numpy(g).to(cuda_device))
        compare_step(sess, exp, "worker")
        workers.append(sess)
        expected.append(exp)
    p0 = (rng.standard_normal(w.n) * 0.01).astype(np.float32)
    params = torch.from_numpy(p0).to(cuda_device)
    aws = torch.empty(B.gd_apply_workspace_bytes(1, len(sizes)), dtype=torch.uint8, device=cuda_device)
    for j in range(w.n_shards):                                    # server j: its shard only, pieces j of all workers
        lo, hi = w.shard_off[j], w.shard_off[j + 1]
        pushes = []
        for sess in workers:
            p = {"idx": sess.out_idx, "shard_cnt_off": sess.out_shard_cnt_off[j:j + 2]}
            if value_mode == B.GD_VALUES_FP32:
                p["val"] = sess.out_val
            else:
                p["means"] = sess.out_means
            pushes.append(p)
        call = B.ApplyCall([params[lo:hi]], [lo, hi], pushes, value_mode, 0.25, aws,
                           w.layer_off if value_mode != B.GD_VALUES_FP32 else None, flags=apply_flags)
        before = B.gd_launch_count()
        B.gd_decompress_apply(call)
        assert B.gd_launch_count() - before == (1 if apply_flags else 3)
    torch.cuda.synchronize()
    got = params.cpu().numpy().astype(np.float64)
    collisions = 0
    for j in range(w.n_shards):
        lo, hi = w.shard_off[j], w.shard_off[j + 1]
        ref, bound = orc.apply_pushes(p0[lo:hi], lo, expected, alpha=0.25, value_mode=value_mode, layer_off=w.layer_off)
        assert np.all(np.abs(got[lo:hi] - ref) <= REL_TOL * bound + 1e-45), f"server {j}"
    hits = np.zeros(w.n, np.int32)
    for exp in expected:
        hits[(exp["idx"] & np.uint32(0x7FFFFFFF)).astype(np.int64)] += 1
    assert (hits >= 2).sum() > 100                                 # the pushes really collide


def test_atomic_apply_of_many_colliding_pushes_keeps_subnormals(cuda_device):
    """Forty workers (more than one launch's worth of pushes) push the same positions into one server at once.
    With values that are small multiples of the smallest subnormal every partial sum is exact in fp32, so the
    atomic apply must give the exact total whatever the order - which an add that flushed subnormals would not -
    and a second set of ordinary values stays within the fp64 reference's tolerance."""
    n, workers = 50_000, 40
    w = W.small_layered(1, [n], 900_000, B.GD_SCOPE_GLOBAL, B.GD_VALUES_FP32, 1)
    tiny = np.float32(1.401298464324817e-45)                      # 2^-149
    rng = np.random.default_rng(5)
    for scale, exact in ((tiny, True), (np.float32(1e-3), False)):
        sessions, expected = [], []
        for wk in range(workers):
            mult = rng.integers(1, 8, n).astype(np.float32)
            sign = rng.choice(np.array([-1.0, 1.0], np.float32), n)
            g = (mult * sign * scale).astype(np.float32) if exact else (rng.laplace(0, 1, n).astype(np.float32) * scale)
            g[rng.random(n) < 0.5] *= np.float32(0.125) if not exact else np.float32(1.0)
            g[::7] = np.float32(64.0) * scale * sign[::7]         # every worker keeps these: they all collide
            sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, 0, cuda_device)
            sess.compress(torch.from_numpy(g).to(cuda_device))
            assert sess.status() == B.GD_OK
            expected.append(orc.compress(g, orc.residual_reset(n), w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode))
            sessions.append(sess)
        params = torch.zeros(n, device=cuda_device)
        aws = torch.empty(B.gd_apply_workspace_bytes(1, 1), dtype=torch.uint8, device=cuda_device)
        call = B.ApplyCall([params], [0, n], [s_.push() for s_ in sessions], B.GD_VALUES_FP32, 1.0, aws, flags=B.GD_APPLY_ATOMIC)
        before = B.gd_launch_count()
        B.gd_decompress_apply(call)
        torch.cuda.synchronize()
        assert B.gd_launch_count() - before == 2                   # forty pushes: a set of 32 and a set of 8
        ref, bound = orc.apply_pushes(np.zeros(n, np.float32), 0, expected)
        got = params.cpu().numpy()
        if exact:
            assert np.array_equal(got.astype(np.float64), ref)     # sums of small multiples of 2^-149: no rounding anywhere
            assert np.count_nonzero(got) > 1000
        else:
            assert np.all(np.abs(got.astype(np.float64) - ref) <= REL_TOL * bound + 1e-45)


# ---------------------------------------------------------------- parameter pulls as dropped deltas
@pytest.mark.parametrize("flags", [0, B.GD_FLAG_NO_PREDICTION])
@pytest.mark.parametrize("layout", ["short", "long_global", "long_per_layer", "long_many"])
def test_delta_pull_matches_oracle_and_client_copy(cuda_device, flags, layout):
    """Section 4, third paragraph: the server sends GradDrop(params - last pulled copy).  The library's
    delta mode must equal the oracle bit for bit, and the server's record of the client's copy must stay
    identical to what the client holds after applying the pull with alpha = 1."""
    rng = np.random.default_rng(23)
    # short vectors are selected densely; the long ones take the predicted path (fused subtraction, candidates,
    # slots cleared in the stream), the last one with more scopes than the kernels keep in shared memory
    sizes = {"short": [70_000, 9, 4096, 130_003], "long_global": [2_500_000, 9, 4096, 900_003],
             "long_per_layer": [2_500_000, 9, 4096, 900_003],
             "long_many": [1_200_000] + [int(x) for x in rng.integers(1, 6000, size=50)] + [1_000_000]}[layout]
    scope = B.GD_SCOPE_GLOBAL if layout in ("short", "long_global") else B.GD_SCOPE_PER_LAYER
    w = W.small_layered(len(sizes), sizes, 980_000, scope, B.GD_VALUES_FP32, 2)
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, flags, cuda_device)
    p_host = (rng.standard_normal(w.n) * 0.1).astype(np.float32)
    last_host = np.zeros(w.n, dtype=np.float32)
    last_dev = torch.zeros(w.n, dtype=torch.float32, device=cuda_device)
    client = torch.zeros(w.n, dtype=torch.float32, device=cuda_device)
    client_views = sess.shard_views(client)
    for step in range(4):
        p_host = p_host + rng.laplace(0, 1e-3, w.n).astype(np.float32)
        p_dev = torch.from_numpy(p_host).to(cuda_device)
        exp = orc.compress_delta(p_host, last_host, w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode)
        sess.compress_delta(p_dev, last_dev)
        compare_step(sess, exp, f"pull {step} flags {flags}")
        if flags == 0:
            assert (sess.stats()["n_scopes_predicted"] >= 1) == (layout != "short"), sess.stats()
        assert np.array_equal(_np_u32(last_dev), exp["last_pulled"].view(np.uint32)), f"pull {step}: last pulled copy"
        assert torch.equal(p_dev.cpu(), torch.from_numpy(p_host)), "parameters were modified"
        sess.apply(client_views, 1.0)
        torch.cuda.synchronize()
        assert torch.equal(client.view(torch.int32), last_dev.view(torch.int32)), f"pull {step}: client copy differs"
        last_host = exp["last_pulled"]


# ---------------------------------------------------------------- sampled threshold (Section 4: select on a 0.1 % sample)
def compare_sampled(sess, exp, tag):
    assert sess.status() == B.GD_OK, f"{tag}: device status {sess.status()}"
    K = exp["idx"].shape[0]
    assert sess.kept() == K, f"{tag}: kept {sess.kept()} vs {K}"
    assert K <= sess.k_total
    assert np.array_equal(_np_u32(sess.out_tau), exp["tau"]), f"{tag}: thresholds"
    assert np.array_equal(_np_u32(sess.out_idx)[:K], exp["idx"]), f"{tag}: indices"
    assert np.array_equal(_np_u32(sess.out_val)[:K], exp["val"].view(np.uint32)), f"{tag}: values"
    assert np.array_equal(_np_u32(sess.residual), exp["residual"].view(np.uint32)), f"{tag}: residual"
    assert np.array_equal(_np_u32(sess.out_shard_cnt_off), exp["shard_cnt_off"]), f"{tag}: shard offsets"


@pytest.mark.parametrize("extra_flags", [0, B.GD_FLAG_NO_EARLY_ZERO])
@pytest.mark.parametrize("scope_mode", [B.GD_SCOPE_GLOBAL, B.GD_SCOPE_PER_LAYER])
def test_sampled_threshold_matches_oracle(cuda_device, scope_mode, extra_flags):
    rng = np.random.default_rng(61)
    sizes = [3000, 0, 4096, 4097, 10, 700_001, 64_000]           # whole-scope samples, 4096-sample scopes, a 0.1 % scope
    for ppm in (990_000, 900_000, 1_000_000):
        w = W.small_layered(len(sizes), sizes, ppm, scope_mode, B.GD_VALUES_FP32, 3)
        sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode,
                               B.GD_FLAG_SAMPLED_THRESHOLD | extra_flags, cuda_device)
        params = torch.zeros(w.n, dtype=torch.float32, device=cuda_device)
        views = sess.shard_views(params)
        r_host = orc.residual_reset(w.n)
        sent = np.zeros(w.n, np.float32)
        for step in range(3):
            g = rng.laplace(0, 1e-3, w.n).astype(np.float32)
            g[rng.random(w.n) < 0.2] = 0.0
            exp = orc.compress_sampled(g, r_host, w.layer_off, w.shard_off, ppm, scope_mode)
            sess.compress(torch.from_numpy(g).to(cuda_device))
            compare_sampled(sess, exp, f"sampled ppm {ppm} step {step}")
            sess.apply(views)
            sent[exp["idx"]] += exp["val"]
            r_host = exp["residual"]
        torch.cuda.synchronize()
        assert np.array_equal(_np_u32(params), sent.view(np.uint32))


def test_sampled_threshold_with_many_scopes(cuda_device):
    """Sixty tensors, each its own scope (the many-scope instantiation of the selection kernel, where lists of a
    single tile are selected inside one CTA), in sampled-threshold mode with its three radix passes."""
    rng = np.random.default_rng(62)
    sizes = [int(x) for x in rng.integers(1, 9000, size=56)] + [0, 4096, 250_000, 1_200_000]
    w = W.small_layered(len(sizes), sizes, 990_000, B.GD_SCOPE_PER_LAYER, B.GD_VALUES_FP32, 4)
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode,
                           B.GD_FLAG_SAMPLED_THRESHOLD, cuda_device)
    r_host = orc.residual_reset(w.n)
    for step in range(3):
        g = rng.laplace(0, 1e-3, w.n).astype(np.float32)
        g[rng.random(w.n) < 0.1] = 0.0
        exp = orc.compress_sampled(g, r_host, w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode)
        sess.compress(torch.from_numpy(g).to(cuda_device))
        compare_sampled(sess, exp, f"sampled, 60 scopes, step {step}")
        r_host = exp["residual"]


def _sampled_band(lo, hi, drop_ppm):
    """Relative error allowed for kept / k of one scope in sampled-threshold mode: the threshold comes from k_m tail
    samples (relative rank error about 1 / sqrt(k_m)), taken as pairs of neighbours (at worst half as many
    independent samples): five such standard deviations.  None for scopes sampled completely."""
    if hi - lo <= 4096:
        return None
    m = orc.sampled_positions(lo, hi, 0).shape[0]
    return 5.0 * (2.0 / max(orc.kept_count(m, drop_ppm), 1)) ** 0.5


@pytest.mark.parametrize("config", [1, 2, 3, 5])
def test_sampled_threshold_kept_count_error_on_the_workloads(cuda_device, config):
    """Section 4, fourth paragraph, as an approximation: on every workload (workload 4 has workload 3's selection),
    three steps with the residual carried, the sampled-threshold result equals its oracle bit for bit and the
    number kept per scope stays within the sampling error of the exact count k - the row-sparse embeddings of
    workload 3 included, where the sample of a tensor that is 98 % zeros still holds more non-zero entries
    than k_m, so the threshold is positive.  Workload 5 runs at its full 2^30 elements; there the oracle states
    the sample positions and the threshold, and the survivors are checked as the set of entries at or above it."""
    full5 = config == 5
    if full5:
        free, _ = torch.cuda.mem_get_info()
        if free < 30 * (1 << 30):
            pytest.skip("needs 30 GiB of free device memory")
    w = W.workload(config, scope_mode=B.GD_SCOPE_PER_LAYER) if config == 2 else W.workload(config)
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode,
                           B.GD_FLAG_SAMPLED_THRESHOLD, cuda_device)
    scopes = orc.scopes_of(w.layer_off, w.scope_mode)
    r_host = None if full5 else orc.residual_reset(w.n)
    for step in range(3):
        g = W.make_gradient(w, step, cuda_device)
        if full5:
            v = g + sess.residual
            sess.compress(g)
            assert sess.status() == B.GD_OK
            pos = orc.sampled_positions(0, w.n, 0)
            sample = v[torch.from_numpy(pos).to(cuda_device)].cpu().numpy()
            m = pos.shape[0]
            t = int(np.sort(orc.magnitude_keys(sample))[m - orc.kept_count(m, w.drop_ppm)])
            assert int(_np_u32(sess.out_tau)[0]) == t
            kept = sess.kept()
            keys = v.view(torch.int32) & 0x7FFFFFFF
            want = torch.nonzero(keys >= t).flatten()
            assert kept == want.numel()
            idx = sess.out_idx[:kept].to(torch.int64) & 0xFFFFFFFF
            assert torch.equal(idx, want)
            assert torch.equal(sess.out_val[:kept].view(torch.int32), v[idx].view(torch.int32))
            v[idx] = 0.0
            assert torch.equal(sess.residual.view(torch.int32), v.view(torch.int32))
            got_idx = idx.cpu().numpy()
            del v, keys, want, idx
        else:
            exp = orc.compress_sampled(g.cpu().numpy(), r_host, w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode)
            sess.compress(g)
            compare_sampled(sess, exp, f"sampled workload {config} step {step}")
            r_host = exp["residual"]
            got_idx = exp["idx"].astype(np.int64)
        for lo, hi in scopes:
            k = orc.kept_count(hi - lo, w.drop_ppm)
            kept_s = int(np.searchsorted(got_idx, hi) - np.searchsorted(got_idx, lo))
            band = _sampled_band(lo, hi, w.drop_ppm)
            if band is None:
                assert kept_s >= k
            else:
                assert abs(kept_s / k - 1.0) <= band, f"workload {config} step {step} scope [{lo}, {hi}): {kept_s} vs {k}"


def test_sampled_threshold_of_zero_is_an_overflow(cuda_device):
    """A scope so sparse that its sample holds fewer non-zero entries than k_m gets the threshold key 0, i.e. every
    entry would be kept: far beyond the capacity, so the call reports GD_ERR_OVERFLOW (its outputs and residual are
    then undefined; a caller that expects such tensors uses the exact selection, which takes the same input).
    0.2 % non-zero entries at a 99 % drop ratio."""
    n = 2_000_000
    g = torch.zeros(n, device=cuda_device)
    g[::500] = 1e-3
    w = W.small_layered(1, [n], 990_000, B.GD_SCOPE_GLOBAL, B.GD_VALUES_FP32, 2)
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode,
                           B.GD_FLAG_SAMPLED_THRESHOLD, cuda_device)
    exp = orc.compress_sampled(g.cpu().numpy(), orc.residual_reset(n), w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode)
    assert int(exp["tau"][0]) == 0 and exp["idx"].shape[0] == n            # the oracle keeps everything
    sess.compress(g)
    assert sess.status() == B.GD_ERR_OVERFLOW
    exact = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, 0, cuda_device)
    exact.compress(g)                                                      # the exact selection takes the same input
    assert exact.status() == B.GD_OK


def test_sampled_threshold_overflow_is_reported(cuda_device):
    n = 1_000_000                                                   # every entry ties with the threshold: all are kept
    w = W.small_layered(1, [n], 990_000, B.GD_SCOPE_GLOBAL, B.GD_VALUES_FP32, 1)
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode,
                           B.GD_FLAG_SAMPLED_THRESHOLD, cuda_device)
    sess.compress(torch.full((n,), 0.25, device=cuda_device))
    assert sess.status() == B.GD_ERR_OVERFLOW
    run_steps(W.workload(1), cuda_device, 1)                        # the context is fine afterwards


# ---------------------------------------------------------------- beyond 2^31 elements (64-bit offsets, full uint32 indices)
@pytest.mark.parametrize("flags", [0, B.GD_FLAG_NO_PREDICTION], ids=["predicted", "dense"])
@pytest.mark.parametrize("n", [(1 << 31) + (1 << 20) + 5, 1 << 32], ids=["2^31+2^20+5", "2^32"])
def test_more_than_2_31_elements(cuda_device, n, flags):
    """n = 2^31 + 2^20 + 5: byte offsets pass 2^33 and indices pass 2^31; n = 2^32: the largest gradient the library
    takes, whose last index is 0xFFFFFFFF.  The oracle's sort does not fit here, so the result is pinned by what
    defines it: tau is the k-th largest key iff #{key > tau} < k <= #{key >= tau}; the kept set is every key above
    tau plus the lowest-index ties; values and residual reassemble v; the push lands on exactly the kept slots."""
    gc.collect()
    torch.cuda.empty_cache()                                              # what earlier tests left in the caching allocator
    free, _ = torch.cuda.mem_get_info()
    need = (16 * n + (12 << 30))
    if free < need:
        pytest.skip(f"needs {need >> 30} GiB of free device memory")
    w = W.small_layered(1, [n], 999_000, B.GD_SCOPE_GLOBAL, B.GD_VALUES_FP32, 3)
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, flags, cuda_device)
    gen = torch.Generator(device=cuda_device).manual_seed(2031)
    g = torch.empty(n, dtype=torch.float32, device=cuda_device)
    chunk = 1 << 26
    for lo in range(0, n, chunk):
        hi = min(lo + chunk, n)
        g[lo:hi] = torch.randn(hi - lo, generator=gen, device=cuda_device) * 1e-3
    g[n - 3:] = torch.tensor([5.0, -6.0, 7.0], device=cuda_device)          # the very last entries must be kept
    g[(1 << 31) - 1] = -8.0
    g[1 << 31] = 9.0
    k = sess.k_total
    for step in range(2):
        r_before = sess.residual.clone()
        sess.compress(g)
        assert sess.status() == B.GD_OK
        assert sess.stats()["n_scopes_dense"] == (1 if flags else 0)
        tau = int(_np_u32(sess.out_tau)[0])
        idx = sess.out_idx[:k].to(torch.int64) & 0xFFFFFFFF
        assert bool((idx[1:] > idx[:-1]).all()) and int(idx[-1]) == n - 1
        n_gt = n_eq = 0
        kept_mask_count = 0
        for lo in range(0, n, chunk):                                      # chunked: no tensor larger than 2^26 here
            hi = min(lo + chunk, n)
            v = g[lo:hi] + r_before[lo:hi]
            keys = v.view(torch.int32) & 0x7FFFFFFF
            n_gt += int((keys > tau).sum())
            n_eq += int((keys == tau).sum())
            sel = idx[(idx >= lo) & (idx < hi)] - lo
            kept = torch.zeros(hi - lo, dtype=torch.bool, device=cuda_device)
            kept[sel] = True
            kept_mask_count += int(kept.sum())
            assert bool((keys[kept] >= tau).all()) and bool((keys[~kept] <= tau).all())
            want_res = torch.where(kept, torch.zeros_like(v), v)
            assert torch.equal(sess.residual[lo:hi].view(torch.int32), want_res.view(torch.int32))
        assert n_gt < k <= n_gt + n_eq and kept_mask_count == k
        v_kept = g[idx] + r_before[idx]
        assert torch.equal(sess.out_val[:k].view(torch.int32), v_kept.view(torch.int32))
        for probe in ((1 << 31) - 1, 1 << 31, n - 3, n - 2, n - 1):
            assert bool((idx == probe).any())                              # the planted large entries, both sides of 2^31
        bounds = torch.tensor(w.shard_off, device=cuda_device)
        assert torch.equal(torch.searchsorted(idx, bounds).to(torch.int32), sess.out_shard_cnt_off)
        del r_before
    # the server side at these indices: p <- 0 + 1 * value on the kept slots of the three shards, nothing else touched
    params = torch.zeros(n, dtype=torch.float32, device=cuda_device)
    sess.apply(sess.shard_views(params))
    assert sess.status() == B.GD_OK
    assert torch.equal(params[idx], sess.out_val[:k])
    touched = 0
    for lo in range(0, n, chunk):
        touched += int(torch.count_nonzero(params[lo:min(lo + chunk, n)]))
    assert touched == int(torch.count_nonzero(sess.out_val[:k]))


def test_sampled_threshold_on_the_largest_gradient(cuda_device):
    """Section 4, fourth paragraph, at n = 2^32: the sample positions (from the oracle's statement of the rule, here
    4.3 M of them, up to index 2^32 - 1) fix the threshold; the survivors are then every entry at or above it."""
    n = 1 << 32
    gc.collect()
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < 12 * n + (12 << 30):
        pytest.skip("needs 60 GiB of free device memory")
    w = W.small_layered(1, [n], 999_000, B.GD_SCOPE_GLOBAL, B.GD_VALUES_FP32, 3)
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode,
                           B.GD_FLAG_SAMPLED_THRESHOLD, cuda_device)
    gen = torch.Generator(device=cuda_device).manual_seed(2032)
    g = torch.empty(n, dtype=torch.float32, device=cuda_device)
    chunk = 1 << 26
    for lo in range(0, n, chunk):
        g[lo:lo + chunk] = torch.randn(chunk, generator=gen, device=cuda_device) * 1e-3
    g[n - 1] = 7.0
    sess.compress(g)                                                       # residual is zero: v = g
    assert sess.status() == B.GD_OK
    pos = orc.sampled_positions(0, n, 0)
    m = pos.shape[0]
    assert m == ((n + 999) // 1000 + 1) // 2 * 2 and int(pos.max()) < n and int(pos.max()) > n - 4000
    sample = g[torch.from_numpy(pos.astype(np.int64)).to(cuda_device)].cpu().numpy()
    k_m = orc.kept_count(m, w.drop_ppm)
    t = int(np.sort(orc.magnitude_keys(sample))[m - k_m])
    assert int(_np_u32(sess.out_tau)[0]) == t
    kept = sess.kept()
    count = 0
    for lo in range(0, n, chunk):
        count += int(((g[lo:lo + chunk].view(torch.int32) & 0x7FFFFFFF) >= t).sum())
    assert kept == count and abs(kept / (n / 1000) - 1.0) < 0.05
    idx = sess.out_idx[:kept].to(torch.int64) & 0xFFFFFFFF
    assert bool((idx[1:] > idx[:-1]).all()) and int(idx[-1]) == n - 1
    assert torch.equal(sess.out_val[:kept].view(torch.int32), g[idx].view(torch.int32))
    assert int(((g[idx].view(torch.int32) & 0x7FFFFFFF) >= t).sum()) == kept
    assert int(torch.count_nonzero(sess.residual[idx])) == 0
    g[idx] = 0.0                                                           # what the residual must be now
    assert torch.equal(sess.residual.view(torch.int32), g.view(torch.int32))
    bounds = torch.tensor(w.shard_off, device=cuda_device)
    assert torch.equal(torch.searchsorted(idx, bounds).to(torch.int32), sess.out_shard_cnt_off)


def test_delta_pull_beyond_2_31_elements(cuda_device):
    """Section 4, third paragraph, with indices on both sides of 2^31: the dropped delta v = params - last pulled copy,
    pinned by the rank counts that define the threshold; the server's copy advances by exactly what was sent and the
    client's copy, which applies the pull, stays identical to it."""
    n = (1 << 31) + (1 << 20) + 5
    gc.collect()
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < 20 * n + (8 << 30):
        pytest.skip("needs 50 GiB of free device memory")
    w = W.small_layered(1, [n], 999_000, B.GD_SCOPE_GLOBAL, B.GD_VALUES_FP32, 3)
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, 0, cuda_device)
    gen = torch.Generator(device=cuda_device).manual_seed(2033)
    chunk = 1 << 26
    params = torch.empty(n, dtype=torch.float32, device=cuda_device)
    for lo in range(0, n, chunk):
        hi = min(lo + chunk, n)
        params[lo:hi] = torch.randn(hi - lo, generator=gen, device=cuda_device) * 0.1
    last = torch.zeros(n, dtype=torch.float32, device=cuda_device)
    client = torch.zeros(n, dtype=torch.float32, device=cuda_device)
    client_views = sess.shard_views(client)
    k = sess.k_total
    for step in range(2):
        for lo in range(0, n, chunk):                                      # the parameters move on between pulls
            hi = min(lo + chunk, n)
            params[lo:hi] += torch.randn(hi - lo, generator=gen, device=cuda_device) * 1e-2
        params[n - 1] += 9.0
        params[1 << 31] -= 8.0
        last_before = last.clone()
        sess.compress_delta(params, last)
        assert sess.status() == B.GD_OK
        tau = int(_np_u32(sess.out_tau)[0])
        idx = sess.out_idx[:k].to(torch.int64) & 0xFFFFFFFF
        assert bool((idx[1:] > idx[:-1]).all()) and int(idx[-1]) == n - 1 and bool((idx == (1 << 31)).any())
        n_gt = n_eq = n_kept = 0
        for lo in range(0, n, chunk):
            hi = min(lo + chunk, n)
            v = params[lo:hi] - last_before[lo:hi]
            keys = v.view(torch.int32) & 0x7FFFFFFF
            n_gt += int((keys > tau).sum())
            n_eq += int((keys == tau).sum())
            kept = torch.zeros(hi - lo, dtype=torch.bool, device=cuda_device)
            kept[idx[(idx >= lo) & (idx < hi)] - lo] = True
            n_kept += int(kept.sum())
            assert bool((keys[kept] >= tau).all()) and bool((keys[~kept] <= tau).all())
            assert torch.equal(sess.residual[lo:hi].view(torch.int32),
                               torch.where(kept, torch.zeros_like(v), v).view(torch.int32))
            assert torch.equal(last[lo:hi].view(torch.int32),
                               torch.where(kept, last_before[lo:hi] + v, last_before[lo:hi]).view(torch.int32))
        assert n_gt < k <= n_gt + n_eq and n_kept == k
        assert torch.equal(sess.out_val[:k].view(torch.int32), (params[idx] - last_before[idx]).view(torch.int32))
        del last_before
        sess.apply(client_views, 1.0)
        assert sess.status() == B.GD_OK
        assert torch.equal(client.view(torch.int32), last.view(torch.int32))


def test_two_means_at_the_packing_limit(cuda_device):
    """n = 2^31, the most a packed word (31 index bits + the sign, Section 5.4's 1-bit values) can address: the last
    element is negative and kept, so its word is 0xFFFFFFFF.  Checked against the definitions: threshold by rank
    counts, sign bits against v, centres against an fp64 mean of the kept values, the push against the centres."""
    n = 1 << 31
    gc.collect()
    torch.cuda.empty_cache()                                              # what earlier tests left in the caching allocator
    free, _ = torch.cuda.mem_get_info()
    if free < 16 * n + (8 << 30):
        pytest.skip("needs 40 GiB of free device memory")
    w = W.small_layered(1, [n], 999_000, B.GD_SCOPE_GLOBAL, B.GD_VALUES_TWO_MEANS, 2)
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, 0, cuda_device)
    gen = torch.Generator(device=cuda_device).manual_seed(2131)
    g = torch.empty(n, dtype=torch.float32, device=cuda_device)
    chunk = 1 << 26
    for lo in range(0, n, chunk):
        g[lo:lo + chunk] = torch.randn(chunk, generator=gen, device=cuda_device) * 1e-3
    g[n - 1] = -4.0
    g[0] = 3.0
    k = sess.k_total
    sess.compress(g)                                                       # residual is zero: v = g
    assert sess.status() == B.GD_OK
    tau = int(_np_u32(sess.out_tau)[0])
    word = sess.out_idx[:k].to(torch.int64) & 0xFFFFFFFF
    idx, sign = word & 0x7FFFFFFF, word >> 31
    assert int(word[-1]) == 0xFFFFFFFF and int(word[0]) == 0
    assert bool((idx[1:] > idx[:-1]).all())
    v_kept = g[idx]
    assert torch.equal(sign, (v_kept.view(torch.int32) >> 31) & 1)
    n_gt = n_eq = 0
    for lo in range(0, n, chunk):
        keys = g[lo:lo + chunk].view(torch.int32) & 0x7FFFFFFF
        n_gt += int((keys > tau).sum())
        n_eq += int((keys == tau).sum())
    assert n_gt < k <= n_gt + n_eq
    assert int(((v_kept.view(torch.int32) & 0x7FFFFFFF) >= tau).sum()) == k
    assert int(torch.count_nonzero(sess.residual[idx])) == 0
    want_res = g.clone()
    want_res[idx] = 0.0
    assert torch.equal(sess.residual.view(torch.int32), want_res.view(torch.int32))
    del want_res
    means = sess.out_means[0].double().cpu().numpy()
    for sgn in (0, 1):
        ref = float(v_kept[sign == sgn].double().mean())
        assert abs(means[sgn] - ref) <= REL_TOL * abs(ref), (sgn, means[sgn], ref)
    params = torch.zeros(n, dtype=torch.float32, device=cuda_device)
    sess.apply(sess.shard_views(params))
    assert sess.status() == B.GD_OK
    assert torch.equal(params[idx], sess.out_means[0][sign])               # 0 + 1 * centre, exactly
    touched = 0
    for lo in range(0, n, chunk):
        touched += int(torch.count_nonzero(params[lo:lo + chunk]))
    assert touched == k


# ---------------------------------------------------------------- column-wise averages (Section 5.4)
@pytest.mark.parametrize("flags", [0, B.GD_FLAG_NO_PREDICTION])
@pytest.mark.parametrize("scope_mode", [B.GD_SCOPE_GLOBAL, B.GD_SCOPE_PER_LAYER])
def test_column_means_small_matrices(cuda_device, flags, scope_mode):
    shapes = [(300, 40), (17,), (64, 500), (1, 33), (2000, 3)]
    sizes = [int(np.prod(s_)) for s_ in shapes]
    cols = [s_[-1] if len(s_) > 1 else 1 for s_ in shapes]
    rng = np.random.default_rng(88)
    w = W.small_layered(len(sizes), sizes, 950_000, scope_mode, B.GD_VALUES_COLUMN_MEANS, 3)
    grads = [torch.from_numpy(rng.laplace(0, 1e-3, w.n).astype(np.float32)) for _ in range(2)]
    run_steps(w, cuda_device, 2, flags=flags, grads=grads, layer_cols=cols, alpha=0.5)


def test_column_means_on_the_nmt_shapes(cuda_device):
    w = W.workload(4)
    w.value_mode = B.GD_VALUES_COLUMN_MEANS
    sess = run_steps(w, cuda_device, 1, method="select", layer_cols=w.layer_cols)
    assert sess.n_pairs == sum(w.layer_cols) == 500 + 500 + 85000 + 1 + 8 * 1000


# ---------------------------------------------------------------- quantisation error fed back into the residual
@pytest.mark.parametrize("flags", [0, B.GD_FLAG_NO_PREDICTION])
@pytest.mark.parametrize("scope_mode", [B.GD_SCOPE_GLOBAL, B.GD_SCOPE_PER_LAYER])
@pytest.mark.parametrize("value_mode", [B.GD_VALUES_TWO_MEANS, B.GD_VALUES_THRESHOLD, B.GD_VALUES_COLUMN_MEANS])
def test_quantisation_error_feedback(cuda_device, flags, scope_mode, value_mode):
    """Kept slots hold v - decoded instead of +0.  The kept magnitudes of a layer span far less than 2^18, so
    the fp64 sums behind the means are exact in any order and the residual is compared bit for bit, over
    three steps with the residual carried (a difference in step 1 would change the selection of step 2)."""
    shapes = [(600, 50), (4097,), (128, 1000), (3,), (5000, 8), (2300, 1000)]   # 2.5 M elements: the predicted path
    sizes = [int(np.prod(s_)) for s_ in shapes]
    cols = [s_[-1] if len(s_) > 1 else 1 for s_ in shapes] if value_mode == B.GD_VALUES_COLUMN_MEANS else None
    rng = np.random.default_rng(4242)
    w = W.small_layered(len(sizes), sizes, 980_000, scope_mode, value_mode, 3)
    grads = [torch.from_numpy(rng.laplace(0, 1e-3, w.n).astype(np.float32)) for _ in range(3)]
    sess = run_steps(w, cuda_device, 3, flags=flags | B.GD_FLAG_QUANT_ERROR_FEEDBACK, grads=grads, layer_cols=cols,
                     alpha=0.5)
    # the fed-back error is not zero: some kept slot holds a non-zero residual
    kept = _np_u32(sess.out_idx)[:sess.k_total] & np.uint32(0x7FFFFFFF)
    assert np.count_nonzero(sess.residual.cpu().numpy()[kept.astype(np.int64)]) > 0


def test_quantisation_error_feedback_on_the_nmt_shapes(cuda_device):
    w = W.workload(4)
    run_steps(w, cuda_device, 2, flags=B.GD_FLAG_QUANT_ERROR_FEEDBACK, method="select")


def test_quantisation_error_feedback_needs_a_one_bit_mode(cuda_device):
    w = W.small_layered(1, [100_000], 990_000, B.GD_SCOPE_GLOBAL, B.GD_VALUES_FP32, 1)
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode,
                           B.GD_FLAG_QUANT_ERROR_FEEDBACK, cuda_device)
    with pytest.raises(B.GdError):
        sess.compress(torch.zeros(w.n, device=cuda_device))


@pytest.mark.parametrize("which", ["grad", "residual"])
def test_vectors_must_be_aligned_to_16_bytes(cuda_device, which):
    """The kernels read and write 128 bits at a time (and the fused pass copies whole tiles in bulk): a gradient or
    residual that starts off a 16-byte boundary is refused, with nothing launched."""
    w = W.small_layered(2, [300_000, 17], 990_000, B.GD_SCOPE_PER_LAYER, B.GD_VALUES_FP32, 1)
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, 0, cuda_device)
    buf = torch.zeros(w.n + 8, dtype=torch.float32, device=cuda_device)
    g = torch.zeros(w.n, dtype=torch.float32, device=cuda_device)
    if which == "grad":
        g = buf[1:1 + w.n]
    else:
        sess.residual = buf[1:1 + w.n]                       # before the first call: the argument block is built then
    before = B.gd_launch_count()
    with pytest.raises(B.GdError):
        sess.compress(g)
    assert B.gd_launch_count() == before


# ---------------------------------------------------------------- randomised layouts
@pytest.mark.parametrize("seed", range(12))
def test_random_layouts_and_modes(cuda_device, seed):
    """Random layer structures (tiny, empty, unaligned, large), drop ratios, scopes, value modes, shard counts and
    value distributions, three steps each with the residual carried; everything compared with the oracle."""
    rng = np.random.default_rng(1000 + seed)
    n_layers = int(rng.integers(1, 9))
    sizes = []
    for _ in range(n_layers):
        kind = rng.integers(0, 5)
        sizes.append(int([0, rng.integers(1, 40), rng.integers(40, 5000), rng.integers(5000, 70_000),
                          rng.integers(70_000, 400_000)][kind]))
    if sum(sizes) == 0:
        sizes[0] = 1234
    ppm = int(rng.choice([0, 300_000, 900_000, 984_000, 990_000, 999_000, 999_999, 1_000_000]))
    scope_mode = int(rng.integers(0, 2))
    value_mode = int(rng.choice([B.GD_VALUES_FP32, B.GD_VALUES_TWO_MEANS, B.GD_VALUES_THRESHOLD, B.GD_VALUES_COLUMN_MEANS]))
    flags = int(rng.choice([0, B.GD_FLAG_PREDICT_ALWAYS, B.GD_FLAG_NO_PREDICTION]))
    shards = int(rng.integers(1, 7))
    cols = None
    if value_mode == B.GD_VALUES_COLUMN_MEANS:
        cols = []
        for s_ in sizes:
            divs = [c for c in (1, 2, 3, 5, 8, 16, 50, 64) if s_ % c == 0] or [1]
            cols.append(int(rng.choice(divs)))
    w = W.small_layered(n_layers, sizes, ppm, scope_mode, value_mode, shards)
    dist = int(rng.integers(0, 4))
    grads = []
    for _ in range(3):
        if dist == 0:
            g = rng.laplace(0, 1e-3, w.n)
        elif dist == 1:
            g = rng.standard_normal(w.n) * 10.0 ** rng.integers(-6, 1, w.n)
        elif dist == 2:
            g = np.where(rng.random(w.n) < 0.02, rng.standard_normal(w.n), 0.0)         # mostly exact zeros
        else:
            g = rng.choice(np.array([0.0, 0.25, -0.25, 0.5, 1.0, -2.0]), w.n)           # few distinct values
        grads.append(torch.from_numpy(g.astype(np.float32)))
    alpha = float(rng.choice([1.0, 0.5, -1.25]))
    if not flags & B.GD_FLAG_NO_PREDICTION and rng.random() < 0.3:
        flags |= B.GD_FLAG_NO_EARLY_ZERO
    if value_mode == B.GD_VALUES_THRESHOLD and rng.random() < 0.5:
        flags |= B.GD_FLAG_QUANT_ERROR_FEEDBACK      # the +-tau table is exact, so the fed-back residual is too
    run_steps(w, cuda_device, 3, flags=flags, grads=grads, layer_cols=cols, alpha=alpha)


@pytest.mark.parametrize("seed", range(8))
def test_random_models_of_few_large_tensors(cuda_device, seed):
    """One to nine tensors of 0.3 to 2.5 M elements (the predicted path with all tables in shared memory), random drop
    ratio, scope, value mode (column-wise means and fed-back threshold quantisation included), flags and value
    distribution (Laplace, mixed scales, mostly zero, heavy-tailed Student t, a run of tied values)."""
    rng = np.random.default_rng(90000 + seed)
    n_layers = int(rng.integers(1, 9))
    sizes = [int(rng.integers(300_000, 2_500_000)) for _ in range(n_layers)]
    if rng.random() < 0.5:
        sizes.append(int(rng.integers(0, 5000)))
    ppm = int(rng.choice([900_000, 984_000, 990_000, 990_000, 999_000, 999_900]))
    scope_mode = int(rng.integers(0, 2))
    value_mode = int(rng.choice([0, 0, 1, 2, 3]))
    flags = int(rng.choice([0, 0, 0, B.GD_FLAG_NO_EARLY_ZERO, B.GD_FLAG_NO_PREDICTION]))
    if value_mode == B.GD_VALUES_THRESHOLD and rng.random() < 0.5:
        flags |= B.GD_FLAG_QUANT_ERROR_FEEDBACK
    if seed % 2 == 1 and not flags & B.GD_FLAG_NO_PREDICTION:
        flags |= B.GD_FLAG_PLAIN_RADIX                # the selection's three plain radix passes instead of its short cut
    if not flags & B.GD_FLAG_NO_PREDICTION:
        flags |= B.GD_FLAG_PREDICT_ALWAYS             # (the models short enough for the one-launch dense kernel too)
    cols = None
    if value_mode == B.GD_VALUES_COLUMN_MEANS:
        cols = []
        for s_ in sizes:
            divs = [c for c in (1, 2, 4, 5, 8, 10, 16, 100, 1000) if s_ % c == 0] or [1]
            cols.append(int(rng.choice(divs)))
    w = W.small_layered(len(sizes), sizes, ppm, scope_mode, value_mode, int(rng.integers(1, 9)))
    dist = int(rng.integers(0, 5))
    grads = []
    for _ in range(2):
        if dist == 0:
            g = rng.laplace(0, 1e-3, w.n)
        elif dist == 1:
            g = rng.standard_normal(w.n) * 10.0 ** rng.integers(-4, 1, w.n)
        elif dist == 2:
            g = np.where(rng.random(w.n) < 0.03, rng.standard_normal(w.n), 0.0)
        elif dist == 3:
            g = rng.standard_t(2.0, w.n) * 1e-3
        else:
            g = rng.laplace(0, 1e-3, w.n)
            a = int(rng.integers(0, w.n - 20000))
            g[a:a + 20000] = rng.choice([0.5, -0.5, 1.0], 20000)
        grads.append(torch.from_numpy(g.astype(np.float32)))
    run_steps(w, cuda_device, 2, flags=flags, grads=grads, layer_cols=cols, alpha=float(rng.choice([1.0, 0.5])))


@pytest.mark.parametrize("seed", range(10))
def test_random_models_of_ten_to_48_tensors(cuda_device, seed):
    """Ten to 48 tensors from empty to 1.2 M elements (on both sides of the 32 scopes whose tables fit shared memory and
    the kernel argument, and of the length the one-launch dense kernel holds), random drop ratio, scope, value mode,
    shard count, flags and value distribution; three steps with the residual carried, everything compared with the
    oracle."""
    rng = np.random.default_rng(770000 + seed)
    n_layers = int(rng.integers(10, 49))
    sizes = []
    for _ in range(n_layers):
        kind = rng.integers(0, 6)
        sizes.append(int([0, rng.integers(1, 40), rng.integers(40, 5000), rng.integers(5000, 70_000),
                          rng.integers(70_000, 400_000), rng.integers(400_000, 1_200_000)][kind]))
    if sum(sizes) == 0:
        sizes[0] = 99_999
    ppm = int(rng.choice([300_000, 900_000, 984_000, 990_000, 990_000, 999_000, 999_900, 1_000_000]))
    scope_mode = int(rng.integers(0, 2))
    value_mode = int(rng.choice([0, 0, 1, 2]))
    flags = int(rng.choice([0, 0, B.GD_FLAG_PREDICT_ALWAYS, B.GD_FLAG_PREDICT_ALWAYS, B.GD_FLAG_NO_PREDICTION]))
    if not flags & B.GD_FLAG_NO_PREDICTION and rng.random() < 0.3:
        flags |= B.GD_FLAG_NO_EARLY_ZERO
    w = W.small_layered(n_layers, sizes, ppm, scope_mode, value_mode, int(rng.integers(1, 9)))
    dist = int(rng.integers(0, 4))
    grads = []
    for _ in range(3):
        if dist == 0:
            g = rng.laplace(0, 1e-3, w.n)
        elif dist == 1:
            g = rng.standard_normal(w.n) * 10.0 ** rng.integers(-6, 1, w.n)
        elif dist == 2:
            g = np.where(rng.random(w.n) < 0.02, rng.standard_normal(w.n), 0.0)
        else:
            g = rng.choice(np.array([0.0, 0.25, -0.25, 0.5, 1.0, -2.0]), w.n)
        grads.append(torch.from_numpy(g.astype(np.float32)))
    run_steps(w, cuda_device, 3, flags=flags, grads=grads, alpha=float(rng.choice([1.0, 0.5])))


@pytest.mark.parametrize("case", ["boundaries_at_every_offset", "dense_rows", "tiny_between_large", "full_lists"])
def test_pipelined_pass_edges(cuda_device, case):
    """What the pipelined fused pass treats specially, each on a layout too long for the one-launch dense kernel:
    scope boundaries at every offset modulo 4 inside a tile (tiles cut by a boundary are read element by element, the
    rest in bulk), a vector whose length is no multiple of 4, runs in which most entries are candidates (a warp's
    stash overflows and it reads its part of the chunk back), scopes shorter than a tile between long ones (chunks of a
    single cut tile), and candidate lists that fill up (a scope of ties: the early clearing is undone, the scope is
    selected densely).  Three steps each, residual carried, everything compared with the oracle."""
    rng = np.random.default_rng({"boundaries_at_every_offset": 1, "dense_rows": 2, "tiny_between_large": 3,
                                 "full_lists": 4}[case])
    if case == "boundaries_at_every_offset":
        sizes = [1_000_001, 500_002, 700_003, 4096 * 60 + 1, 300_007, 1_234_567 + 2]
    elif case == "dense_rows":
        sizes = [2_000_000, 1_500_000]
    elif case == "tiny_between_large":
        sizes = [1_200_000, 3, 0, 4095, 1, 1_300_000, 17, 4097, 900_000]
    else:
        sizes = [1_500_000, 1_000_000, 800_000]
    w = W.small_layered(len(sizes), sizes, 990_000, B.GD_SCOPE_PER_LAYER, B.GD_VALUES_FP32, 3)
    assert w.n > 2368 * 1024                                     # (more than the one-launch dense kernel holds)
    grads = []
    for step in range(3):
        g = rng.laplace(0, 1e-3, w.n).astype(np.float32)
        if case == "dense_rows":
            g[:] = 0.0                                            # row-sparse: 2 % of the rows of 500 are non-zero
            rows = rng.choice(w.n // 500, w.n // 500 // 50, replace=False)
            for r_ in rows[:2000]:
                g[r_ * 500:(r_ + 1) * 500] = rng.standard_normal(500).astype(np.float32) * 1e-3
            g[100_000:160_000] = rng.standard_normal(60_000).astype(np.float32)      # and one long run far above the rest
        elif case == "full_lists":
            lo, hi = w.layer_off[1], w.layer_off[2]
            g[lo:hi] = 0.25                                       # every entry of the second scope ties
        grads.append(torch.from_numpy(g))
    sess = run_steps(w, cuda_device, 3, grads=grads)
    st = sess.stats()
    if case == "full_lists":
        assert st["n_scopes_dense"] == 1 and st["n_scopes_predicted"] == 2, st
    else:
        assert st["n_scopes_dense"] == 0, st


@pytest.mark.parametrize("n_layers", [25, 26, 32])
def test_as_many_scopes_as_the_shared_tables_hold(cuda_device, n_layers):
    """Up to 32 tensors - as many scopes as the kernels keep in shared memory - the start of the call, the prediction
    and the tables travel in one launch's argument (4.6 KB of tables at 32), and the fused pass starts under that
    launch and waits for each scope's mark.  Empty, tiny and long tensors mixed, two
    means per tensor, three steps."""
    rng = np.random.default_rng(2400 + n_layers)
    sizes = [int(x) for x in rng.integers(1, 20_000, size=n_layers)]
    sizes[0], sizes[3], sizes[7], sizes[n_layers - 1] = 900_000, 0, 1_400_001, 700_003
    sizes[5] = 1
    w = W.small_layered(n_layers, sizes, 990_000, B.GD_SCOPE_PER_LAYER, B.GD_VALUES_TWO_MEANS, 4)
    assert w.n > 2368 * 1024
    grads = [torch.from_numpy(rng.laplace(0, 1e-3, w.n).astype(np.float32)) for _ in range(3)]
    sess = run_steps(w, cuda_device, 3, grads=grads)
    st = sess.stats()
    assert st["n_scopes_dense"] == 0 and st["n_scopes_predicted"] == n_layers, st
    before = B.gd_launch_count()
    sess.compress(grads[0].to(cuda_device))
    assert B.gd_launch_count() - before == 3          # setup + prediction, fused pass, selection + compaction


def test_empty_scopes_leave_their_neighbours_alone(cuda_device):
    """Empty tensors between others: the start of a call clears the state of every scope without a sample, and must
    clear exactly that (a store that reached 16 bytes into the next scope's state used to wipe that scope's
    prediction whenever it landed late, which sent the scope down the dense path: right results, at a cost).
    Thirty calls; every non-empty scope must stay on the predicted path in each, and the first two are compared with
    the oracle."""
    sizes = [1_500_000, 0, 4095, 0, 1_300_000, 0, 0, 17, 600_000]
    w = W.small_layered(len(sizes), sizes, 990_000, B.GD_SCOPE_PER_LAYER, B.GD_VALUES_FP32, 2)
    gen = torch.Generator().manual_seed(99)
    grads = [torch.randn(w.n, generator=gen) * 1e-3 for _ in range(2)]
    sess = run_steps(w, cuda_device, 2, grads=grads, with_apply=False)
    g = grads[0].to(cuda_device)
    for call in range(30):
        sess.compress(g)
        st = sess.stats()
        assert st["status"] == B.GD_OK and st["n_scopes_dense"] == 0 and st["n_scopes_predicted"] == len(sizes), (call, st)


@pytest.mark.parametrize("scope_mode", [B.GD_SCOPE_GLOBAL, B.GD_SCOPE_PER_LAYER])
def test_threshold_far_above_the_prediction(cuda_device, scope_mode):
    """Magnitudes spread evenly over 120 binades: the prediction's safety margin (a multiple of the expected rank for
    the small sample of a short tensor) then lies binades below the real threshold, beyond the range in which the
    selection among the candidates can start from the fused pass's histogram, so it runs its plain radix passes
    by itself.  Mixed with ordinary tensors in one call; three steps, residual carried."""
    rng = np.random.default_rng(314)
    sizes = [2_000_000, 20_000, 40_000, 1_000_000, 9_000]
    w = W.small_layered(len(sizes), sizes, 990_000, scope_mode, B.GD_VALUES_FP32, 3)
    grads = []
    for _ in range(3):
        g = rng.laplace(0, 1e-3, w.n).astype(np.float32)
        for l in (1, 2, 4):
            lo, hi = w.layer_off[l], w.layer_off[l + 1]
            mag = np.exp2(rng.uniform(-126.0, -6.0, hi - lo))
            g[lo:hi] = (mag * rng.choice([-1.0, 1.0], hi - lo)).astype(np.float32)
        grads.append(torch.from_numpy(g))
    run_steps(w, cuda_device, 3, grads=grads)


@pytest.mark.parametrize("scope_mode", [B.GD_SCOPE_GLOBAL, B.GD_SCOPE_PER_LAYER])
def test_more_scopes_than_the_tile_table_holds(cuda_device, scope_mode):
    """2600 tensors: more scopes than the shared-memory table of candidate tiles covers (2048), so the kernels over the
    candidate lists fall back to the numbering by capacity and to the tables in global memory."""
    rng = np.random.default_rng(2600)
    sizes = [int(x) for x in rng.integers(1, 2000, size=2600)]
    sizes[100], sizes[1500], sizes[2599] = 700_000, 300_000, 5
    w = W.small_layered(len(sizes), sizes, 990_000, scope_mode, B.GD_VALUES_FP32, 3)
    assert w.n > (1 << 21)
    grads = [torch.from_numpy(rng.laplace(0, 1e-3, w.n).astype(np.float32)) for _ in range(2)]
    sess = run_steps(w, cuda_device, 2, grads=grads)
    assert sess.stats()["n_scopes_predicted"] >= 1


@pytest.mark.parametrize("seed", range(6))
def test_random_models_of_many_tensors(cuda_device, seed):
    """Models of 40 to 400 tensors with log-uniform sizes (1 to 300 k elements, a few of 2 M), long enough for the
    predicted path: CTAs of the selection kernels cross many scopes, single-tile lists are selected locally,
    the candidate tiles are renumbered over hundreds of scopes."""
    rng = np.random.default_rng(7000 + seed)
    n_layers = int(rng.integers(40, 401))
    sizes = [int(np.exp(rng.uniform(0, np.log(300_000)))) for _ in range(n_layers)]
    for _ in range(3):
        sizes[int(rng.integers(0, n_layers))] = int(rng.integers(1_000_000, 2_000_000))
    sizes[int(rng.integers(0, n_layers))] = 0
    ppm = int(rng.choice([900_000, 990_000, 990_000, 999_000]))
    scope_mode = int(rng.choice([B.GD_SCOPE_PER_LAYER, B.GD_SCOPE_PER_LAYER, B.GD_SCOPE_GLOBAL]))
    value_mode = int(rng.choice([B.GD_VALUES_FP32, B.GD_VALUES_FP32, B.GD_VALUES_TWO_MEANS, B.GD_VALUES_THRESHOLD]))
    w = W.small_layered(n_layers, sizes, ppm, scope_mode, value_mode, int(rng.integers(1, 9)))
    assert w.n > (1 << 21)
    grads = []
    for _ in range(2):
        g = rng.laplace(0, 1e-3, w.n).astype(np.float32)
        for _ in range(4):                                      # some layers all zero, some nearly so, some tied
            l = int(rng.integers(0, n_layers))
            lo, hi = w.layer_off[l], w.layer_off[l + 1]
            kind = int(rng.integers(0, 3))
            if kind == 0:
                g[lo:hi] = 0.0
            elif kind == 1:
                g[lo:hi] = np.where(rng.random(hi - lo) < 0.003, g[lo:hi], 0.0)
            else:
                g[lo:hi] = rng.choice(np.array([0.0, 0.5, -0.5, 1.0], dtype=np.float32), hi - lo)
        grads.append(torch.from_numpy(g))
    run_steps(w, cuda_device, 2, grads=grads, alpha=0.5, flags=int(rng.choice([0, 0, B.GD_FLAG_NO_EARLY_ZERO])))


def test_config5_full_scale_against_the_oracle(cuda_device):
    """One step of workload 5 at its full 2^30 elements, compared with the oracle itself (selection on the
    composite keys: tens of GB of host memory, about a minute of host time)."""
    import psutil
    gc.collect()
    torch.cuda.empty_cache()                                              # what earlier tests left in the caching allocator
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * (1 << 30) or psutil.virtual_memory().available < 90 * (1 << 30):
        pytest.skip("needs 40 GiB of device memory and 90 GiB of host memory")
    w = W.workload(5)
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, 0, cuda_device)
    g = W.make_gradient(w, 0, cuda_device)
    r0 = W.make_gradient(w, 7, cuda_device) * 0.25                 # a non-trivial residual to start from
    sess.residual.copy_(r0)
    exp = orc.compress(g.cpu().numpy(), r0.cpu().numpy(), w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode,
                       method="select")
    del r0
    sess.compress(g)
    compare_step(sess, exp, "workload 5, 2^30 elements, oracle")
    assert sess.stats()["n_scopes_dense"] == 0
