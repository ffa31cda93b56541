"""The entry points around gd_compress / gd_decompress_apply, through the C ABI on a GPU:

  gd_step_host         the whole step for a caller whose gradient is in host memory (what the benchmark's
                       end-to-end figure times): what it copies back to the host is compared with the oracle;
  gd_profile_enable /  the event pairs the benchmark's roofline figure is read from: one pair per kernel,
  gd_profile_collect   tagged in launch order;
  gd_launch_count      the benchmark's count of kernel launches.
"""
import numpy as np
import pytest
import torch

from oracle import graddrop_oracle as orc
from paper_1704_05021_b200 import binding as B
from paper_1704_05021_b200 import workloads as W
from paper_1704_05021_b200.session import GradDropSession

pytestmark = pytest.mark.gpu

REL_TOL = 1e-6   # means and applied parameters against the fp64 reference


def _layout(value_mode):
    # long enough for the predicted path (sample, fused pass, candidate selection, compaction), ragged, 3 shards
    return W.small_layered(4, [1_700_000, 13, 900_003, 4096], 990_000, B.GD_SCOPE_PER_LAYER, value_mode, 3)


@pytest.mark.parametrize("with_apply", [True, False], ids=["apply", "compress_only"])
@pytest.mark.parametrize("value_mode", [B.GD_VALUES_FP32, B.GD_VALUES_TWO_MEANS], ids=["fp32", "two_means"])
def test_step_host_matches_oracle(cuda_device, value_mode, with_apply):
    """Two steps through gd_step_host, residual carried: the push as it arrives in host memory, the residual
    and the applied parameters equal the oracle's (bit for bit; means and parameters within 1e-6)."""
    w = _layout(value_mode)
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, 0, cuda_device)
    k = sess.k_total
    two = value_mode == B.GD_VALUES_TWO_MEANS
    params = torch.randn(w.n, device=cuda_device) * 0.01
    views = sess.shard_views(params)
    g_dev = torch.empty(w.n, dtype=torch.float32, device=cuda_device)        # the device buffer the step copies into
    g_host = torch.empty(w.n, dtype=torch.float32).pin_memory()
    idx_host = torch.zeros(k, dtype=torch.int32).pin_memory()
    val_host = torch.zeros(k, dtype=torch.float32).pin_memory()
    off_host = torch.zeros(w.n_shards + 1, dtype=torch.int32).pin_memory()
    means_host = torch.zeros(len(w.layer_off) - 1, 2, dtype=torch.float32).pin_memory()
    call = sess.compress_call(g_dev)
    acall = sess.apply_call(views) if with_apply else None
    gen = torch.Generator().manual_seed(11)
    r_host = orc.residual_reset(w.n)
    for step in range(2):
        g_host.copy_(torch.randn(w.n, generator=gen) * 1e-3)
        exp = orc.compress(g_host.numpy(), r_host, w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode)
        p_before = params.cpu().numpy().copy()
        B.gd_step_host(call, acall, g_host, idx_host, None if two else val_host, off_host, means_host if two else None)
        # gd_step_host has synchronised the stream: the host buffers are final
        tag = f"step {step}"
        assert np.array_equal(idx_host.numpy().view(np.uint32), exp["idx"]), f"{tag}: positions on the host"
        assert np.array_equal(off_host.numpy().view(np.uint32), exp["shard_cnt_off"]), f"{tag}: shard offsets on the host"
        if two:
            ref = np.where(exp["counts"] > 0, exp["sums"] / np.maximum(exp["counts"], 1), 0.0)
            got = means_host.numpy().astype(np.float64)
            assert np.all(np.abs(got - ref) <= REL_TOL * np.abs(ref)), f"{tag}: means on the host"
        else:
            assert np.array_equal(val_host.numpy().view(np.uint32), exp["val"].view(np.uint32)), f"{tag}: values on the host"
        assert np.array_equal(g_dev.cpu().numpy().view(np.uint32), g_host.numpy().view(np.uint32)), f"{tag}: gradient copy"
        assert np.array_equal(sess.residual.cpu().numpy().view(np.uint32), exp["residual"].view(np.uint32)), f"{tag}: residual"
        assert np.array_equal(sess.out_tau.cpu().numpy().view(np.uint32), exp["tau"]), f"{tag}: thresholds"
        got_p = params.cpu().numpy()
        if with_apply:
            push = {"idx": exp["idx"], "val": exp.get("val"), "means": exp.get("means")}
            for j in range(w.n_shards):
                lo, hi = w.shard_off[j], w.shard_off[j + 1]
                ref_p, bound = orc.apply_pushes(p_before[lo:hi], lo, [push], value_mode=value_mode, layer_off=w.layer_off)
                assert np.all(np.abs(got_p[lo:hi].astype(np.float64) - ref_p) <= REL_TOL * bound + 1e-45), f"{tag}: shard {j}"
        else:
            assert np.array_equal(got_p.view(np.uint32), p_before.view(np.uint32)), f"{tag}: parameters touched"
        r_host = exp["residual"]
    assert sess.stats()["n_scopes_predicted"] >= 2


def test_step_host_rejects_missing_gradient(cuda_device):
    w = _layout(B.GD_VALUES_FP32)
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, 0, cuda_device)
    call = sess.compress_call(torch.zeros(w.n, device=cuda_device))
    with pytest.raises(B.GdError) as err:
        B.gd_step_host(call, None, None)
    assert err.value.code == B.GD_ERR_INVALID_ARG


def _one_step(sess, g, views):
    sess.compress(g)
    sess.apply(views)
    torch.cuda.synchronize()
    assert sess.status() == B.GD_OK


@pytest.mark.parametrize("path", ["predicted", "dense", "dense_short_vector"])
def test_profile_pairs_and_launch_count(cuda_device, path):
    """Every kernel of a step is one launch and, with the hooks on, one tagged event pair, in launch order."""
    w = _layout(B.GD_VALUES_FP32)
    if path == "dense_short_vector":                             # what one launch of the dense kernel holds
        w = W.small_layered(4, [700_000, 13, 300_003, 4096], 990_000, B.GD_SCOPE_PER_LAYER, B.GD_VALUES_FP32, 3)
    flags = B.GD_FLAG_NO_PREDICTION if path == "dense" else 0
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, flags, cuda_device)
    params = torch.zeros(w.n, device=cuda_device)
    views = sess.shard_views(params)
    g = torch.randn(w.n, device=cuda_device) * 1e-3
    _one_step(sess, g, views)                                    # warm-up: caches, event pool
    expected = B.STEP_KERNELS[path] + ["apply"]

    B.gd_profile_enable(0)
    B.gd_profile_collect()
    before = B.gd_launch_count()
    _one_step(sess, g, views)
    assert B.gd_launch_count() - before == len(expected)
    assert B.gd_profile_collect() == []                          # hooks off: nothing recorded

    B.gd_profile_enable(2)                                       # every kernel
    try:
        before = B.gd_launch_count()
        _one_step(sess, g, views)
        _one_step(sess, g, views)
        assert B.gd_launch_count() - before == 2 * len(expected)
        pairs = B.gd_profile_collect(with_tags=True)
        assert [t for t, _ in pairs] == expected * 2
        assert all(0.0 < ms < 1e3 for _, ms in pairs)
        assert B.gd_profile_collect() == []                      # a collect forgets what it returned

        B.gd_profile_enable(1)                                   # the fused full pass only
        _one_step(sess, g, views)
        pairs = B.gd_profile_collect(with_tags=True)
        assert [t for t, _ in pairs] == ["dense_fused" if path == "dense_short_vector" else "add_emit"]
        # the fused pass streams 12 bytes per element: its duration must be consistent with the device
        assert pairs[0][1] > 12.0 * w.n / 20e12 * 1e3            # not faster than 20 TB/s
    finally:
        B.gd_profile_enable(0)
    _one_step(sess, g, views)
    assert B.gd_profile_collect() == []


def test_profile_enable_rejects_unknown_modes(cuda_device):
    with pytest.raises(B.GdError):
        B.gd_profile_enable(3)
    with pytest.raises(B.GdError):
        B.gd_profile_enable(-1)


def test_apply_with_two_alphas_in_one_session(cuda_device):
    """Section 3's server update with two step sizes in a row on one session: each call uses its own alpha."""
    w = _layout(B.GD_VALUES_FP32)
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, 0, cuda_device)
    g = torch.randn(w.n, device=cuda_device) * 1e-3
    sess.compress(g)
    exp = orc.compress(g.cpu().numpy(), orc.residual_reset(w.n), w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode)
    params = torch.zeros(w.n, device=cuda_device)
    views = sess.shard_views(params)
    sess.apply(views)                 # alpha = 1
    sess.apply(views, 0.5)
    sess.apply(views, -2.0)
    torch.cuda.synchronize()
    push = {"idx": exp["idx"], "val": exp["val"]}
    got = params.cpu().numpy().astype(np.float64)
    ref, bound = np.zeros(w.n), np.zeros(w.n)
    for alpha in (1.0, 0.5, -2.0):                       # the oracle's fp64 sum, one push per step size
        r, b = orc.apply_pushes(np.zeros(w.n, np.float32), 0, [push], alpha=alpha)
        ref += r
        bound += b
    assert np.all(np.abs(got - ref) <= REL_TOL * bound + 1e-45)
    assert np.count_nonzero(got) == np.count_nonzero(ref)


def test_per_step_metrics_log(cuda_device, tmp_path):
    """One JSON line per step: status, counters, survivors per shard (they add up to k), threshold keys."""
    import json
    w = _layout(B.GD_VALUES_FP32)
    sess = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, 0, cuda_device)
    path = tmp_path / "steps.jsonl"
    with open(path, "w") as fh:
        for step in range(3):
            sess.compress(torch.randn(w.n, device=cuda_device) * 1e-3)
            sess.log_step(fh, step, note="test")
    recs = [json.loads(line) for line in open(path)]
    assert [r["step"] for r in recs] == [0, 1, 2]
    for r in recs:
        assert r["status"] == B.GD_OK and r["n_kept"] == sess.k_total and sum(r["kept_per_shard"]) == sess.k_total
        assert r["n_scopes"] == len(w.layer_off) - 1 and len(r["tau_keys"]) == r["n_scopes"] and r["note"] == "test"
