"""gd_compress_static: the entry point for callers that cannot allocate a workspace.

A runtime that fixed its device-memory plan before the first step (or a plug-in that is not
allowed to call cudaMalloc) still owns its gradient, residual and output buffers, but has no
scratch buffer to lend.  gd_compress_static runs the same compression on a scratch area built
into the library.  This test drives it through the C ABI and requires the same bytes as
gd_compress with a caller-owned workspace, on two calls in a row (the second call finds the
scratch area as the first one left it, and carries the residual of the first).

Collected last on purpose (file name), so that a failure here cannot hide another test's result.
"""
import pytest
import torch

from paper_1704_05021_b200 import binding as B
from paper_1704_05021_b200 import workloads as W
from paper_1704_05021_b200.session import GradDropSession

pytestmark = pytest.mark.gpu


def _bits(t):
    return t.view(torch.int32)


@pytest.mark.parametrize("value_mode", [B.GD_VALUES_FP32, B.GD_VALUES_TWO_MEANS])
def test_static_scratch_matches_caller_workspace(cuda_device, value_mode):
    sizes = [300_000, 17, 0, 150_001, 4096]
    w = W.small_layered(len(sizes), sizes, 990_000, B.GD_SCOPE_PER_LAYER, value_mode, 3)
    assert B.gd_workspace_bytes(w.layer_off, w.n_shards, w.scope_mode, w.drop_ppm) <= B.GD_STATIC_WORKSPACE_BYTES
    ref = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, 0, cuda_device)
    sta = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, 0, cuda_device)
    gen = torch.Generator(device=cuda_device).manual_seed(77)
    for call_no in range(2):
        g = torch.randn(w.n, generator=gen, device=cuda_device) * 1e-3
        ref.compress(g)
        call = sta.compress_call(g)
        call.args.workspace = None          # the caller has no workspace to give
        call.args.workspace_bytes = 0
        scratch = B.gd_compress_static(call)
        assert scratch != 0
        assert B.gd_status_at(scratch) == B.GD_OK and ref.status() == B.GD_OK
        k = ref.k_total
        assert torch.equal(_bits(sta.out_idx[:k]), _bits(ref.out_idx[:k])), f"call {call_no}: indices"
        assert torch.equal(_bits(sta.residual), _bits(ref.residual)), f"call {call_no}: residual"
        assert torch.equal(sta.out_tau, ref.out_tau), f"call {call_no}: thresholds"
        assert torch.equal(sta.out_shard_cnt_off, ref.out_shard_cnt_off), f"call {call_no}: shard offsets"
        if value_mode == B.GD_VALUES_FP32:
            assert torch.equal(_bits(sta.out_val[:k]), _bits(ref.out_val[:k])), f"call {call_no}: values"
        else:   # the two means: same tolerance as the parity tests (1e-6 relative)
            a, b = sta.out_means.double(), ref.out_means.double()
            assert bool(((a - b).abs() <= 1e-6 * b.abs()).all()), f"call {call_no}: means"


@pytest.mark.parametrize("flags", [0, B.GD_FLAG_SAMPLED_THRESHOLD], ids=["exact", "sampled_threshold"])
def test_static_scratch_on_the_predicted_path(cuda_device, flags):
    """A gradient long enough for the path that predicts the threshold from a sample (so that the sample, the
    candidate lists and the kernels that work on them all run on the built-in scratch), and one call with the
    threshold taken on a sample; two calls in a row each, same bytes as with a caller-owned workspace."""
    w = W.workload(5, scale_log2=23)               # 2^23 elements, 99.9 %, 8 shards: about 3 MiB of scratch
    assert B.gd_workspace_bytes(w.layer_off, w.n_shards, w.scope_mode, w.drop_ppm) <= B.GD_STATIC_WORKSPACE_BYTES
    ref = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, flags, cuda_device)
    sta = GradDropSession(w.layer_off, w.shard_off, w.drop_ppm, w.scope_mode, w.value_mode, flags, cuda_device)
    for call_no in range(2):
        g = W.make_gradient(w, call_no, cuda_device)
        ref.compress(g)
        call = sta.compress_call(g)
        call.args.workspace = None
        call.args.workspace_bytes = 0
        scratch = B.gd_compress_static(call)
        st = B.gd_get_stats_at(scratch)
        assert st["status"] == B.GD_OK and ref.status() == B.GD_OK
        assert st["n_scopes_predicted"] == 1 and st["n_scopes_dense"] == 0, st
        k = ref.kept()
        assert int(sta.out_shard_cnt_off[-1]) == k if flags else True
        assert torch.equal(_bits(sta.out_idx[:k]), _bits(ref.out_idx[:k])), f"call {call_no}: indices"
        assert torch.equal(_bits(sta.out_val[:k]), _bits(ref.out_val[:k])), f"call {call_no}: values"
        assert torch.equal(_bits(sta.residual), _bits(ref.residual)), f"call {call_no}: residual"
        assert torch.equal(sta.out_tau, ref.out_tau), f"call {call_no}: thresholds"
        assert torch.equal(sta.out_shard_cnt_off, ref.out_shard_cnt_off), f"call {call_no}: shard offsets"


def test_static_scratch_refuses_oversized_calls(cuda_device):
    w = W.workload(5)    # 2^30 elements: needs about twice the scratch the built-in area holds
    assert B.gd_workspace_bytes(w.layer_off, w.n_shards, w.scope_mode, w.drop_ppm) > B.GD_STATIC_WORKSPACE_BYTES
    a = B._CompressArgs()
    lo = B._u64_array(w.layer_off)
    so = B._u64_array(w.shard_off)
    a.layer_off, a.n_layers, a.shard_off, a.n_shards, a.n = lo, 1, so, w.n_shards, w.n
    a.drop_ppm, a.scope_mode = w.drop_ppm, w.scope_mode
    import ctypes as C
    assert B.load_library().gd_compress_static(C.byref(a), None, None) == B.GD_ERR_TOO_LARGE
