"""Host-side checks of libgd.so that need no GPU: exports, sizing helpers, argument validation."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import graddrop_oracle as orc
from paper_1704_05021_b200 import binding as B
from paper_1704_05021_b200 import build as gd_build
from paper_1704_05021_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    gd_build.build_library()
    return B.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "gd.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(gd_[a-z_]+)\s*\(", header))
    assert declared == set(B.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_status_strings(lib):
    for code in range(-6, 1):
        assert B.status_string(code) not in ("", "unknown status")
    assert B.status_string(-99) == "unknown status"


def test_kept_counts_match_oracle(lib):
    rng = np.random.default_rng(0)
    for _ in range(200):
        n = int(rng.integers(0, 1 << 32))
        ppm = int(rng.integers(0, 1_000_001))
        assert B.gd_kept_count(n, ppm) == orc.kept_count(n, ppm)
    assert B.gd_kept_count(1 << 30, 999_000) == 1_073_742
    with pytest.raises(B.GdError):
        B.gd_kept_count(10, 1_000_001)
    with pytest.raises(B.GdError):
        B.gd_kept_count((1 << 32) + 1, 5)


def test_total_kept_on_the_five_workloads(lib):
    want = {1: 10_486, 2: 200_377, 3: 1_375_850, 4: 1_375_850, 5: 1_073_742}
    for cfg, k in want.items():
        w = W.workload(cfg)
        assert B.gd_total_kept(w.layer_off, w.scope_mode, w.drop_ppm) == k
        scopes = orc.scopes_of(w.layer_off, w.scope_mode)
        assert sum(orc.kept_count(hi - lo, w.drop_ppm) for lo, hi in scopes) == k
    w = W.workload(2, scope_mode=B.GD_SCOPE_PER_LAYER)
    assert B.gd_total_kept(w.layer_off, w.scope_mode, w.drop_ppm) == 200_379


def test_workspace_sizes_are_modest(lib):
    for cfg in (1, 2, 3, 5):
        w = W.workload(cfg)
        b = B.gd_workspace_bytes(w.layer_off, w.n_shards, w.scope_mode, w.drop_ppm)
        assert 0 < b < 0.25 * 4 * w.n + (1 << 20)
    assert B.gd_apply_workspace_bytes(8, 12) >= 8 * 8 + 9 * 8 + 13 * 8


def test_bad_arguments_are_rejected_on_the_host(lib):
    with pytest.raises(B.GdError) as e:
        B.gd_total_kept([0, 5, 3], B.GD_SCOPE_GLOBAL, 990_000)          # offsets not ascending
    assert e.value.code == B.GD_ERR_INVALID_ARG
    with pytest.raises(B.GdError):
        B.gd_total_kept([1, 5], B.GD_SCOPE_GLOBAL, 990_000)             # first offset not 0
    with pytest.raises(B.GdError):
        B.gd_total_kept([0, 5], 7, 990_000)                             # bad scope mode
    with pytest.raises(B.GdError) as e:
        B.gd_workspace_bytes([0, (1 << 32) + 4], 1, B.GD_SCOPE_GLOBAL, 990_000)
    assert e.value.code == B.GD_ERR_TOO_LARGE
    # gd_compress validates before touching CUDA: NULL buffers, missing workspace
    a = B._CompressArgs()
    assert lib.gd_compress(None, None) == B.GD_ERR_INVALID_ARG
    lo = (C.c_uint64 * 2)(0, 100)
    a.layer_off, a.n_layers, a.shard_off, a.n_shards, a.n, a.drop_ppm = lo, 1, lo, 1, 100, 990_000
    assert lib.gd_compress(C.byref(a), None) == B.GD_ERR_INVALID_ARG    # grad/residual NULL
    a.grad, a.residual = 0x1000, 0x2008
    assert lib.gd_compress(C.byref(a), None) == B.GD_ERR_INVALID_ARG    # residual not 16-byte aligned
    a.residual = 0x2000
    a.out_idx, a.out_val, a.out_shard_cnt_off = 0x3000, 0x4000, 0x5000
    assert lib.gd_compress(C.byref(a), None) == B.GD_ERR_WORKSPACE
    a.n = 99
    assert lib.gd_compress(C.byref(a), None) == B.GD_ERR_INVALID_ARG    # n disagrees with the offsets
    # the packed 1-bit value modes address 31 index bits; full 32-bit indices are for fp32 values only
    big = (1 << 31) + 16
    lo_big = (C.c_uint64 * 2)(0, big)
    a.layer_off, a.shard_off, a.n, a.out_means = lo_big, lo_big, big, 0x6000
    a.value_mode = B.GD_VALUES_TWO_MEANS
    assert lib.gd_compress(C.byref(a), None) == B.GD_ERR_TOO_LARGE
    a.value_mode = B.GD_VALUES_FP32
    assert lib.gd_compress(C.byref(a), None) == B.GD_ERR_WORKSPACE      # accepted as far as the (missing) workspace
    ap = B._ApplyArgs()
    assert lib.gd_decompress_apply(C.byref(ap), None) == B.GD_ERR_INVALID_ARG
    assert lib.gd_residual_reset(None, 5, None) == B.GD_ERR_INVALID_ARG
    assert lib.gd_residual_reset(None, 0, None) == B.GD_OK


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(gd_build, "LIB_PATH", str(tmp_path / "libgd.so"))
    with pytest.raises(RuntimeError):
        B.load_library()


def test_header_is_plain_c_and_links_from_c(lib, tmp_path):
    """include/gd.h compiles as C99 without CUDA headers, and a C program links against libgd.so and calls the
    host-only entry points (sizes, counts, status strings: nothing that needs a GPU)."""
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no C compiler here")
    src = tmp_path / "use_gd.c"
    src.write_text(r'''
#include <stdio.h>
#include "gd.h"
int main(void) {
  uint64_t k = 0, total = 0, cap = 0, pairs = 0;
  size_t ws = 0, aws = 0;
  const uint64_t layer_off[3] = {0, 1000000, 1048576};
  const uint32_t cols[2] = {1000, 1};
  gd_compress_args a;
  gd_apply_args b;
  gd_push p;
  (void)a; (void)b; (void)p;
  if (gd_kept_count(1048576, 990000, &k) != GD_OK || k != 10486) return 1;
  if (gd_total_kept(layer_off, 2, GD_SCOPE_PER_LAYER, 990000, &total) != GD_OK || total != 10000 + 486) return 2;
  if (gd_sampled_capacity(layer_off, 2, GD_SCOPE_GLOBAL, 990000, &cap) != GD_OK || cap < k) return 3;
  if (gd_means_pairs(2, cols, GD_VALUES_COLUMN_MEANS, &pairs) != GD_OK || pairs != 1001) return 4;
  if (gd_workspace_bytes(layer_off, 2, cols, 4, GD_SCOPE_PER_LAYER, 990000, &ws) != GD_OK || ws == 0) return 5;
  if (gd_apply_workspace_bytes(4, 2, &aws) != GD_OK || aws == 0) return 6;
  if (gd_compress(NULL, NULL) != GD_ERR_INVALID_ARG) return 7;
  printf("%s|%llu|%llu\n", gd_status_string(GD_ERR_WORKSPACE), (unsigned long long)k, (unsigned long long)total);
  return 0;
}
''')
    exe = tmp_path / "use_gd"
    libdir = os.path.dirname(gd_build.LIB_PATH)
    cmd = ["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"), str(src),
           "-L", libdir, "-l:libgd.so", "-Wl,-rpath," + libdir, "-o", str(exe)]
    res = subprocess.run(cmd, capture_output=True, text=True)
    assert res.returncode == 0, res.stderr
    out = subprocess.run([str(exe)], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0, (out.returncode, out.stderr)
    assert out.stdout.strip() == "workspace missing or too small|10486|10486"


def test_planner_under_address_and_undefined_behaviour_sanitizers(tmp_path):
    """The host-side planner (scopes, sample sizes, capacities, tile tables, workspace layout: offset arithmetic
    that runs on every call) built by itself with -fsanitize=address,undefined and driven over a few thousand
    layouts; the driver checks the invariants the kernels rely on."""
    import shutil
    import subprocess
    gxx = shutil.which("g++")
    if gxx is None:
        pytest.skip("no host compiler")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    exe = str(tmp_path / "plan_sanitize")
    build = subprocess.run([gxx, "-std=c++17", "-O1", "-g", "-fsanitize=address,undefined", "-fno-sanitize-recover=all",
                            "-I", os.path.join(root, "include"), "-I", os.path.join(root, "paper_1704_05021_b200", "csrc"),
                            os.path.join(root, "tests", "host", "plan_sanitize.cpp"), "-o", exe],
                           capture_output=True, text=True)
    if build.returncode != 0 and "sanitize" in build.stderr and "cannot find" in build.stderr:
        pytest.skip("the sanitizer run-time libraries are not installed")
    assert build.returncode == 0, build.stderr
    run = subprocess.run([exe], capture_output=True, text=True, env=dict(os.environ, ASAN_OPTIONS="detect_leaks=1"))
    assert run.returncode == 0, run.stdout + run.stderr
    assert run.stdout.startswith("ok ") and int(run.stdout.split()[1]) > 2000
