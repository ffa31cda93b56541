"""CPU oracle for the gradient-dropping hot path (Aji & Heafield 2017, Section 4, Algorithm 1).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the CUDA library is
checked against.  It shares no code with the CUDA path, imports nothing from the product
package, and may be imported only by tests, by the smoke check and by the benchmark's
cpu-baseline leg.  Every function is pinned by tests that do not go through this module's own
formulas (brute-force rank counts, closed forms, library selection routines, the payload ratios
the paper prints); no function here is "parity unpinned".

What the path computes (Algorithm 1, in its order):

  1. grad += residuals                      (fp32 add, round to nearest even)
  2. choose the threshold below which a fraction R of the |grad| values lies  (one threshold on |value|, Section 4 par. 1)
  3. kept[i] = grad[i] where |grad[i]| is above the threshold, else 0
  4. residuals = grad - kept                 (the dropped mass stays local)
  5. return sparse(kept)                     (index + value pairs, 8 bytes per survivor;
                                              the factor 50 at 99 % in Section 5.1)

Readings taken where the paper is silent:
  * exactly k = n - floor(n * drop_ppm / 1e6) entries are kept per threshold scope; the
    order used is (|v| bit pattern descending, index ascending), so ties at the cut go to
    the lower index; the reported threshold tau is the smallest kept |v| bit pattern
    (0xFFFFFFFF when nothing is kept);
  * a scope is either the whole gradient ("global") or each parameter tensor on its own
    (the per-matrix thresholds of Section 4, last paragraph);
  * two-value quantisation (Section 5.4, centres = the means of the values they replace): one pair
    (mean of kept entries with sign bit 0, mean of kept entries with sign bit 1) per layer,
    survivors packed as index | signbit << 31; the residual still holds only the dropped mass;
  * column-wise averages (Section 5.4: centres chosen per column rather than per tensor):
    a layer is a row-major matrix with layer_cols[l] columns and every column has its own pair;
  * threshold quantisation (Section 5.4: every surviving value is mapped to the dropping
    threshold, i.e. the smallest magnitude that survived): same packing; the pair of a
    layer is (+t, -t) with t the float whose bit pattern is the tau of the scope holding the layer;
  * the server applies a push as p[idx - shard_start] += alpha * value (Section 3: a server
    owns 1/N of the parameters); this oracle evaluates that sum in fp64.
"""
from __future__ import annotations

import numpy as np

SCOPE_GLOBAL = 0
SCOPE_PER_LAYER = 1
VALUES_FP32 = 0
VALUES_TWO_MEANS = 1
VALUES_THRESHOLD = 2
VALUES_COLUMN_MEANS = 3

_ABS_MASK = np.uint32(0x7FFFFFFF)
TAU_NONE = 0xFFFFFFFF


def kept_count(n: int, drop_ppm: int) -> int:
    """Entries kept out of n when drop_ppm parts per million are dropped (Algorithm 1, step 2).

    dropped = floor(n * drop_ppm / 1e6), kept = the rest; Python integers, so no rounding.
    """
    if n < 0 or not (0 <= drop_ppm <= 1_000_000):
        raise ValueError("bad n or drop_ppm")
    return n - (n * drop_ppm) // 1_000_000


def scopes_of(layer_off, scope_mode: int):
    """Index ranges over which one threshold is selected (Section 4, last paragraph)."""
    layer_off = [int(x) for x in layer_off]
    if scope_mode == SCOPE_GLOBAL:
        return [(layer_off[0], layer_off[-1])]
    if scope_mode == SCOPE_PER_LAYER:
        return [(layer_off[i], layer_off[i + 1]) for i in range(len(layer_off) - 1)]
    raise ValueError("bad scope_mode")


def magnitude_keys(v: np.ndarray) -> np.ndarray:
    """|v| as the unsigned integer whose order equals the order of |v| for finite floats."""
    assert v.dtype == np.float32
    return v.view(np.uint32) & _ABS_MASK


def _kept_in_scope(keys: np.ndarray, k: int, method: str):
    """Indices (local, ascending) of the k largest keys, ties to the lower index, and tau.

    The order is made strict by the composite  key << 32 | (0xFFFFFFFF - index): a larger
    composite means larger |v|, or equal |v| and a lower index.  "sort" sorts all composites;
    "select" uses a partial selection of the same composites (the k-th element of a strict
    total order is unique, so both give the same set).
    """
    n = keys.shape[0]
    if k == 0:
        return np.empty(0, dtype=np.int64), TAU_NONE
    comp = (keys.astype(np.uint64) << np.uint64(32)) | (
        np.uint64(0xFFFFFFFF) - np.arange(n, dtype=np.uint64))
    if method == "sort":
        top = np.sort(comp)[n - k:]
    elif method == "select":
        top = np.partition(comp, n - k)[n - k:]
    else:
        raise ValueError("bad method")
    tau = int(top.min() >> np.uint64(32))
    local = (np.uint64(0xFFFFFFFF) - (top & np.uint64(0xFFFFFFFF))).astype(np.int64)
    local.sort()
    return local, tau


def _mix32(x: np.ndarray) -> np.ndarray:
    """A fixed 32-bit integer mix (the position hash of the sampled-threshold mode), in uint32 arithmetic."""
    x = x.astype(np.uint32)
    x = x ^ (x >> np.uint32(16))
    x = (x * np.uint32(0x7FEB352D)).astype(np.uint32)
    x = x ^ (x >> np.uint32(15))
    x = (x * np.uint32(0x846CA68B)).astype(np.uint32)
    x = x ^ (x >> np.uint32(16))
    return x


def sampled_positions(lo: int, hi: int, scope_index: int) -> np.ndarray:
    """Positions read by the sampled-threshold mode in scope [lo, hi) (Section 4, fourth paragraph: a 0.1 % sample).

    Scopes of up to 4096 elements are sampled completely.  Longer ones are sampled in pairs of neighbours
    (both reads of a pair fall into one 32-byte sector of memory): m = max(4096, ceil(n_s / 1000)) rounded up
    to an even number; the pairs are (first + 2 j, first + 2 j + 1) with first = the smallest even index
    >= lo and j < P = floor((hi - first) / 2); the P pairs are cut into m / 2 strata, the first (P mod m/2)
    of floor(P / (m/2)) + 1 pairs and the rest of floor(P / (m/2)), and stratum i contributes the pair
    start_i + (mix32(i * 0x9E3779B9 + scope_index) mod width_i).  The rule is part of this mode's
    definition, which is why the CUDA library restates it; nothing else is shared.
    """
    ns = hi - lo
    if ns <= 4096:
        return np.arange(lo, hi, dtype=np.int64)
    m = max(4096, -(-ns // 1000))
    m += m & 1
    first = lo + (lo & 1)
    pairs, strata = (hi - first) // 2, m // 2
    w, rem = pairs // strata, pairs % strata
    i = np.arange(strata, dtype=np.uint64)
    a = i * np.uint64(w) + np.minimum(i, np.uint64(rem))
    width = np.uint64(w) + (i < np.uint64(rem)).astype(np.uint64)
    with np.errstate(over="ignore"):
        h = _mix32((i.astype(np.uint32) * np.uint32(0x9E3779B9) + np.uint32(scope_index)).astype(np.uint32))
    off = np.where(width > 1, h.astype(np.uint64) % np.maximum(width, np.uint64(1)), np.uint64(0))
    even = np.uint64(first) + np.uint64(2) * (a + off)
    return np.stack([even, even + np.uint64(1)], axis=1).reshape(-1).astype(np.int64)


def compress_sampled(grad, residual, layer_off, shard_off, drop_ppm, scope_mode=SCOPE_GLOBAL):
    """GradDrop with the threshold selected on a sample (Section 4, fourth paragraph).

    Per scope: the threshold key t is the k_m-th largest key among the sampled entries,
    k_m = m - floor(m * drop_ppm / 1e6), and every entry of the scope with key >= t is kept
    (nothing if k_m = 0).  The number of survivors therefore varies from call to call.
    """
    g = np.ascontiguousarray(grad, dtype=np.float32)
    r = np.ascontiguousarray(residual, dtype=np.float32)
    n = g.shape[0]
    v = g + r
    keys = magnitude_keys(v)
    kept_parts, taus = [], []
    for si, (lo, hi) in enumerate(scopes_of(layer_off, scope_mode)):
        pos = sampled_positions(lo, hi, si)
        m = pos.shape[0]
        k_m = kept_count(m, drop_ppm)
        if k_m == 0:
            taus.append(TAU_NONE)
            continue
        t = np.sort(keys[pos])[m - k_m]                      # the k_m-th largest sample key
        taus.append(int(t))
        kept_parts.append(lo + np.flatnonzero(keys[lo:hi] >= t))
    kept = np.concatenate(kept_parts).astype(np.int64) if kept_parts else np.empty(0, dtype=np.int64)
    new_residual = v.copy()
    new_residual[kept] = np.float32(0.0)
    return {
        "idx": kept.astype(np.uint32),
        "val": v[kept],
        "residual": new_residual,
        "tau": np.asarray(taus, dtype=np.uint32),
        "shard_cnt_off": np.searchsorted(kept, np.asarray([int(x) for x in shard_off], dtype=np.int64),
                                         side="left").astype(np.uint32),
        "v": v,
    }


def compress_delta(params, last_pulled, layer_off, shard_off, drop_ppm, scope_mode=SCOPE_GLOBAL, method="sort"):
    """GradDrop applied to a parameter pull (Section 4, third paragraph).

    The server keeps `last_pulled`, the copy the client is known to hold, and sends the dropped
    delta  v = params - last_pulled  (one fp32 subtraction per element).  Whatever is sent is added
    to last_pulled with one fp32 add, which is exactly what the client does to its own copy, so the
    two stay equal; what is dropped stays inside the next delta, so no separate residual is read.
    Returns the dict of compress() (its "residual" is v where dropped, +0 where kept) plus
    "last_pulled", the updated copy.
    """
    p = np.ascontiguousarray(params, dtype=np.float32)
    last = np.ascontiguousarray(last_pulled, dtype=np.float32)
    v = p - last
    out = compress(v, np.full_like(v, -0.0), layer_off, shard_off, drop_ppm, scope_mode, VALUES_FP32, method)
    # (v + -0.0 is v bit for bit, so compress() selects on v itself)
    new_last = last.copy()
    kept = out["idx"].astype(np.int64)
    new_last[kept] = last[kept] + out["val"]
    out["last_pulled"] = new_last
    return out


def pair_index(pos, layer_off, layer_cols=None):
    """The (mean+, mean-) pair each position belongs to: its layer, or its layer and column."""
    lo = np.asarray([int(x) for x in layer_off], dtype=np.int64)
    n_layers = lo.shape[0] - 1
    cols = np.ones(n_layers, dtype=np.int64) if layer_cols is None else np.asarray(layer_cols, dtype=np.int64)
    pair_off = np.concatenate([[0], np.cumsum(cols)])
    pos = np.asarray(pos, dtype=np.int64)
    layer = np.searchsorted(lo, pos, side="right") - 1
    return pair_off[layer] + (pos - lo[layer]) % cols[layer], int(pair_off[-1])


def compress(grad, residual, layer_off, shard_off, drop_ppm, scope_mode=SCOPE_GLOBAL,
             value_mode=VALUES_FP32, method="sort", layer_cols=None, error_feedback=False):
    """One GradDrop call (Algorithm 1) for one worker's flat fp32 gradient.

    grad, residual : float32 arrays of n elements (not modified).
    layer_off      : n_layers + 1 ascending offsets, first 0, last n.
    shard_off      : n_shards + 1 ascending offsets, first 0, last n (Section 3's 1/N pieces).
    Returns a dict with
      idx       uint32[k_total]  survivor positions, ascending (two-means: idx | sign << 31)
      val       float32[k_total] survivor values, bit-for-bit v[idx]  (fp32 mode)
      residual  float32[n]       v where dropped, +0.0 where kept
      tau       uint32[n_scopes] smallest kept |v| bit pattern per scope (0xFFFFFFFF: none kept)
      shard_cnt_off uint32[n_shards+1] survivors with index below each shard boundary
      means     float32[n_layers, 2], counts int64[n_layers, 2], sums float64[n_layers, 2]
                (two-means mode; column 0 = sign bit clear, column 1 = sign bit set)
    error_feedback (1-bit value modes only): the paper is silent on whether the error of the 1-bit
    quantisation stays local; Algorithm 1 keeps the dropped mass only (the default).  With the option
    a kept entry leaves v minus its decoded fp32 value in the residual (one fp32 subtraction), the
    error feedback of 1-bit SGD that Section 2 describes.
    """
    g = np.ascontiguousarray(grad, dtype=np.float32)
    r = np.ascontiguousarray(residual, dtype=np.float32)
    n = g.shape[0]
    assert r.shape[0] == n
    layer_off = [int(x) for x in layer_off]
    shard_off = [int(x) for x in shard_off]
    assert layer_off[0] == 0 and layer_off[-1] == n
    assert shard_off[0] == 0 and shard_off[-1] == n

    v = g + r                                   # step 1: one IEEE binary32 add per element
    keys = magnitude_keys(v)

    kept_parts, taus = [], []
    for lo, hi in scopes_of(layer_off, scope_mode):
        k = kept_count(hi - lo, drop_ppm)       # step 2
        local, tau = _kept_in_scope(keys[lo:hi], k, method)
        kept_parts.append(local + lo)
        taus.append(tau)
    kept = np.concatenate(kept_parts) if kept_parts else np.empty(0, dtype=np.int64)

    new_residual = v.copy()                     # step 4: residuals = grad - kept
    new_residual[kept] = np.float32(0.0)
    val = v[kept]                               # step 3/5: the values that travel

    shard_cnt_off = np.searchsorted(kept, np.asarray(shard_off, dtype=np.int64),
                                    side="left").astype(np.uint32)
    out = {
        "idx": kept.astype(np.uint32),
        "val": val,
        "residual": new_residual,
        "tau": np.asarray(taus, dtype=np.uint32),
        "shard_cnt_off": shard_cnt_off,
        "v": v,
    }
    if value_mode in (VALUES_TWO_MEANS, VALUES_COLUMN_MEANS):
        if n > (1 << 31):
            raise ValueError("packed indices need n <= 2^31")
        if value_mode == VALUES_COLUMN_MEANS:
            assert layer_cols is not None
            for l in range(len(layer_off) - 1):
                assert layer_cols[l] >= 1 and (layer_off[l + 1] - layer_off[l]) % layer_cols[l] == 0
        pair, n_pairs = pair_index(kept, layer_off, layer_cols if value_mode == VALUES_COLUMN_MEANS else None)
        sums = np.zeros((n_pairs, 2), dtype=np.float64)
        cnts = np.zeros((n_pairs, 2), dtype=np.int64)
        sign = (val.view(np.uint32) >> np.uint32(31)).astype(np.int64)
        # unbuffered accumulation: one fp64 add per survivor, in ascending index order
        np.add.at(sums, (pair, sign), val.astype(np.float64))
        np.add.at(cnts, (pair, sign), 1)
        with np.errstate(invalid="ignore", divide="ignore"):
            means = np.where(cnts > 0, sums / np.maximum(cnts, 1), 0.0).astype(np.float32)
        out["idx"] = (kept.astype(np.uint32) | (sign.astype(np.uint32) << np.uint32(31)))
        out["means"], out["counts"], out["sums"] = means, cnts, sums
    elif value_mode == VALUES_THRESHOLD:
        if n > (1 << 31):
            raise ValueError("threshold packing needs n <= 2^31")
        n_layers = len(layer_off) - 1
        sign = (val.view(np.uint32) >> np.uint32(31))
        means = np.zeros((n_layers, 2), dtype=np.float32)
        for l in range(n_layers):
            tau = taus[0] if scope_mode == SCOPE_GLOBAL else taus[l]
            bits = np.uint32(0 if tau == TAU_NONE else tau)
            means[l, 0] = bits.view(np.float32)                       # +t: the smallest kept |v| of the scope
            means[l, 1] = (bits | np.uint32(0x80000000)).view(np.float32)
        out["idx"] = kept.astype(np.uint32) | (sign << np.uint32(31))
        out["means"] = means
    elif value_mode != VALUES_FP32:
        raise ValueError("bad value_mode")
    if error_feedback:
        if value_mode == VALUES_FP32:
            raise ValueError("error feedback needs a 1-bit value mode")
        _, decoded = decode_push(out["idx"], None, value_mode, out["means"], layer_off, layer_cols)
        new_residual[kept] = val - decoded          # fp32 - fp32, rounded once
    return out


def decode_push(push_idx, push_val, value_mode=VALUES_FP32, means=None, layer_off=None, layer_cols=None):
    """Positions and fp32 values a push stands for (the server-side decompress)."""
    idx = np.asarray(push_idx, dtype=np.uint32)
    if value_mode == VALUES_FP32:
        return idx.astype(np.int64), np.asarray(push_val, dtype=np.float32)
    pos = (idx & _ABS_MASK).astype(np.int64)
    sign = (idx >> np.uint32(31)).astype(np.int64)
    pair, _ = pair_index(pos, layer_off, layer_cols if value_mode == VALUES_COLUMN_MEANS else None)
    return pos, np.asarray(means, dtype=np.float32)[pair, sign]


def apply_pushes(params, shard_start, pushes, alpha=1.0, value_mode=VALUES_FP32, layer_off=None, layer_cols=None):
    """fp64 reference of the server-side scatter-add into one parameter shard (Section 3).

    params  : float32[shard_len], the shard's parameters before the pushes.
    pushes  : list of dicts with "idx" (+ "val", or "means" in two-means mode); only entries
              whose position falls in [shard_start, shard_start + shard_len) are applied.
    Returns (ref, bound): ref = p0 + sum alpha * value in fp64, and bound = |p0| + sum
    |alpha * value| (the magnitude the 1e-6 relative tolerance is taken against).
    """
    p0 = np.asarray(params, dtype=np.float32)
    ref = p0.astype(np.float64)
    bound = np.abs(ref)
    a = float(np.float32(alpha))
    lo, hi = int(shard_start), int(shard_start) + p0.shape[0]
    for push in pushes:
        pos, val = decode_push(push["idx"], push.get("val"), value_mode, push.get("means"),
                               layer_off, layer_cols)
        m = (pos >= lo) & (pos < hi)
        contrib = a * val[m].astype(np.float64)
        np.add.at(ref, pos[m] - lo, contrib)
        np.add.at(bound, pos[m] - lo, np.abs(contrib))
    return ref, bound


def residual_reset(n: int) -> np.ndarray:
    """The state before the first call: nothing has been dropped yet (Section 4, par. 2)."""
    return np.zeros(n, dtype=np.float32)
