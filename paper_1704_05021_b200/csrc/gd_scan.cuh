// Single-pass decoupled look-back over the tiles of one scope, shared by the fused pass and the
// survivor compaction.  Internal to libgd.so.
#pragma once

#include "gd_internal.cuh"

namespace gd {

// One descriptor per tile: {flag:2 | count_a:62, count_b:64}, written and read as one 128-bit
// access so that the flag and both counts are always seen together.
__device__ __forceinline__ void st_desc(uint4* p, uint64_t lo, uint64_t hi) {
  asm volatile("{\n\t.reg .b128 t;\n\tmov.b128 t, {%1, %2};\n\tst.relaxed.gpu.global.b128 [%0], t;\n\t}"
               ::"l"(p), "l"(lo), "l"(hi) : "memory");
}
__device__ __forceinline__ void ld_desc(const uint4* p, uint64_t& lo, uint64_t& hi) {
  asm volatile("{\n\t.reg .b128 t;\n\tld.relaxed.gpu.global.b128 t, [%2];\n\tmov.b128 {%0, %1}, t;\n\t}"
               : "=l"(lo), "=l"(hi) : "l"(p) : "memory");
}

__device__ __forceinline__ uint64_t warp_sum(uint64_t x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
  return x;
}

// Run by one full warp.  Publishes this tile's totals (unless `published`: see tile_publish), waits (bounded) for
// the tiles [first, t) of the same scope and returns their sums.  Tile ids come from an atomic ticket, so every tile waited
// on has already started.  A wait gives up after spin_limit polls and budget_ns of time (whichever
// comes later; budget_ns = 0: the polls alone).  A wait that runs out marks the tile aborted, records
// GD_ERR_DEVICE_TIMEOUT and returns false; a tile that meets an aborted predecessor aborts too, so
// nothing waits on a tile that gave up.
__device__ __forceinline__ bool tile_lookback(uint4* desc, uint32_t t, uint32_t first, uint64_t tot_a, uint64_t tot_b,
                                              uint64_t& ex_a, uint64_t& ex_b, Ctl* ctl,
                                              uint32_t spin_limit = kLookbackSpinLimit, uint64_t budget_ns = kWaitBudgetNs,
                                              bool published = false) {
  const uint32_t lane = lane_id();
  ex_a = 0;
  ex_b = 0;
  if (t == first) {
    if (lane == 0 && !published) st_desc(desc + t, pack_desc(F_PREFIX, tot_a), tot_b);
    return true;
  }
  if (lane == 0 && !published) st_desc(desc + t, pack_desc(F_AGG, tot_a), tot_b);
  bool ok = true;
  int64_t cur = (int64_t)t - 1;
  for (;;) {
    const int64_t my = cur - (int64_t)lane;
    const bool real = my >= (int64_t)first;      // lanes before the scope's first tile act as a zero prefix
    uint64_t lo = pack_desc(F_PREFIX, 0), hi = 0;
    uint32_t nearest = 32, flag = F_PREFIX, spins = 0;
    uint64_t t0 = 0;                               // read when the wait starts to sleep
    for (;;) {
      if (real) ld_desc(desc + my, lo, hi);
      flag = (uint32_t)(lo & 3u);
      const uint32_t stop = __ballot_sync(0xFFFFFFFFu, flag >= F_PREFIX);
      const uint32_t inv = __ballot_sync(0xFFFFFFFFu, flag == F_INVALID);
      nearest = stop ? (uint32_t)__ffs((int)stop) - 1u : 32u;
      const uint32_t need = nearest >= 32u ? 0xFFFFFFFFu : ((1u << nearest) - 1u);
      if ((inv & need) == 0u) break;
      ++spins;
      if (spins == 8) t0 = global_timer_ns();
      if (__any_sync(0xFFFFFFFFu, wait_expired(spins, spin_limit, t0, budget_ns))) { ok = false; break; }
      if (spins > 8) __nanosleep(64);
    }
    if (!ok) break;
    const bool take = lane <= nearest;
    ex_a += warp_sum(take ? (lo >> 2) : 0ull);
    ex_b += warp_sum(take ? hi : 0ull);
    if (nearest < 32u) {
      const uint32_t ab = __ballot_sync(0xFFFFFFFFu, flag == F_ABORT);
      if ((ab >> nearest) & 1u) ok = false;
      break;
    }
    cur -= 32;
  }
  if (lane == 0) {
    if (ok) {
      st_desc(desc + t, pack_desc(F_PREFIX, ex_a + tot_a), ex_b + tot_b);
    } else {
      st_desc(desc + t, pack_desc(F_ABORT, 0), 0);
      atomicCAS(&ctl->status, (int)GD_OK, (int)GD_ERR_DEVICE_TIMEOUT);
    }
  }
  return ok;
}

// The first half alone, for callers that know a tile's totals long before they can afford to wait for its
// predecessors (a persistent kernel whose CTAs each hold several tiles): the totals are made known at once, and
// tile_lookback(..., published = true) sums the tiles before it later.  (Looking at four descriptors per lane and
// step instead of one was measured too, on 148 CTAs with two or three tiles in flight each: slower.)
__device__ __forceinline__ void tile_publish(uint4* desc, uint32_t t, uint32_t first, uint64_t tot_a, uint64_t tot_b) {
  st_desc(desc + t, pack_desc(t == first ? F_PREFIX : F_AGG, tot_a), tot_b);
}

}  // namespace gd
