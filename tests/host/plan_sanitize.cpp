// Exercises the host-side planner of gd_compress (csrc/gd_plan.hpp) on its own, so that it can run under the host
// compiler's address and undefined-behaviour sanitizers: the five workloads' layouts, ragged, empty, tiny and huge
// layers, hundreds of layers, every flag combination and drop ratio.  Checks the invariants the kernels rely on
// and prints "ok <plans>".  Exit code 1 and a message on the first violation.
#include <cstdio>
#include <cstdlib>
#include <initializer_list>
#include <random>

#include "gd_plan.hpp"

using namespace gd;

#define REQUIRE(cond)                                                        \
  do {                                                                       \
    if (!(cond)) {                                                           \
      std::fprintf(stderr, "line %d: %s failed\n", __LINE__, #cond);         \
      std::exit(1);                                                          \
    }                                                                        \
  } while (0)

static uint64_t kept(uint64_t n, uint32_t ppm) { return n - n * ppm / 1000000ull; }

static int check(const std::vector<uint64_t>& sizes, uint32_t n_shards, int scope_mode, uint32_t ppm, uint32_t flags,
                 const uint32_t* cols, uint64_t fused_units = 0) {
  std::vector<uint64_t> off(sizes.size() + 1, 0);
  for (size_t i = 0; i < sizes.size(); ++i) off[i + 1] = off[i] + sizes[i];
  const uint64_t n = off.back();
  Plan P;
  const int rc = make_plan(off.data(), (uint32_t)sizes.size(), cols, n_shards, scope_mode, ppm, flags, &P, fused_units);
  if (n > (1ull << 32)) { REQUIRE(rc == GD_ERR_TOO_LARGE); return 0; }
  REQUIRE(rc == GD_OK);
  const uint32_t ns = scope_mode == GD_SCOPE_GLOBAL ? 1u : (uint32_t)sizes.size();
  REQUIRE(P.n_scopes == ns && P.scopes.size() == ns);
  uint64_t out = 0, cand = 0, samp = 0;
  for (uint32_t s = 0; s < ns; ++s) {
    const ScopeDesc& d = P.scopes[s];
    REQUIRE(d.lo <= d.hi && d.hi <= n);
    if (s) REQUIRE(d.lo == P.scopes[s - 1].hi);
    const uint64_t len = d.hi - d.lo;
    REQUIRE(d.k == kept(len, ppm) && d.k <= len);
    REQUIRE(d.out_base == out && d.cand_base == cand && d.samp_base == samp);
    REQUIRE(d.cand_base % 4 == 0);                       // 16-byte aligned lists
    REQUIRE(d.cand_cap <= len && d.samp_m <= len && d.samp_rank <= d.samp_m);
    if (d.samp_m && !(flags & GD_FLAG_SAMPLED_THRESHOLD)) REQUIRE(d.samp_rank >= 1 && d.cand_cap >= (d.k < len ? d.k : len));
    if (d.samp_cluster > 1 && d.samp_m) {                // the last stratum's last group lies inside the scope
      const uint64_t first = (d.lo + d.samp_cluster - 1) / d.samp_cluster * d.samp_cluster;
      const uint64_t strata = d.samp_m / d.samp_cluster;
      const uint64_t groups = strata * d.samp_w + d.samp_rem;
      REQUIRE(d.samp_rem < strata || strata == 0);
      REQUIRE(first + groups * d.samp_cluster <= d.hi);
    } else if (d.samp_m) {
      REQUIRE(d.samp_m * d.samp_w + d.samp_rem == len);
    }
    out += d.k;
    cand += (d.cand_cap + 3) / 4 * 4;
    samp += d.samp_m;
  }
  REQUIRE(P.k_total == out && P.cand_total == cand && P.samp_total == samp);
  for (int l = 0; l < L_COUNT; ++l) {
    REQUIRE(P.tile0[l].size() == ns + 1 && P.tile0[l][0] == 0 && P.tile0[l][ns] == P.tiles[l]);
    for (uint32_t s = 0; s < ns; ++s) REQUIRE(P.tile0[l][s] <= P.tile0[l][s + 1]);
  }
  // the workspace regions ascend, are 256-byte aligned and end inside total_bytes
  const size_t regions[] = {P.off_ctl, P.off_state, P.off_hist, P.off_sums, P.off_cnts, P.off_desc_emit, P.off_desc_cand,
                            P.off_desc_dcomp, P.off_tables, P.off_flags, P.off_agg, P.off_samp, P.off_cand_idx, P.off_cand_val};
  for (size_t i = 0; i < sizeof(regions) / sizeof(regions[0]); ++i) {
    REQUIRE(regions[i] % 256 == 0 && regions[i] <= P.total_bytes);
    if (i) REQUIRE(regions[i - 1] <= regions[i]);
  }
  REQUIRE(P.zero_bytes == P.off_tables && P.off_tables + P.tables_bytes <= P.off_flags);
  REQUIRE(P.off_cand_val + 4 * P.cand_total <= P.total_bytes);
  REQUIRE(P.t_layer_cols + 4 * sizes.size() <= P.tables_bytes);
  REQUIRE(P.emit_chunk_tiles == 1 || P.emit_chunk_tiles == 2 || P.emit_chunk_tiles == 4 || P.emit_chunk_tiles == 8);
  REQUIRE(P.dense_sel_tile >= kTile && P.dense_sel_tile <= kDenseSelTileMax);
  REQUIRE(P.dense_chunk_tiles >= 1 && P.dense_chunk_tiles <= kDenseChunkTilesMax);
  if (P.local_predict) {
    REQUIRE(P.predict && P.tables_bytes <= kSetupBlobBytes);
    for (uint32_t s = 0; s < ns; ++s) REQUIRE(P.scopes[s].samp_m <= kLocalSampleMax);
    REQUIRE(P.samp_tile == 256 || P.samp_tile == 512 || P.samp_tile == 1024);
  }
  if (P.dense_bound) REQUIRE(!P.predict && !P.dense_fused && ns <= kSmemScopes);
  uint64_t units = 0;
  for (uint32_t s = 0; s < ns; ++s) units += (P.scopes[s].hi - P.scopes[s].lo + 1023) / 1024;
  REQUIRE(P.dense_units == units);
  if (P.dense_fused) REQUIRE(!P.predict && ns <= kSmemScopes && units <= fused_units);
  if (flags & GD_FLAG_PREDICT_ALWAYS) REQUIRE(P.predict && !P.dense_fused && !P.dense_bound);
  if (flags & GD_FLAG_NO_PREDICTION) REQUIRE(!P.predict);
  if (fused_units >= units && ns <= kSmemScopes && !(flags & (GD_FLAG_SAMPLED_THRESHOLD | GD_FLAG_PREDICT_ALWAYS)))
    REQUIRE(P.dense_fused);
  return 1;
}

int main() {
  long plans = 0;
  const std::vector<std::vector<uint64_t>> layouts = {
      {1ull << 20},
      {784 * 4096, 4096, 4096 * 4096, 4096, 40960, 10},
      {42500000, 42500000, 42500000, 85000, 1500000, 1000000, 1500000, 1000000, 1500000, 1000000, 1500000, 1000000},
      {1ull << 30},
      {1ull << 32},
      {(1ull << 32) + 1},
      {(1ull << 31) + (1ull << 20) + 5},
      {0},
      {0, 0, 0},
      {1},
      {3, 0, 1, 4097, 8192, 8193, 0, 123457},
      {300000, 17, 0, 150001, 4096},
      {1500000, 13, 900003},
  };
  for (const auto& sizes : layouts)
    for (int scope : {GD_SCOPE_GLOBAL, GD_SCOPE_PER_LAYER})
      for (uint32_t ppm : {0u, 300000u, 900000u, 990000u, 999000u, 999999u, 1000000u})
        for (uint32_t flags : {0u, (uint32_t)GD_FLAG_NO_PREDICTION, (uint32_t)GD_FLAG_SAMPLED_THRESHOLD, (uint32_t)GD_FLAG_NO_EARLY_ZERO})
          for (uint32_t shards : {1u, 4u, 33u}) plans += check(sizes, shards, scope, ppm, flags, nullptr);
  // with the one-launch kernel for short vectors on offer (a small and a large device), and prediction forced
  for (const auto& sizes : layouts)
    for (int scope : {GD_SCOPE_GLOBAL, GD_SCOPE_PER_LAYER})
      for (uint32_t flags : {0u, (uint32_t)GD_FLAG_NO_PREDICTION, (uint32_t)GD_FLAG_SAMPLED_THRESHOLD, (uint32_t)GD_FLAG_PREDICT_ALWAYS})
        for (uint64_t fused_units : {(uint64_t)1, (uint64_t)296, (uint64_t)2368, ~(uint64_t)0})
          plans += check(sizes, 3, scope, 990000u, flags, nullptr, fused_units);
  // hundreds of layers of random sizes (the tables no longer fit a kernel argument), with and without columns
  std::mt19937_64 rng(7);
  for (int rep = 0; rep < 40; ++rep) {
    const size_t layers = 1 + rng() % 600;
    std::vector<uint64_t> sizes(layers);
    std::vector<uint32_t> cols(layers);
    for (size_t i = 0; i < layers; ++i) {
      cols[i] = 1 + (uint32_t)(rng() % 64);
      sizes[i] = cols[i] * (rng() % ((rep % 4 == 0) ? 200000 : 3000));
    }
    for (int scope : {GD_SCOPE_GLOBAL, GD_SCOPE_PER_LAYER})
      for (uint32_t flags : {0u, (uint32_t)GD_FLAG_NO_PREDICTION, (uint32_t)GD_FLAG_SAMPLED_THRESHOLD})
        plans += check(sizes, 1 + (uint32_t)(rng() % 40), scope, 990000u, flags, rep % 2 ? cols.data() : nullptr);
  }
  // how large a sample is: short lists (at most 2^19 entries kept by the call) stay within what the launch that starts
  // the call selects from, down to 32 expected samples above the threshold; long lists and thinner samples do not
  {
    auto plan_of = [](const std::vector<uint64_t>& sizes, int scope, uint32_t ppm, Plan* P) {
      std::vector<uint64_t> off(sizes.size() + 1, 0);
      for (size_t i = 0; i < sizes.size(); ++i) off[i + 1] = off[i] + sizes[i];
      REQUIRE(make_plan(off.data(), (uint32_t)sizes.size(), nullptr, 4, scope, ppm, 0, P) == GD_OK);
    };
    Plan P;
    const std::vector<uint64_t> nmt = {42500000, 42500000, 42500000, 85000, 1500000, 1000000, 1500000, 1000000, 1500000, 1000000, 1500000, 1000000};
    for (uint32_t ppm : {990000u, 999000u}) {
      plan_of({1ull << 24}, GD_SCOPE_GLOBAL, ppm, &P);
      REQUIRE(P.predict && P.local_predict);
      plan_of(nmt, GD_SCOPE_PER_LAYER, ppm, &P);
      REQUIRE(P.predict && P.local_predict);
      for (const ScopeDesc& d : P.scopes)                  // at least 32 expected hits, unless a sixteenth of the scope is sampled
        if (d.samp_m + 8 < (d.hi - d.lo) / 16) REQUIRE((double)d.k * (double)d.samp_m >= 31.0 * (double)(d.hi - d.lo));
    }
    plan_of({1ull << 28}, GD_SCOPE_GLOBAL, 999000u, &P);   // 268 435 kept: still short
    REQUIRE(P.local_predict && P.scopes[0].samp_m == kLocalSampleMax);
    plan_of({1ull << 30}, GD_SCOPE_GLOBAL, 999000u, &P);   // 1 073 742 kept: the sample keeps its 256 expected hits
    REQUIRE(P.predict && !P.local_predict && P.scopes[0].samp_m > kLocalSampleMax);
    plan_of({1ull << 24}, GD_SCOPE_GLOBAL, 999500u, &P);   // 32 hits would need more than one CTA holds
    REQUIRE(P.predict && !P.local_predict);
    plan_of({1ull << 30}, GD_SCOPE_GLOBAL, 990000u, &P);   // long lists at R = 99 %: 256 hits are 25 600 samples
    REQUIRE(P.local_predict && P.scopes[0].samp_m >= 25000 && P.scopes[0].samp_m <= 26000);
    plan_of({1ull << 24}, GD_SCOPE_GLOBAL, 990000u, &P);   // short lists at R = 99 %: 128 hits
    REQUIRE(P.local_predict && P.scopes[0].samp_m >= 12500 && P.scopes[0].samp_m <= 13000);
  }
  // arguments that must be refused
  {
    Plan P;
    uint64_t bad[] = {0, 10, 5};
    REQUIRE(make_plan(bad, 2, nullptr, 1, GD_SCOPE_GLOBAL, 990000, 0, &P) == GD_ERR_INVALID_ARG);
    uint64_t good[] = {0, 10};
    REQUIRE(make_plan(good, 1, nullptr, 0, GD_SCOPE_GLOBAL, 990000, 0, &P) == GD_ERR_INVALID_ARG);
    REQUIRE(make_plan(good, 1, nullptr, 1, 7, 990000, 0, &P) == GD_ERR_INVALID_ARG);
    REQUIRE(make_plan(good, 1, nullptr, 1, GD_SCOPE_GLOBAL, 1000001, 0, &P) == GD_ERR_INVALID_ARG);
    uint32_t c3[] = {3};
    REQUIRE(make_plan(good, 1, c3, 1, GD_SCOPE_GLOBAL, 990000, 0, &P) == GD_ERR_INVALID_ARG);   // 10 is no multiple of 3
    REQUIRE(make_plan(nullptr, 1, nullptr, 1, GD_SCOPE_GLOBAL, 990000, 0, &P) == GD_ERR_INVALID_ARG);
  }
  std::printf("ok %ld\n", plans);
  return 0;
}
