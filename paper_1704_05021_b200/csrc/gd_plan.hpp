// The host-side planner of gd_compress: from the layer offsets, the drop ratio and the flags to scopes, sample sizes,
// candidate capacities, tile tables and the byte layout of the workspace.  Plain C++ (no CUDA), so that it can be
// built with the host compiler's address and undefined-behaviour sanitizers and exercised on its own.
#pragma once

#include <cmath>
#include <vector>

#include "gd_layout.h"

namespace gd {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// Sample size per scope: the sample is sized for a number of expected samples above the threshold
// ("hits") that grows with the scope's k.  A sample costs scattered reads in proportion to its size; a
// small one costs a wider safety margin, i.e. extra candidates in proportion to k / sqrt(hits).  The sum
// is smallest near hits ~ k^(2/3) (the measured costs per sample and per candidate are about equal;
// factors of 0.12, 0.25 and 0.5 were timed on layered models of 12 to 387 tensors), so:
// hits = kHitsFactor * k^(2/3) within [kHitsMin, kHitsMax], and never more than kSampleMax samples or a
// sixteenth of the scope.
// While the lists are short - the call keeps at most kShortListsK entries in all - the sample is on the critical path (the
// fused pass waits for the prediction) and a longer list costs next to nothing: the cap is 128 there (step time at
// R = 99 %, 256 / 128 / 64 hits: 2^22 elements 65 / 62 / 60 us, 2^24 94 / 91 / 89 us, 2^25 136 / 133 / 132 us, the MNIST-shaped
// model 104 / 103 / 104 us; from 2^26 elements on 256 is as good or better, and on the NMT-shaped model 128 costs 16 us:
// its lists then outgrow the shared-memory stage of the kernel that selects among them).
constexpr double kHitsFactor = 0.25, kHitsMin = 32.0, kHitsMax = 256.0, kHitsMaxShortLists = 128.0, kSampleMax = 262144.0;
constexpr uint64_t kShortListsK = 1ull << 19;
constexpr uint64_t kSampleAllMax = 8192;         // scopes up to this length are sampled completely
constexpr uint64_t kClusterMaxStride = 1024;      // strata up to this many elements wide are sampled in groups of 8
constexpr uint64_t kAutoDenseMax = 3ull << 18;   // vectors up to this length skip the prediction (measured, step time
                                                 // with L2 flushed: dense 56 us against 58 us predicted at 2^19 elements,
                                                 // 65 against 59 at 2^20, 83 against 63 at 2^21) - and so do all that the
                                                 // one-launch kernel for short vectors can hold (38 / 40 / 46 / 54 us against
                                                 // 56 / 58 / 60 / 65 us predicted at 2^18 .. 2^21 elements)

inline uint64_t kept_count(uint64_t n, uint32_t drop_ppm) {
  return n - (n * (uint64_t)drop_ppm) / 1000000ull;   // n <= 2^32, drop_ppm <= 1e6: no overflow
}

// How one scope is sampled for the prediction and how many candidate slots it gets.  A scope of
// ns elements keeping k: m stratified samples are read and the predicted lower bound is the rank-th
// largest sample key.  rank is chosen so that, for independent samples, the number of entries at or
// above the prediction is at least k with a margin of six standard deviations plus 12.5 %.  Small
// scopes are sampled completely, which makes the prediction the exact threshold.  None of this
// affects results: a scope whose prediction fails is selected densely.
inline void plan_prediction(uint64_t ns, uint64_t k, double hits_max, uint64_t* m, uint64_t* rank, uint64_t* cap,
                            uint32_t* cluster) {
  *cluster = 1;
  if (k == 0 || ns == 0) { *m = 0; *rank = 0; *cap = 0; return; }
  double hits = kHitsFactor * std::cbrt((double)k * (double)k);
  if (hits < kHitsMin) hits = kHitsMin;
  if (hits > hits_max) hits = hits_max;
  double target = hits * (double)ns / (double)k;
#ifndef GD_NO_LOCAL_CLAMP
  // Short lists (hits_max below kHitsMax): a sample that one CTA can hold is predicted from in the launch that starts
  // the call (kLocalSampleMax values; gd_predict.cu) instead of two launches more - worth a wider margin, as long as
  // the expected hits stay at or above kHitsMin.
  if (hits_max < kHitsMax && target > (double)kLocalSampleMax && (double)kLocalSampleMax * (double)k >= kHitsMin * (double)ns)
    target = (double)kLocalSampleMax;
#endif
  if (target > kSampleMax) target = kSampleMax;
  if (target > (double)ns / 16.0) target = (double)ns / 16.0;
  uint64_t mt = (uint64_t)target;
  if (ns <= kSampleAllMax || mt < 64) {
    *m = ns;
    *rank = k;
    uint64_t c = 3 * k + 1024;
    *cap = c < ns ? c : ns;
    return;
  }
  // The sample is bound by the rate of scattered DRAM reads (about 22 G/s, two per sample).  Narrow strata (a
  // sample every few sectors): whole groups of 8 consecutive elements are sampled, an eighth of the reads.  Wide
  // strata: pairs of neighbours, half the reads; larger groups there would leave too few distinct places (rows
  // of a matrix) in the sample - a pair at most doubles the variance the rank's margin of six sigma is sized for.
  if (ns / mt <= kClusterMaxStride) {
    mt &= ~7ull;
    *cluster = 8;
  } else {
    mt &= ~1ull;
    *cluster = 2;
  }
  *m = mt;
  const double x = (double)k * (double)mt / (double)ns;
  const double y = 3.0 + std::sqrt(9.0 + 1.125 * x + 1.0);
  uint64_t r = (uint64_t)std::ceil(y * y);
  if (r > mt) r = mt;
  if (r < 1) r = 1;
  *rank = r;
  uint64_t c = 3 * k + 128 * (ns / mt) + 1024;
  *cap = c < ns ? c : ns;
}

// Sampled-threshold mode (Section 4): sample size and output capacity of one scope.
inline uint64_t sampled_m(uint64_t ns) {
  if (ns <= 4096) return ns;            // sampled completely, element by element
  uint64_t m = (ns + 999) / 1000;
  if (m < 4096) m = 4096;
  return m + (m & 1);                   // longer scopes: pairs of neighbours
}
inline uint64_t sampled_cap(uint64_t ns, uint64_t k) {
  const uint64_t c = 4 * k + 8192;
  return c < ns ? c : ns;
}

struct Plan {
  std::vector<ScopeDesc> scopes;
  std::vector<uint32_t> tile0[L_COUNT];
  std::vector<uint64_t> samp_off;
  uint32_t tiles[L_COUNT] = {0, 0, 0, 0, 0};
  uint64_t samp_total = 0, cand_total = 0, k_total = 0;
  uint32_t n_scopes = 0;
  bool predict = true;
  bool local_predict = false;   // the prediction shares a launch with the start of the call (gd_predict.cu)
  bool dense_bound = false;     // no sample: the lower bounds come from a histogram pass over the dense vector (gd_dense.cu)
  bool dense_fused = false;     // no sample, short vector: add, selection and compaction in one launch (gd_candidates.cu)
  uint64_t dense_units = 0;     // the scopes' lengths in units of 1024 elements, summed
  uint32_t emit_chunk_tiles = 1, dense_sel_tile = kDenseSelTileMax, dense_chunk_tiles = kDenseChunkTilesMax;
  uint32_t samp_tile = kTile;
  // workspace layout (byte offsets)
  size_t off_ctl = 0, off_state = 0, off_hist = 0, off_sums = 0, off_cnts = 0, off_desc_emit = 0,
         off_desc_cand = 0, off_desc_dcomp = 0, zero_bytes = 0;
  size_t off_tables = 0, tables_bytes = 0;
  size_t t_scopes = 0, t_tile0[L_COUNT] = {0, 0, 0, 0, 0}, t_samp_off = 0, t_layer_off = 0, t_shard_off = 0,
         t_pair_off = 0, t_layer_cols = 0;
  std::vector<uint64_t> pair_off;
  std::vector<uint32_t> layer_cols;
  uint64_t n_pairs = 0;
  size_t off_agg = 0, off_flags = 0, off_samp = 0, off_cand_idx = 0, off_cand_val = 0, total_bytes = 0;
};

inline int check_offsets(const uint64_t* off, uint32_t count, uint64_t* n_out) {
  if (!off || count == 0) return GD_ERR_INVALID_ARG;
  if (off[0] != 0) return GD_ERR_INVALID_ARG;
  for (uint32_t i = 0; i < count; ++i)
    if (off[i + 1] < off[i]) return GD_ERR_INVALID_ARG;
  *n_out = off[count];
  return GD_OK;
}

// layer_cols == NULL: one (mu+, mu-) pair per layer.
inline int make_plan(const uint64_t* layer_off, uint32_t n_layers, const uint32_t* layer_cols, uint32_t n_shards, int scope_mode,
              uint32_t drop_ppm, uint32_t flags, Plan* P, uint64_t fused_units = 0) {
  uint64_t n = 0;
  int rc = check_offsets(layer_off, n_layers, &n);
  if (rc != GD_OK) return rc;
  if (n_shards == 0 || drop_ppm > 1000000u) return GD_ERR_INVALID_ARG;
  if (scope_mode != GD_SCOPE_GLOBAL && scope_mode != GD_SCOPE_PER_LAYER) return GD_ERR_INVALID_ARG;
  if (n > (1ull << 32)) return GD_ERR_TOO_LARGE;
  const bool sampled = (flags & GD_FLAG_SAMPLED_THRESHOLD) != 0;
  const uint32_t ns_planned = scope_mode == GD_SCOPE_GLOBAL ? 1u : n_layers;
  // fused_units: how many units of 1024 elements the one-launch kernel for short vectors holds on this device (0: not
  // available).  A scope's last unit may be partial.
  uint64_t units = 0;
  if (scope_mode == GD_SCOPE_GLOBAL) units = (n + 1023) / 1024;
  else for (uint32_t l = 0; l < n_layers; ++l) units += (layer_off[l + 1] - layer_off[l] + 1023) / 1024;
  P->dense_units = units;
  const bool fused_fits = ns_planned <= kSmemScopes && units <= fused_units;
  // Short vectors are selected densely right away: below about 2^20 elements the three dense passes
  // run out of L2 and cost less than sampling, predicting and selecting among candidates.
  const bool predict = !(flags & GD_FLAG_NO_PREDICTION) && (sampled || (flags & GD_FLAG_PREDICT_ALWAYS) || (!fused_fits && n > kAutoDenseMax));
  P->predict = predict;
  P->dense_fused = !predict && fused_fits;
  // Without a sample, long vectors still go through the candidate lists: one histogram pass over the dense vector
  // gives every scope an exact lower bound of its threshold (gd_dense.cu).  Short vectors, whose passes run out
  // of L2, and calls with more scopes than the kernels over the lists keep in shared memory take the plain dense
  // selection and compaction.
  P->dense_bound = !predict && !P->dense_fused && n > kAutoDenseMax && ns_planned <= kSmemScopes;
  P->pair_off.assign((size_t)n_layers + 1, 0);
  P->layer_cols.assign(n_layers, 1);
  for (uint32_t l = 0; l < n_layers; ++l) {
    const uint64_t size = layer_off[l + 1] - layer_off[l];
    uint32_t cols = layer_cols ? layer_cols[l] : 1u;
    if (cols == 0 || (size % cols) != 0) return GD_ERR_INVALID_ARG;   // a layer is rows x cols, row-major
    P->layer_cols[l] = cols;
    P->pair_off[l + 1] = P->pair_off[l] + cols;
  }
  P->n_pairs = P->pair_off[n_layers];
  // The fused pass works in chunks of 1, 2, 4 or 8 tiles.  One CTA per chunk (more than 32 scopes, gd_emit.cu): as
  // large as still leaves a wave and a half of CTAs (4 per SM on 148 SMs) for the whole vector.  (Measured on
  // 2^21 .. 2^26 elements: four waves, the first rule, cost 20-30 % more time at 2^23 .. 2^25; one wave loses to the
  // tail.)  The persistent pipeline (gd_emit_pipe.cu) hides a chunk's start-up and look-back, so its chunks are
  // smaller - the last ones end closer together - but not so small that the look-back, two chunks deep, falls behind.
  const uint64_t dense_tiles = (n + kTile - 1) / kTile;
  uint32_t chunk_tiles = ns_planned <= kSmemScopes ? 4 : 8;
  const uint64_t per_size = ns_planned <= kSmemScopes ? 296u : 888u;
  while (chunk_tiles > 1 && dense_tiles < (uint64_t)chunk_tiles * per_size) chunk_tiles >>= 1;
#ifdef GD_FORCE_CHUNK
  chunk_tiles = GD_FORCE_CHUNK;
#endif
  P->emit_chunk_tiles = chunk_tiles;
  const uint64_t CH = (uint64_t)chunk_tiles * kTile;
  // The dense kernels (used when a prediction fails) take large tiles on long vectors, where the
  // chain of look-backs and the flushes of histograms must stay rare, and small ones on short
  // vectors, which otherwise would not fill the GPU.
  uint32_t sel_tile = kDenseSelTileMax, dchunk = kDenseChunkTilesMax;
  while (sel_tile > kTile && n / sel_tile < 592u) sel_tile >>= 1;
  // (chunks of the dense compaction: about 48 per resident CTA, so that scopes whose survivors crowd at one
  // end - a sparse layer whose kept zeros are its first ones - still spread over the GPU)
  while (dchunk > 1 && n / ((uint64_t)dchunk * kTile) < 7104u) dchunk >>= 1;
  P->dense_sel_tile = sel_tile;
  P->dense_chunk_tiles = dchunk;
  const uint32_t ns_count = scope_mode == GD_SCOPE_GLOBAL ? 1u : n_layers;
  P->n_scopes = ns_count;
  P->scopes.resize(ns_count);
  for (int l = 0; l < L_COUNT; ++l) P->tile0[l].assign(ns_count + 1, 0);
  P->samp_off.assign(ns_count + 1, 0);
  uint64_t tiles[L_COUNT] = {0, 0, 0, 0, 0};
  uint64_t out_base = 0, cand_base = 0, samp_base = 0;
  const double hits_max = kept_count(n, drop_ppm) <= kShortListsK ? kHitsMaxShortLists : kHitsMax;
  for (uint32_t s = 0; s < ns_count; ++s) {
    ScopeDesc& d = P->scopes[s];
    d.lo = scope_mode == GD_SCOPE_GLOBAL ? 0 : layer_off[s];
    d.hi = scope_mode == GD_SCOPE_GLOBAL ? n : layer_off[s + 1];
    const uint64_t ns = d.hi - d.lo;
    d.k = kept_count(ns, drop_ppm);
    d.out_base = out_base;
    out_base += d.k;
    uint64_t m = 0, rank = 0, cap = 0;
    uint32_t cluster = 1;
    if (sampled) {
      m = sampled_m(ns);
      cluster = ns <= 4096 ? 1u : 2u;
      rank = kept_count(m, drop_ppm);
      cap = sampled_cap(ns, d.k);
    } else if (predict) {
      plan_prediction(ns, d.k, hits_max, &m, &rank, &cap, &cluster);
    } else if (P->dense_bound) {
      // the candidates are the keys above the bin of the k-th largest key (fewer than k) and that bin itself
      const uint64_t c = 3 * d.k + 4096;
      cap = c < ns ? c : ns;
    }
    d.cand_base = cand_base;
    d.cand_cap = cap;
    cand_base += (cap + 3) / 4 * 4;
    d.samp_base = samp_base;
    d.samp_m = m;
    d.samp_rank = rank;
    d.samp_cluster = cluster;
    if (cluster > 1) {   // strata of groups of 8 (or 2) elements, from the first multiple of that at or after lo
      const uint64_t first = (d.lo + cluster - 1) & ~(uint64_t)(cluster - 1);
      const uint64_t groups = (d.hi - first) / cluster, strata = m / cluster;
      d.samp_w = groups / strata;
      d.samp_rem = (uint32_t)(groups % strata);
    } else {
      d.samp_w = m ? ns / m : 0;
      d.samp_rem = m ? (uint32_t)(ns % m) : 0;
    }
    samp_base += m;
    for (int l = 0; l < L_COUNT; ++l) P->tile0[l][s] = (uint32_t)tiles[l];
    P->samp_off[s] = d.samp_base;
    if (ns) {
      tiles[L_EMIT] += (d.hi + CH - 1) / CH - d.lo / CH;
      tiles[L_DSEL] += (ns + sel_tile - 1) / sel_tile;
      tiles[L_DCOMP] += (ns + (uint64_t)dchunk * kTile - 1) / ((uint64_t)dchunk * kTile);
    }
    tiles[L_SAMP] += (m + kTile - 1) / kTile;
    tiles[L_CAND] += (cap + kTile - 1) / kTile;
  }
  for (int l = 0; l < L_COUNT; ++l) {
    if (tiles[l] > 0x7FFFFFFFull) return GD_ERR_TOO_LARGE;
    P->tile0[l][ns_count] = (uint32_t)tiles[l];
    P->tiles[l] = (uint32_t)tiles[l];
  }
  // The sample is gathered with scattered reads, of which one SM keeps only so many in flight: a short
  // sample is cut into tiles of 1024 so that its gather spreads over all SMs.
  P->samp_tile = kTile;
  while (P->samp_tile > 1024u && samp_base / P->samp_tile < 2u * 148u) P->samp_tile >>= 2;
  if (P->samp_tile != kTile) {
    uint64_t t = 0;
    for (uint32_t s = 0; s < ns_count; ++s) {
      P->tile0[L_SAMP][s] = (uint32_t)t;
      t += (P->scopes[s].samp_m + P->samp_tile - 1) / P->samp_tile;
    }
    P->tile0[L_SAMP][ns_count] = (uint32_t)t;
    P->tiles[L_SAMP] = (uint32_t)t;
  }
  P->samp_off[ns_count] = samp_base;
  P->samp_total = samp_base;
  P->cand_total = cand_base;
  P->k_total = out_base;

  size_t off = 0;
  P->off_ctl = off;          off = align_up(off + sizeof(Ctl));
  P->off_state = off;        off = align_up(off + sizeof(ScopeState) * ns_count);
  P->off_hist = off;         off = align_up(off + sizeof(unsigned long long) * kHistBinsPerScope * (size_t)ns_count);
  P->off_sums = off;         off = align_up(off + sizeof(double) * 2 * (size_t)P->n_pairs);
  P->off_cnts = off;         off = align_up(off + sizeof(unsigned long long) * 2 * (size_t)P->n_pairs);
  P->off_desc_emit = off;    off = align_up(off + 16 * (size_t)P->tiles[L_EMIT]);
  P->off_desc_cand = off;    off = align_up(off + 16 * (size_t)P->tiles[L_CAND]);
  P->off_desc_dcomp = off;   off = align_up(off + 16 * (size_t)P->tiles[L_DCOMP]);
  P->zero_bytes = off;
  P->off_tables = off;
  size_t t = 0;
  auto sub = [](size_t x) { return (x + 15) / 16 * 16; };   // tables are packed at 16-byte steps
  P->t_scopes = t;           t = sub(t + sizeof(ScopeDesc) * ns_count);
  for (int l = 0; l < L_COUNT; ++l) { P->t_tile0[l] = t; t = sub(t + sizeof(uint32_t) * (ns_count + 1)); }
  P->t_samp_off = t;         t = sub(t + sizeof(uint64_t) * (ns_count + 1));
  P->t_layer_off = t;        t = sub(t + sizeof(uint64_t) * ((size_t)n_layers + 1));
  P->t_shard_off = t;        t = sub(t + sizeof(uint64_t) * ((size_t)n_shards + 1));
  P->t_pair_off = t;         t = sub(t + sizeof(uint64_t) * ((size_t)n_layers + 1));
  P->t_layer_cols = t;       t = sub(t + sizeof(uint32_t) * (size_t)n_layers);
  t = align_up(t);
  P->tables_bytes = t;
  off += t;
  // Samples of at most kLocalSampleMax values per scope are gathered in tiles of 256 by the kernel that also starts
  // the call; it marks every finished tile in an array of flags.
  P->local_predict = predict && !sampled && P->tables_bytes <= kSetupBlobBytes;
  for (uint32_t s = 0; P->local_predict && s < ns_count; ++s)
    if (P->scopes[s].samp_m > kLocalSampleMax) P->local_predict = false;
  if (P->local_predict) {
    // tiles of 256 samples spread a short sample over many SMs; larger tiles keep all CTAs resident at once
    for (P->samp_tile = 256;; P->samp_tile *= 2) {
      uint64_t tt = 0;
      for (uint32_t s = 0; s < ns_count; ++s) {
        P->tile0[L_SAMP][s] = (uint32_t)tt;
        tt += (P->scopes[s].samp_m + P->samp_tile - 1) / P->samp_tile;
      }
      P->tile0[L_SAMP][ns_count] = (uint32_t)tt;
      P->tiles[L_SAMP] = (uint32_t)tt;
      if (tt <= 2u * 148u || P->samp_tile == 1024u) break;
    }
  }
  // (marks of the sample tiles, then one per scope - its prediction is written - and one per CTA that clears: not cleared)
  P->off_flags = off;        off = align_up(off + sizeof(uint32_t) * ((size_t)P->tiles[L_SAMP] + kSmemScopes + kStartMarks));
  P->off_agg = off;          off = align_up(off + 32 * (size_t)kSelectCompactMaxGrid);   // per-CTA records, not cleared
  P->off_samp = off;         off = align_up(off + sizeof(float) * P->samp_total);
  P->off_cand_idx = off;     off = align_up(off + sizeof(uint32_t) * P->cand_total);
  P->off_cand_val = off;     off = align_up(off + sizeof(float) * P->cand_total);
  P->total_bytes = off;
  return GD_OK;
}

}  // namespace gd
