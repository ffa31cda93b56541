// Host side of libgd.so: argument checks, the per-call plan (scopes, tile tables, workspace
// layout) and the C entry points declared in include/gd.h.
#include <atomic>
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "gd_internal.cuh"

namespace gd {

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// Sample size per scope: the sample is sized for a number of expected samples above the threshold
// ("hits") that grows with the scope's k.  A sample costs scattered reads in proportion to its size; a
// small one costs a wider safety margin, i.e. extra candidates in proportion to k / sqrt(hits).  The sum
// is smallest near hits ~ k^(2/3) (the measured costs per sample and per candidate are about equal;
// factors of 0.12, 0.25 and 0.5 were timed on layered models of 12 to 387 tensors), so:
// hits = kHitsFactor * k^(2/3) within [kHitsMin, kHitsMax], and never more than kSampleMax samples or a
// sixteenth of the scope.
constexpr double kHitsFactor = 0.25, kHitsMin = 32.0, kHitsMax = 256.0, kSampleMax = 262144.0;
constexpr uint64_t kSampleAllMax = 8192;         // scopes up to this length are sampled completely
constexpr uint64_t kClusterMaxStride = 1024;      // strata up to this many elements wide are sampled in groups of 8
constexpr uint64_t kAutoDenseMax = 3ull << 19;   // vectors up to this length skip the prediction (measured: dense 69 us
                                                 // against 87 us at 2^20, 93 against 89 at 2^21)

inline uint64_t kept_count(uint64_t n, uint32_t drop_ppm) {
  return n - (n * (uint64_t)drop_ppm) / 1000000ull;   // n <= 2^32, drop_ppm <= 1e6: no overflow
}

// How one scope is sampled for the prediction and how many candidate slots it gets.  A scope of
// ns elements keeping k: m stratified samples are read and the predicted lower bound is the rank-th
// largest sample key.  rank is chosen so that, for independent samples, the number of entries at or
// above the prediction is at least k with a margin of six standard deviations plus 12.5 %.  Small
// scopes are sampled completely, which makes the prediction the exact threshold.  None of this
// affects results: a scope whose prediction fails is selected densely.
void plan_prediction(uint64_t ns, uint64_t k, uint64_t* m, uint64_t* rank, uint64_t* cap, uint32_t* cluster) {
  *cluster = 1;
  if (k == 0 || ns == 0) { *m = 0; *rank = 0; *cap = 0; return; }
  double hits = kHitsFactor * std::cbrt((double)k * (double)k);
  if (hits < kHitsMin) hits = kHitsMin;
  if (hits > kHitsMax) hits = kHitsMax;
  double target = hits * (double)ns / (double)k;
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

int check_offsets(const uint64_t* off, uint32_t count, uint64_t* n_out) {
  if (!off || count == 0) return GD_ERR_INVALID_ARG;
  if (off[0] != 0) return GD_ERR_INVALID_ARG;
  for (uint32_t i = 0; i < count; ++i)
    if (off[i + 1] < off[i]) return GD_ERR_INVALID_ARG;
  *n_out = off[count];
  return GD_OK;
}

// layer_cols == NULL: one (mu+, mu-) pair per layer.
int make_plan(const uint64_t* layer_off, uint32_t n_layers, const uint32_t* layer_cols, uint32_t n_shards, int scope_mode,
              uint32_t drop_ppm, uint32_t flags, Plan* P) {
  uint64_t n = 0;
  int rc = check_offsets(layer_off, n_layers, &n);
  if (rc != GD_OK) return rc;
  if (n_shards == 0 || drop_ppm > 1000000u) return GD_ERR_INVALID_ARG;
  if (scope_mode != GD_SCOPE_GLOBAL && scope_mode != GD_SCOPE_PER_LAYER) return GD_ERR_INVALID_ARG;
  if (n > (1ull << 32)) return GD_ERR_TOO_LARGE;
  const bool sampled = (flags & GD_FLAG_SAMPLED_THRESHOLD) != 0;
  // Short vectors are selected densely right away: below about 2^21 elements the three dense passes
  // run out of L2 and cost less than sampling, predicting and selecting among candidates.
  const bool predict = !(flags & GD_FLAG_NO_PREDICTION) && (sampled || n > kAutoDenseMax);
  P->predict = predict;
  // Without a sample, long vectors still go through the candidate lists: one histogram pass over the dense vector
  // gives every scope an exact lower bound of its threshold (gd_dense.cu).  Short vectors, whose passes run out
  // of L2, and calls with more scopes than the kernels over the lists keep in shared memory take the plain dense
  // selection and compaction.
  const uint32_t ns_planned = scope_mode == GD_SCOPE_GLOBAL ? 1u : n_layers;
  P->dense_bound = !predict && !sampled && n > kAutoDenseMax && ns_planned <= kSmemScopes;
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
  // The fused pass gives each CTA a chunk of 1, 2, 4 or 8 tiles: as large as still leaves a wave and a
  // half of CTAs (4 per SM on 148 SMs) for the whole vector.  (Measured on 2^21 .. 2^26 elements: four
  // waves, the first rule, cost 20-30 % more time at 2^23 .. 2^25; one wave loses to the tail.)
  const uint64_t dense_tiles = (n + kTile - 1) / kTile;
  uint32_t chunk_tiles = 8;
  while (chunk_tiles > 1 && dense_tiles < (uint64_t)chunk_tiles * 888u) chunk_tiles >>= 1;
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
      plan_prediction(ns, d.k, &m, &rank, &cap, &cluster);
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
  // Samples of at most local_sample_max() values per scope are gathered in tiles of 256 by the kernel that also starts
  // the call; it marks every finished tile in an array of flags.
  P->local_predict = predict && !sampled && P->tables_bytes <= kSetupBlobBytes;
  for (uint32_t s = 0; P->local_predict && s < ns_count; ++s)
    if (P->scopes[s].samp_m > local_sample_max()) P->local_predict = false;
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
  P->off_flags = off;        off = align_up(off + sizeof(uint32_t) * (size_t)P->tiles[L_SAMP]);   // not cleared
  P->off_agg = off;          off = align_up(off + 32 * (size_t)select_compact_max_grid());   // per-CTA records, not cleared
  P->off_samp = off;         off = align_up(off + sizeof(float) * P->samp_total);
  P->off_cand_idx = off;     off = align_up(off + sizeof(uint32_t) * P->cand_total);
  P->off_cand_val = off;     off = align_up(off + sizeof(float) * P->cand_total);
  P->total_bytes = off;
  return GD_OK;
}

// Start of a call in one launch: clears the control region of the workspace and writes the small
// host-built tables, which travel as a kernel argument, behind it.

__global__ void __launch_bounds__(kThreads) setup_kernel(const __grid_constant__ SetupBlob blob, uint4* tables_dst,
                                                         uint32_t tables_vec, uint4* zero_dst, uint64_t zero_vec) {
  const uint64_t stride = (uint64_t)gridDim.x * kThreads;
  const uint64_t g = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
  for (uint64_t i = g; i < zero_vec; i += stride) zero_dst[i] = make_uint4(0u, 0u, 0u, 0u);
  const uint4* src = reinterpret_cast<const uint4*>(blob.bytes);
  for (uint64_t i = g; i < tables_vec; i += stride) tables_dst[i] = src[i];
}

// A named range per entry point, visible to profilers that understand NVTX (no cost to speak of otherwise).
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
};

// measurement hooks
constexpr uint32_t kProfilePairs = 4096;
int g_profile_mode = 0;   // 0 off, 1 the fused pass only, 2 every kernel
cudaEvent_t g_ev_begin[kProfilePairs], g_ev_end[kProfilePairs];
uint32_t g_ev_tag[kProfilePairs];
uint32_t g_ev_created = 0, g_ev_used = 0;
bool g_pair_open = false;
std::atomic<uint64_t> g_launches{0};   // calls may come from several host threads

}  // namespace

void note_launches(uint32_t count) { g_launches.fetch_add(count, std::memory_order_relaxed); }

cudaError_t launch_setup(void* tables_dst, const void* tables_src, size_t tables_bytes, void* zero_dst, size_t zero_bytes,
                         cudaStream_t stream) {
  if (tables_bytes > kSetupBlobBytes) {   // many layers: the tables do not fit a kernel argument
    cudaError_t e = cudaMemsetAsync(zero_dst, 0, zero_bytes, stream);
    if (e != cudaSuccess) return e;
    return cudaMemcpyAsync(tables_dst, tables_src, tables_bytes, cudaMemcpyHostToDevice, stream);
  }
  ProfileScope prof(stream, PT_SETUP);
  SetupBlob blob;
  std::memcpy(blob.bytes, tables_src, tables_bytes);
  const uint64_t zero_vec = zero_bytes / 16;   // both regions are 256-byte aligned and padded
  uint64_t blocks = (zero_vec + kThreads * 8 - 1) / (kThreads * 8);
  const uint64_t cap = (uint64_t)sm_count() * 4;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  setup_kernel<<<(unsigned)blocks, kThreads, 0, stream>>>(blob, (uint4*)tables_dst, (uint32_t)(tables_bytes / 16),
                                                         (uint4*)zero_dst, zero_vec);
  GD_LAUNCH_CHECK();
  return cudaSuccess;
}

int sm_count() {
  static std::atomic<int> cached{0};
  if (cached.load(std::memory_order_relaxed) > 0) return cached.load(std::memory_order_relaxed);
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
    return 148;   // B200; only sizes grids
  cached.store(sms, std::memory_order_relaxed);
  return sms;
}

void profile_mark(cudaStream_t stream, bool begin, uint32_t tag) {
  if (g_profile_mode == 0 || (g_profile_mode == 1 && tag != PT_ADD_EMIT)) return;
  if (begin) {
    g_pair_open = false;
    if (g_ev_used >= kProfilePairs) return;
    if (g_ev_used >= g_ev_created) {
      if (cudaEventCreate(&g_ev_begin[g_ev_created]) != cudaSuccess) return;
      if (cudaEventCreate(&g_ev_end[g_ev_created]) != cudaSuccess) { cudaEventDestroy(g_ev_begin[g_ev_created]); return; }
      ++g_ev_created;
    }
    if (cudaEventRecord(g_ev_begin[g_ev_used], stream) == cudaSuccess) g_pair_open = true;
  } else if (g_pair_open) {
    cudaEventRecord(g_ev_end[g_ev_used], stream);
    g_ev_tag[g_ev_used] = tag;
    ++g_ev_used;
    g_pair_open = false;
  }
}

}  // namespace gd

using namespace gd;

extern "C" {

const char* gd_status_string(int status) {
  switch (status) {
    case GD_OK: return "ok";
    case GD_ERR_INVALID_ARG: return "invalid argument";
    case GD_ERR_TOO_LARGE: return "gradient too large for 32-bit indices";
    case GD_ERR_WORKSPACE: return "workspace missing or too small";
    case GD_ERR_CUDA: return "CUDA runtime error";
    case GD_ERR_DEVICE_TIMEOUT: return "bounded device-side wait timed out";
    case GD_ERR_INTERNAL: return "device-side consistency check failed";
    case GD_ERR_OVERFLOW: return "more survivors than the sampled-threshold capacity";
    default: return "unknown status";
  }
}

int gd_kept_count(uint64_t n_scope, uint32_t drop_ppm, uint64_t* k_out) {
  if (!k_out || drop_ppm > 1000000u) return GD_ERR_INVALID_ARG;
  if (n_scope > (1ull << 32)) return GD_ERR_TOO_LARGE;
  *k_out = kept_count(n_scope, drop_ppm);
  return GD_OK;
}

int gd_total_kept(const uint64_t* layer_off, uint32_t n_layers, int scope_mode, uint32_t drop_ppm,
                  uint64_t* k_total_out) {
  if (!k_total_out || drop_ppm > 1000000u) return GD_ERR_INVALID_ARG;
  if (scope_mode != GD_SCOPE_GLOBAL && scope_mode != GD_SCOPE_PER_LAYER) return GD_ERR_INVALID_ARG;
  uint64_t n = 0;
  int rc = check_offsets(layer_off, n_layers, &n);
  if (rc != GD_OK) return rc;
  if (n > (1ull << 32)) return GD_ERR_TOO_LARGE;
  uint64_t total = 0;
  if (scope_mode == GD_SCOPE_GLOBAL) {
    total = kept_count(n, drop_ppm);
  } else {
    for (uint32_t l = 0; l < n_layers; ++l) total += kept_count(layer_off[l + 1] - layer_off[l], drop_ppm);
  }
  *k_total_out = total;
  return GD_OK;
}

int gd_sampled_capacity(const uint64_t* layer_off, uint32_t n_layers, int scope_mode, uint32_t drop_ppm,
                        uint64_t* capacity_out) {
  if (!capacity_out) return GD_ERR_INVALID_ARG;
  try {
    Plan P;
    int rc = make_plan(layer_off, n_layers, nullptr, 1, scope_mode, drop_ppm, GD_FLAG_SAMPLED_THRESHOLD, &P);
    if (rc != GD_OK) return rc;
    *capacity_out = P.cand_total;
    return GD_OK;
  } catch (const std::bad_alloc&) {
    return GD_ERR_INVALID_ARG;
  }
}

int gd_means_pairs(uint32_t n_layers, const uint32_t* layer_cols, int value_mode, uint64_t* pairs_out) {
  if (!pairs_out) return GD_ERR_INVALID_ARG;
  if (value_mode == GD_VALUES_FP32) { *pairs_out = 0; return GD_OK; }
  if (value_mode == GD_VALUES_TWO_MEANS || value_mode == GD_VALUES_THRESHOLD) { *pairs_out = n_layers; return GD_OK; }
  if (value_mode != GD_VALUES_COLUMN_MEANS || !layer_cols) return GD_ERR_INVALID_ARG;
  uint64_t total = 0;
  for (uint32_t l = 0; l < n_layers; ++l) {
    if (layer_cols[l] == 0) return GD_ERR_INVALID_ARG;
    total += layer_cols[l];
  }
  *pairs_out = total;
  return GD_OK;
}

int gd_workspace_bytes(const uint64_t* layer_off, uint32_t n_layers, const uint32_t* layer_cols, uint32_t n_shards,
                       int scope_mode, uint32_t drop_ppm, size_t* bytes_out) {
  if (!bytes_out) return GD_ERR_INVALID_ARG;
  try {
    size_t most = 0;                                       // whichever mode is used
    for (uint32_t flags : {0u, (uint32_t)GD_FLAG_SAMPLED_THRESHOLD, (uint32_t)GD_FLAG_NO_PREDICTION}) {
      Plan P;
      int rc = make_plan(layer_off, n_layers, layer_cols, n_shards, scope_mode, drop_ppm, flags, &P);
      if (rc != GD_OK) return rc;
      if (P.total_bytes > most) most = P.total_bytes;
    }
    *bytes_out = most;
    return GD_OK;
  } catch (const std::bad_alloc&) {
    return GD_ERR_INVALID_ARG;
  }
}

int gd_compress(const gd_compress_args* a, void* stream_v) {
  NvtxRange range("gd_compress");
  if (!a) return GD_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)stream_v;
  try {
    Plan P;
    if (a->value_mode == GD_VALUES_COLUMN_MEANS && !a->layer_cols) return GD_ERR_INVALID_ARG;
    int rc = make_plan(a->layer_off, a->n_layers, a->value_mode == GD_VALUES_COLUMN_MEANS ? a->layer_cols : nullptr,
                       a->n_shards, a->scope_mode, a->drop_ppm, a->flags, &P);
    if (rc != GD_OK) return rc;
    uint64_t n_sh = 0;
    rc = check_offsets(a->shard_off, a->n_shards, &n_sh);
    if (rc != GD_OK) return rc;
    const uint64_t n = a->layer_off[a->n_layers];
    if (n_sh != n || a->n != n) return GD_ERR_INVALID_ARG;
    if (a->value_mode < GD_VALUES_FP32 || a->value_mode > GD_VALUES_COLUMN_MEANS) return GD_ERR_INVALID_ARG;
    if (a->value_mode != GD_VALUES_FP32 && n > (1ull << 31)) return GD_ERR_TOO_LARGE;
    if (a->flags & ~(uint32_t)(GD_FLAG_NO_PREDICTION | GD_FLAG_SAMPLED_THRESHOLD | GD_FLAG_QUANT_ERROR_FEEDBACK |
                               GD_FLAG_NO_EARLY_ZERO | GD_FLAG_PLAIN_RADIX))
      return GD_ERR_INVALID_ARG;
    if ((a->flags & GD_FLAG_QUANT_ERROR_FEEDBACK) && a->value_mode == GD_VALUES_FP32) return GD_ERR_INVALID_ARG;
    const bool sampled = (a->flags & GD_FLAG_SAMPLED_THRESHOLD) != 0;
    if (sampled && ((a->flags & GD_FLAG_NO_PREDICTION) || a->value_mode != GD_VALUES_FP32)) return GD_ERR_INVALID_ARG;
    if (n && (!a->grad || !a->residual)) return GD_ERR_INVALID_ARG;
    if (((uintptr_t)a->grad | (uintptr_t)a->residual) & 15u) return GD_ERR_INVALID_ARG;
    if (a->delta_base && (a->value_mode != GD_VALUES_FP32 || ((uintptr_t)a->delta_base & 15u))) return GD_ERR_INVALID_ARG;
    if (!a->out_shard_cnt_off) return GD_ERR_INVALID_ARG;
    if ((P.k_total || (sampled && P.cand_total)) && !a->out_idx) return GD_ERR_INVALID_ARG;
    if (P.k_total && a->value_mode == GD_VALUES_FP32 && !a->out_val) return GD_ERR_INVALID_ARG;
    if (a->value_mode != GD_VALUES_FP32 && !a->out_means) return GD_ERR_INVALID_ARG;
    if (!a->workspace || ((uintptr_t)a->workspace & (kAlign - 1))) return GD_ERR_WORKSPACE;
    if (a->workspace_bytes < P.total_bytes) return GD_ERR_WORKSPACE;

    // host image of the tables
    std::vector<unsigned char> blob(P.tables_bytes, 0);
    std::memcpy(blob.data() + P.t_scopes, P.scopes.data(), sizeof(ScopeDesc) * P.n_scopes);
    for (int l = 0; l < L_COUNT; ++l)
      std::memcpy(blob.data() + P.t_tile0[l], P.tile0[l].data(), sizeof(uint32_t) * (P.n_scopes + 1));
    std::memcpy(blob.data() + P.t_samp_off, P.samp_off.data(), sizeof(uint64_t) * (P.n_scopes + 1));
    std::memcpy(blob.data() + P.t_layer_off, a->layer_off, sizeof(uint64_t) * ((size_t)a->n_layers + 1));
    std::memcpy(blob.data() + P.t_shard_off, a->shard_off, sizeof(uint64_t) * ((size_t)a->n_shards + 1));
    std::memcpy(blob.data() + P.t_pair_off, P.pair_off.data(), sizeof(uint64_t) * ((size_t)a->n_layers + 1));
    std::memcpy(blob.data() + P.t_layer_cols, P.layer_cols.data(), sizeof(uint32_t) * (size_t)a->n_layers);

    unsigned char* ws = (unsigned char*)a->workspace;
    DevTables T;
    std::memset(&T, 0, sizeof(T));
    T.grad = a->grad;
    T.residual = a->residual;
    T.delta_base = a->delta_base;
    T.n = n;
    T.n_scopes = P.n_scopes;
    T.n_layers = a->n_layers;
    T.n_shards = a->n_shards;
    T.flags = P.predict ? a->flags : (a->flags | GD_FLAG_NO_PREDICTION);
    T.value_mode = a->value_mode;
    T.k_total = P.k_total;
    T.emit_chunk_tiles = P.emit_chunk_tiles;
    T.sample_passes = sampled ? 3u : 2u;
    T.samp_tile = P.samp_tile;
    T.dense_sel_tile = P.dense_sel_tile;
    T.dense_chunk_tiles = P.dense_chunk_tiles;
    if (sampled) T.k_total = P.cand_total;   // capacity of the outputs; the count is found on the device
    T.ctl = (Ctl*)(ws + P.off_ctl);
    T.state = (ScopeState*)(ws + P.off_state);
    T.hist = (unsigned long long*)(ws + P.off_hist);
    T.sums = (double*)(ws + P.off_sums);
    T.cnts = (unsigned long long*)(ws + P.off_cnts);
    T.desc_emit = (uint64_t*)(ws + P.off_desc_emit);
    T.desc_cand = (uint64_t*)(ws + P.off_desc_cand);
    T.desc_dcomp = (uint64_t*)(ws + P.off_desc_dcomp);
    const unsigned char* tb = ws + P.off_tables;
    T.scopes = (const ScopeDesc*)(tb + P.t_scopes);
    for (int l = 0; l < L_COUNT; ++l) T.tile0[l] = (const uint32_t*)(tb + P.t_tile0[l]);
    T.samp_off = (const uint64_t*)(tb + P.t_samp_off);
    T.layer_off = (const uint64_t*)(tb + P.t_layer_off);
    T.shard_off = (const uint64_t*)(tb + P.t_shard_off);
    T.pair_off = (const uint64_t*)(tb + P.t_pair_off);
    T.layer_cols = (const uint32_t*)(tb + P.t_layer_cols);
    T.n_pairs = P.n_pairs;
    T.cta_agg = ws + P.off_agg;
    T.samp_val = (float*)(ws + P.off_samp);
    T.cand_idx = (uint32_t*)(ws + P.off_cand_idx);
    T.cand_val = (float*)(ws + P.off_cand_val);
    T.out_idx = a->out_idx;
    T.out_val = a->out_val;
    T.out_shard_cnt_off = a->out_shard_cnt_off;
    T.out_tau = a->out_tau;
    T.out_means = a->out_means;

    uint32_t tiles[L_COUNT];
    for (int l = 0; l < L_COUNT; ++l) tiles[l] = P.tiles[l];
    // The start of the call (clearing the control region, writing the tables) shares a launch with the prediction
    // when every scope's sample is small enough for one CTA; otherwise it is a launch of its own.
    const bool local_predict = P.local_predict;
    if (local_predict) {
      if (launch_setup_predict(T, tiles[L_SAMP], P.samp_tile, (uint32_t*)(ws + P.off_flags), ws + P.off_tables, blob.data(), P.tables_bytes, ws, P.zero_bytes, P.off_state,
                               P.t_scopes, P.t_tile0[L_SAMP], stream) != cudaSuccess)
        return GD_ERR_CUDA;
    } else if (launch_setup(ws + P.off_tables, blob.data(), P.tables_bytes, ws, P.zero_bytes, stream) != cudaSuccess) {
      return GD_ERR_CUDA;
    }
    if (sampled) {
      if (launch_sample_select(T, tiles, stream) != cudaSuccess) return GD_ERR_CUDA;
      if (launch_add_emit(T, tiles, stream) != cudaSuccess) return GD_ERR_CUDA;
      if (launch_pack_sampled(T, tiles, stream) != cudaSuccess) return GD_ERR_CUDA;
      return GD_OK;
    }
    const bool predict = P.predict;
    if (predict && !local_predict && launch_sample_select(T, tiles, stream) != cudaSuccess) return GD_ERR_CUDA;
    if (predict && launch_add_emit(T, tiles, stream) != cudaSuccess) return GD_ERR_CUDA;
    // Without a prediction: the selection and compaction over the dense range.  With one: the two kernels over
    // the candidate lists, which first do the dense work of the scopes whose prediction failed (usually none).
    // The compaction that runs last also finishes the call (thresholds, shard offsets, means).
    if (P.dense_bound) {
      // histogram pass over grad + residual -> exact lower bounds -> the usual fused pass and the kernel over the lists
      if (launch_dense_bound(T, tiles, stream) != cudaSuccess) return GD_ERR_CUDA;
      DevTables U = T;
      U.flags = (T.flags & ~(uint32_t)GD_FLAG_NO_PREDICTION) | GD_FLAG_NO_EARLY_ZERO | kFlagDenseBound;
      if (launch_add_emit(U, tiles, stream) != cudaSuccess) return GD_ERR_CUDA;
      if (launch_select_compact(U, tiles, P.cand_total, stream) != cudaSuccess) return GD_ERR_CUDA;
    } else if (!predict) {
      if (launch_add_emit(T, tiles, stream) != cudaSuccess) return GD_ERR_CUDA;
      if (launch_dense_select(T, tiles, stream) != cudaSuccess) return GD_ERR_CUDA;
      if (launch_compact(T, tiles, true, true, stream) != cudaSuccess) return GD_ERR_CUDA;
    } else if (P.n_scopes <= kSmemScopes) {
      // selection among the candidates and compaction in one cooperative launch
      if (launch_select_compact(T, tiles, P.cand_total, stream) != cudaSuccess) return GD_ERR_CUDA;
    } else {
      if (launch_candidate_select(T, tiles, stream) != cudaSuccess) return GD_ERR_CUDA;
      if (launch_compact(T, tiles, false, true, stream) != cudaSuccess) return GD_ERR_CUDA;
    }
    if ((a->value_mode == GD_VALUES_TWO_MEANS || a->value_mode == GD_VALUES_COLUMN_MEANS) && P.n_pairs > kInlineMeansPairs &&
        launch_means(T, stream) != cudaSuccess)
      return GD_ERR_CUDA;
    if ((a->flags & GD_FLAG_QUANT_ERROR_FEEDBACK) && launch_feedback(T, stream) != cudaSuccess) return GD_ERR_CUDA;
    return GD_OK;
  } catch (const std::bad_alloc&) {
    return GD_ERR_INVALID_ARG;
  }
}

int gd_residual_reset(float* residual, uint64_t n, void* stream) {
  if (n == 0) return GD_OK;
  if (!residual) return GD_ERR_INVALID_ARG;
  if (cudaMemsetAsync(residual, 0, sizeof(float) * n, (cudaStream_t)stream) != cudaSuccess) return GD_ERR_CUDA;
  return GD_OK;
}

int gd_get_stats(const void* workspace, void* stream, gd_stats* out) {
  if (!workspace || !out) return GD_ERR_INVALID_ARG;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return GD_ERR_CUDA;
  Ctl c;
  if (cudaMemcpy(&c, workspace, sizeof(Ctl), cudaMemcpyDeviceToHost) != cudaSuccess) return GD_ERR_CUDA;
  out->status = c.status;
  out->n_scopes = c.n_scopes;
  out->n_scopes_predicted = c.n_scopes_predicted;
  out->n_scopes_dense = c.n_scopes_dense;
  out->n_candidates = c.n_candidates;
  out->n_kept = c.n_kept;
  return GD_OK;
}

int gd_status(const void* workspace, void* stream) {
  gd_stats s;
  int rc = gd_get_stats(workspace, stream, &s);
  return rc != GD_OK ? rc : s.status;
}

// Scratch of gd_compress_static: lives in the library's device image, one copy per GPU that loads it.
static __device__ __align__(256) unsigned char g_static_workspace[GD_STATIC_WORKSPACE_BYTES];

int gd_compress_static(const gd_compress_args* a, void* stream, const void** workspace_out) {
  if (!a) return GD_ERR_INVALID_ARG;
  size_t need = 0;
  int rc = gd_workspace_bytes(a->layer_off, a->n_layers, a->value_mode == GD_VALUES_COLUMN_MEANS ? a->layer_cols : nullptr,
                              a->n_shards, a->scope_mode, a->drop_ppm, &need);
  if (rc != GD_OK) return rc;
  if (need > (size_t)GD_STATIC_WORKSPACE_BYTES) return GD_ERR_TOO_LARGE;
  // In host code g_static_workspace is only a handle: its device address has to be asked for, once
  // per device, with that device current.
  constexpr int kMaxDevices = 64;
  static void* scratch_of_device[kMaxDevices] = {nullptr};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GD_ERR_CUDA;
  if (!scratch_of_device[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_workspace) != cudaSuccess || !p) return GD_ERR_CUDA;
    scratch_of_device[dev] = p;
  }
  gd_compress_args b = *a;
  b.workspace = scratch_of_device[dev];
  b.workspace_bytes = (size_t)GD_STATIC_WORKSPACE_BYTES;
  if (workspace_out) *workspace_out = b.workspace;
  return gd_compress(&b, stream);
}

int gd_profile_enable(int mode) {
  if (mode < 0 || mode > 2) return GD_ERR_INVALID_ARG;
  g_profile_mode = mode;
  if (mode == 0) g_ev_used = 0;
  return GD_OK;
}

int gd_profile_collect(float* ms_out, uint32_t* tags_out, uint32_t capacity, uint32_t* count_out) {
  if (!count_out || (capacity && !ms_out)) return GD_ERR_INVALID_ARG;
  uint32_t w = 0;
  int rc = GD_OK;
  for (uint32_t i = 0; i < g_ev_used; ++i) {
    float ms = 0.f;
    if (cudaEventSynchronize(g_ev_end[i]) != cudaSuccess ||
        cudaEventElapsedTime(&ms, g_ev_begin[i], g_ev_end[i]) != cudaSuccess) {
      rc = GD_ERR_CUDA;
      break;
    }
    if (w < capacity) {
      ms_out[w] = ms;
      if (tags_out) tags_out[w] = g_ev_tag[i];
      ++w;
    }
  }
  g_ev_used = 0;
  *count_out = w;
  return rc;
}

int gd_selftest_bounded_wait(void* workspace, size_t workspace_bytes, uint32_t spin_limit, void* stream) {
  if (!workspace || ((uintptr_t)workspace & (kAlign - 1)) || workspace_bytes < 512) return GD_ERR_WORKSPACE;
  if (spin_limit == 0 || spin_limit > kLookbackSpinLimit) return GD_ERR_INVALID_ARG;
  if (launch_bounded_wait_selftest(workspace, spin_limit, (cudaStream_t)stream) != cudaSuccess) return GD_ERR_CUDA;
  return GD_OK;
}

int gd_launch_count(uint64_t* count_out) {
  if (!count_out) return GD_ERR_INVALID_ARG;
  *count_out = g_launches.load(std::memory_order_relaxed);
  return GD_OK;
}

int gd_step_host(const gd_compress_args* a, const gd_apply_args* apply, const gd_host_io* io, void* stream_v) {
  if (!a || !io || !io->grad_host) return GD_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)stream_v;
  uint64_t k_total = 0;
  int rc = (a->flags & GD_FLAG_SAMPLED_THRESHOLD)
               ? gd_sampled_capacity(a->layer_off, a->n_layers, a->scope_mode, a->drop_ppm, &k_total)
               : gd_total_kept(a->layer_off, a->n_layers, a->scope_mode, a->drop_ppm, &k_total);
  if (rc != GD_OK) return rc;
  if (a->n && cudaMemcpyAsync((void*)a->grad, io->grad_host, sizeof(float) * a->n, cudaMemcpyHostToDevice, stream) !=
                  cudaSuccess)
    return GD_ERR_CUDA;
  rc = gd_compress(a, stream_v);
  if (rc != GD_OK) return rc;
  if (apply) {
    rc = gd_decompress_apply(apply, stream_v);
    if (rc != GD_OK) return rc;
  }
  cudaError_t e = cudaSuccess;
  if (io->idx_host && k_total)
    e = cudaMemcpyAsync(io->idx_host, a->out_idx, sizeof(uint32_t) * k_total, cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess && io->val_host && k_total && a->value_mode == GD_VALUES_FP32)
    e = cudaMemcpyAsync(io->val_host, a->out_val, sizeof(float) * k_total, cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess && io->shard_cnt_off_host)
    e = cudaMemcpyAsync(io->shard_cnt_off_host, a->out_shard_cnt_off, sizeof(uint32_t) * ((size_t)a->n_shards + 1),
                        cudaMemcpyDeviceToHost, stream);
  uint64_t pairs = 0;
  if (io->means_host && gd_means_pairs(a->n_layers, a->layer_cols, a->value_mode, &pairs) != GD_OK) return GD_ERR_INVALID_ARG;
  if (e == cudaSuccess && io->means_host && a->value_mode != GD_VALUES_FP32)
    e = cudaMemcpyAsync(io->means_host, a->out_means, sizeof(float) * 2 * (size_t)pairs, cudaMemcpyDeviceToHost, stream);
  if (e != cudaSuccess) return GD_ERR_CUDA;
  return gd_status(a->workspace, stream_v);
}

}  // extern "C"
