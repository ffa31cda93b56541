// Host side of libgd.so: argument checks, the per-call plan (scopes, tile tables, workspace
// layout) and the C entry points declared in include/gd.h.
#include <atomic>
#include <cmath>
#include <cstring>
#include <memory>
#include <mutex>
#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "gd_internal.cuh"
#include "gd_plan.hpp"

namespace gd {

namespace {

// Start of a call in one launch: clears the control region of the workspace and writes the small
// host-built tables, which travel as a kernel argument, behind it.

__global__ void __launch_bounds__(kThreads) setup_kernel(const __grid_constant__ SetupBlob blob, uint4* tables_dst,
                                                         uint32_t tables_vec, uint4* zero_dst, uint64_t zero_vec) {
  pdl_trigger();
  pdl_wait();      // (may have been brought onto the GPU early: see launch_dependent)
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
int g_profile_mode = 0;   // 0 off, 1 the pass over the dense vector only, 2 every kernel
cudaEvent_t g_ev_begin[kProfilePairs], g_ev_end[kProfilePairs];
uint32_t g_ev_tag[kProfilePairs];
uint32_t g_ev_created = 0, g_ev_used = 0;
bool g_pair_open = false;
std::atomic<uint64_t> g_launches{0};   // calls may come from several host threads

// Plans are pure functions of the layout arguments and are kept: a training loop calls with the same layout every
// step, and should not pay for vectors, square roots and table images again.  Entries are immutable once stored and
// never dropped (a full cache just stops caching), so a pointer to one stays valid.
struct PlanEntry {
  std::vector<uint64_t> layer_off, shard_off;
  std::vector<uint32_t> layer_cols;
  int scope_mode = 0;
  uint32_t drop_ppm = 0, plan_flags = 0;
  uint64_t fused_units = 0;             // what the device the plan was made for takes in one launch (part of the key)
  Plan P;
  std::vector<unsigned char> blob;      // host image of the tables
  unsigned char* pinned = nullptr;      // the same in page-locked memory, for tables too large for a kernel argument
};
constexpr size_t kPlanCacheEntries = 64;
std::mutex g_plan_mutex;
std::vector<std::unique_ptr<PlanEntry>> g_plans;

bool same_layout(const PlanEntry& e, const gd_compress_args* a, const uint32_t* cols, uint32_t plan_flags, uint64_t fused_units) {
  if (e.scope_mode != a->scope_mode || e.drop_ppm != a->drop_ppm || e.plan_flags != plan_flags || e.fused_units != fused_units) return false;
  if (e.layer_off.size() != (size_t)a->n_layers + 1 || e.shard_off.size() != (size_t)a->n_shards + 1) return false;
  if (e.layer_cols.empty() != (cols == nullptr)) return false;
  if (std::memcmp(e.layer_off.data(), a->layer_off, sizeof(uint64_t) * e.layer_off.size()) != 0) return false;
  if (std::memcmp(e.shard_off.data(), a->shard_off, sizeof(uint64_t) * e.shard_off.size()) != 0) return false;
  return !cols || std::memcmp(e.layer_cols.data(), cols, sizeof(uint32_t) * e.layer_cols.size()) == 0;
}

// The plan and table image for these arguments: from the cache, or built now (and stored if there is room).
// *owned receives the entry when it was not stored.  may_allocate: whether page-locked memory may be asked for.
int plan_for(const gd_compress_args* a, bool may_allocate, const PlanEntry** out, std::unique_ptr<PlanEntry>* owned) {
  if (!a->layer_off || !a->shard_off || a->n_layers == 0 || a->n_shards == 0) return GD_ERR_INVALID_ARG;
  const uint32_t* cols = a->value_mode == GD_VALUES_COLUMN_MEANS ? a->layer_cols : nullptr;
  const uint32_t plan_flags = a->flags & (GD_FLAG_NO_PREDICTION | GD_FLAG_SAMPLED_THRESHOLD | GD_FLAG_PREDICT_ALWAYS);
  const uint64_t fused_units = dense_fused_capacity();     // (of the current device: plans differ between unlike devices)
  {
    std::lock_guard<std::mutex> lock(g_plan_mutex);
    for (const auto& e : g_plans)
      if (same_layout(*e, a, cols, plan_flags, fused_units)) { *out = e.get(); return GD_OK; }
  }
  std::unique_ptr<PlanEntry> e(new PlanEntry);
  int rc = make_plan(a->layer_off, a->n_layers, cols, a->n_shards, a->scope_mode, a->drop_ppm, a->flags, &e->P, fused_units);
  if (rc != GD_OK) return rc;
  uint64_t n_sh = 0;
  rc = check_offsets(a->shard_off, a->n_shards, &n_sh);
  if (rc != GD_OK) return rc;
  if (n_sh != a->layer_off[a->n_layers]) return GD_ERR_INVALID_ARG;
  e->layer_off.assign(a->layer_off, a->layer_off + a->n_layers + 1);
  e->shard_off.assign(a->shard_off, a->shard_off + a->n_shards + 1);
  if (cols) e->layer_cols.assign(cols, cols + a->n_layers);
  e->scope_mode = a->scope_mode;
  e->drop_ppm = a->drop_ppm;
  e->plan_flags = plan_flags;
  e->fused_units = fused_units;
  const Plan& P = e->P;
  e->blob.assign(P.tables_bytes, 0);
  unsigned char* b = e->blob.data();
  std::memcpy(b + P.t_scopes, P.scopes.data(), sizeof(ScopeDesc) * P.n_scopes);
  for (int l = 0; l < L_COUNT; ++l) std::memcpy(b + P.t_tile0[l], P.tile0[l].data(), sizeof(uint32_t) * (P.n_scopes + 1));
  std::memcpy(b + P.t_samp_off, P.samp_off.data(), sizeof(uint64_t) * (P.n_scopes + 1));
  std::memcpy(b + P.t_layer_off, a->layer_off, sizeof(uint64_t) * ((size_t)a->n_layers + 1));
  std::memcpy(b + P.t_shard_off, a->shard_off, sizeof(uint64_t) * ((size_t)a->n_shards + 1));
  std::memcpy(b + P.t_pair_off, P.pair_off.data(), sizeof(uint64_t) * ((size_t)a->n_layers + 1));
  std::memcpy(b + P.t_layer_cols, P.layer_cols.data(), sizeof(uint32_t) * (size_t)a->n_layers);
  std::lock_guard<std::mutex> lock(g_plan_mutex);
  for (const auto& other : g_plans)                        // (another thread may have stored the same layout meanwhile)
    if (same_layout(*other, a, cols, plan_flags, fused_units)) { *out = other.get(); return GD_OK; }
  if (g_plans.size() < kPlanCacheEntries) {
    if (may_allocate && P.tables_bytes > kSetupBlobBytes) {
      void* p = nullptr;
      if (cudaHostAlloc(&p, P.tables_bytes, cudaHostAllocDefault) == cudaSuccess && p) {
        std::memcpy(p, b, P.tables_bytes);
        e->pinned = (unsigned char*)p;
      } else {
        (void)cudaGetLastError();                          // no page-locked image: the tables go up in pieces
      }
    }
    *out = e.get();
    g_plans.push_back(std::move(e));
  } else {
    *out = e.get();
    *owned = std::move(e);
  }
  return GD_OK;
}

}  // namespace

void note_launches(uint32_t count) { g_launches.fetch_add(count, std::memory_order_relaxed); }

// Writes `bytes` (a multiple of 16) of host data to device memory in pieces that travel as kernel arguments: no
// staging buffer, nothing that blocks the host, and the host data may be freed when the call returns.
cudaError_t upload_by_launches(void* dst, const void* src, size_t bytes, cudaStream_t stream) {
  SetupBlob blob;
  for (size_t off = 0; off < bytes; off += kSetupBlobBytes) {
    const size_t len = bytes - off < kSetupBlobBytes ? bytes - off : kSetupBlobBytes;
    std::memcpy(blob.bytes, (const unsigned char*)src + off, len);
    setup_kernel<<<1, kThreads, 0, stream>>>(blob, (uint4*)((unsigned char*)dst + off), (uint32_t)(len / 16), nullptr, 0);
    GD_LAUNCH_CHECK();
  }
  return cudaSuccess;
}

cudaError_t launch_setup(void* tables_dst, const void* tables_src, size_t tables_bytes, void* zero_dst, size_t zero_bytes,
                         cudaStream_t stream, bool src_is_pinned) {
  ProfileScope prof(stream, PT_SETUP);
  const uint64_t zero_vec = zero_bytes / 16;   // both regions are 256-byte aligned and padded
  uint64_t blocks = (zero_vec + kThreads * 8 - 1) / (kThreads * 8);
  const uint64_t cap = (uint64_t)sm_count() * 4;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  // Tables of up to kSetupBlobBytes travel with the launch that clears the control region.  Larger ones (models
  // with many tensors) are copied from the page-locked image kept with the cached plan - an asynchronous copy -
  // or, where there is no such image, in pieces by further launches.  Never from pageable memory: that copy would
  // block the host and could not be captured.
  SetupBlob blob;
  const size_t first = tables_bytes <= kSetupBlobBytes ? tables_bytes : (src_is_pinned ? 0 : kSetupBlobBytes);
  std::memcpy(blob.bytes, tables_src, first);
  const cudaError_t le = launch_dependent(setup_kernel, dim3((unsigned)blocks), dim3(kThreads), 0, stream, blob, (uint4*)tables_dst,
                                          (uint32_t)(first / 16), (uint4*)zero_dst, zero_vec);
  if (le != cudaSuccess) return le;
  GD_LAUNCH_CHECK();
  if (first == tables_bytes) return cudaSuccess;
  if (src_is_pinned) return cudaMemcpyAsync(tables_dst, tables_src, tables_bytes, cudaMemcpyHostToDevice, stream);
  return upload_by_launches((unsigned char*)tables_dst + first, (const unsigned char*)tables_src + first, tables_bytes - first,
                            stream);
}

int sm_count() {
  static PerDeviceInt cached;
  int dev = -1;
  int sms = cached.get(&dev);
  if (sms > 0) return sms;
  if (dev < 0 && cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return 148;   // B200; only sizes grids
  if (dev < kMaxDevices) cached.set(dev, sms);
  return sms;
}

void profile_mark(cudaStream_t stream, bool begin, uint32_t tag) {
  if (g_profile_mode == 0 || (g_profile_mode == 1 && tag != PT_ADD_EMIT && tag != PT_DENSE_FUSED)) return;
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
    size_t most = 0;                                       // whichever mode is used, on whichever device
    for (uint32_t flags : {0u, (uint32_t)GD_FLAG_SAMPLED_THRESHOLD, (uint32_t)GD_FLAG_NO_PREDICTION, (uint32_t)GD_FLAG_PREDICT_ALWAYS}) {
      for (uint64_t fused_units : {(uint64_t)0, ~(uint64_t)0}) {
        Plan P;
        int rc = make_plan(layer_off, n_layers, layer_cols, n_shards, scope_mode, drop_ppm, flags, &P, fused_units);
        if (rc != GD_OK) return rc;
        if (P.total_bytes > most) most = P.total_bytes;
      }
    }
    *bytes_out = most;
    return GD_OK;
  } catch (const std::bad_alloc&) {
    return GD_ERR_INVALID_ARG;
  }
}

namespace {

int compress_impl(const gd_compress_args* a, void* stream_v, bool may_allocate) {
  NvtxRange range("gd_compress");
  if (!a) return GD_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)stream_v;
  try {
    if (a->value_mode == GD_VALUES_COLUMN_MEANS && !a->layer_cols) return GD_ERR_INVALID_ARG;
    const PlanEntry* entry = nullptr;
    std::unique_ptr<PlanEntry> owned;
    int rc = plan_for(a, may_allocate, &entry, &owned);
    if (rc != GD_OK) return rc;
    const Plan& P = entry->P;
    const uint64_t n = a->layer_off[a->n_layers];
    if (a->n != n) return GD_ERR_INVALID_ARG;
    if (a->value_mode < GD_VALUES_FP32 || a->value_mode > GD_VALUES_COLUMN_MEANS) return GD_ERR_INVALID_ARG;
    if (a->value_mode != GD_VALUES_FP32 && n > (1ull << 31)) return GD_ERR_TOO_LARGE;
    if (a->flags & ~(uint32_t)(GD_FLAG_NO_PREDICTION | GD_FLAG_SAMPLED_THRESHOLD | GD_FLAG_QUANT_ERROR_FEEDBACK |
                               GD_FLAG_NO_EARLY_ZERO | GD_FLAG_PLAIN_RADIX | GD_FLAG_PREDICT_ALWAYS))
      return GD_ERR_INVALID_ARG;
    if ((a->flags & GD_FLAG_NO_PREDICTION) && (a->flags & GD_FLAG_PREDICT_ALWAYS)) return GD_ERR_INVALID_ARG;
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
    const unsigned char* tables_image = entry->pinned ? entry->pinned : entry->blob.data();
    const bool image_is_pinned = entry->pinned != nullptr;

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
    EmitEarly early;
    const EmitEarly* early_ptr = nullptr;
    // (short vectors: the one launch that does everything also starts the call, where the tables fit its argument)
    const bool fused_starts = P.dense_fused && !sampled && P.tables_bytes <= kSetupBlobBytes && P.zero_bytes != 0;
    if (fused_starts) {
    } else if (local_predict) {
      uint32_t call = 0, clearing_ctas = 0;
      if (launch_setup_predict(T, tiles[L_SAMP], P.samp_tile, (uint32_t*)(ws + P.off_flags), ws + P.off_tables, tables_image, P.tables_bytes, ws, P.zero_bytes, P.off_state,
                               P.t_scopes, P.t_tile0[L_SAMP], stream, &call, &clearing_ctas) != cudaSuccess)
        return GD_ERR_CUDA;
      // the fused pass may start while that launch is still selecting: it gets the tables itself and waits only for
      // the marks of what it is about to use (at most 32 scopes)
      if (P.n_scopes <= kSmemScopes) {
        early.tables_src = tables_image;
        early.tables_bytes = P.tables_bytes;
        early.scopes_off = P.t_scopes;
        early.tile0_emit_off = P.t_tile0[L_EMIT];
        early.ready = (const uint32_t*)(ws + P.off_flags) + tiles[L_SAMP];
        early.cleared = early.ready + kSmemScopes;
        early.call = call;
        early.clearing_ctas = clearing_ctas;
#ifndef GD_NO_EARLY
        early_ptr = &early;
#endif
      }
    } else if (launch_setup(ws + P.off_tables, tables_image, P.tables_bytes, ws, P.zero_bytes, stream, image_is_pinned) != cudaSuccess) {
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
    if (predict && launch_add_emit(T, tiles, stream, early_ptr) != cudaSuccess) return GD_ERR_CUDA;
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
      // short vectors: add, select and compact over the dense range in one cooperative launch where the vector
      // fits its CTAs' shared memory and the scopes its tables (the plan says); else the three separate kernels
      if (P.dense_fused) {
        if (launch_dense_fused(T, P.dense_units, stream, ws + P.off_tables, fused_starts ? tables_image : nullptr, P.tables_bytes, ws,
                               P.zero_bytes) != cudaSuccess)
          return GD_ERR_CUDA;
      } else {
        if (launch_add_emit(T, tiles, stream) != cudaSuccess) return GD_ERR_CUDA;
        if (launch_dense_select(T, tiles, stream) != cudaSuccess) return GD_ERR_CUDA;
        if (launch_compact(T, tiles, true, true, stream) != cudaSuccess) return GD_ERR_CUDA;
      }
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

}  // namespace

int gd_compress(const gd_compress_args* a, void* stream) { return compress_impl(a, stream, true); }

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
  if (a->value_mode == GD_VALUES_COLUMN_MEANS && !a->layer_cols) return GD_ERR_INVALID_ARG;
  const PlanEntry* entry = nullptr;
  std::unique_ptr<PlanEntry> owned;
  int rc;
  try {
    rc = plan_for(a, false, &entry, &owned);
  } catch (const std::bad_alloc&) {
    return GD_ERR_INVALID_ARG;
  }
  if (rc != GD_OK) return rc;
  if (entry->P.total_bytes > (size_t)GD_STATIC_WORKSPACE_BYTES) return GD_ERR_TOO_LARGE;   // what THIS call needs
  // In host code g_static_workspace is only a handle: its device address has to be asked for, once
  // per device, with that device current.
  static std::atomic<void*> scratch_of_device[kMaxDevices];
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GD_ERR_CUDA;
  void* scratch = scratch_of_device[dev].load(std::memory_order_acquire);
  if (!scratch) {
    if (cudaGetSymbolAddress(&scratch, g_static_workspace) != cudaSuccess || !scratch) return GD_ERR_CUDA;
    scratch_of_device[dev].store(scratch, std::memory_order_release);   // (two threads may both ask: same answer)
  }
  gd_compress_args b = *a;
  b.workspace = scratch;
  b.workspace_bytes = (size_t)GD_STATIC_WORKSPACE_BYTES;
  if (workspace_out) *workspace_out = b.workspace;
  return compress_impl(&b, stream, false);   // (nothing is allocated on this path, page-locked host memory included)
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
  // the waits on mbarriers (the pipelined fused pass) are bounded by time: 100 ns per poll of the other limit
  if (launch_mbar_wait_selftest(workspace, 100ull * spin_limit, (cudaStream_t)stream) != cudaSuccess) return GD_ERR_CUDA;
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
