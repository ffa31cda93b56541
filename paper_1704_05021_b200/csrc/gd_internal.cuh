// Shared declarations of the gradient-dropping kernels (device tables, workspace layout,
// small PTX helpers).  Internal to libgd.so; the public interface is include/gd.h.
#pragma once

#include <atomic>
#include <utility>

#include <cuda_runtime.h>
#include <stdint.h>

#include "gd_layout.h"

namespace gd {

#define GD_LAUNCH_CHECK()                         \
  do {                                            \
    cudaError_t e_ = cudaPeekAtLastError();       \
    if (e_ != cudaSuccess) return e_;             \
    note_launches(1);                             \
  } while (0)

struct DevTables {       // passed by value to every kernel
  const float* grad;
  float* residual;
  float* delta_base;                 // delta mode: v = grad - delta_base, survivors are added back to it
  uint64_t n;
  uint32_t n_scopes, n_layers, n_shards;
  uint32_t flags;
  int32_t value_mode;
  uint32_t emit_chunk_tiles;         // tiles of kTile elements one CTA of the fused pass streams (1, 2, 4 or 8)
  uint32_t sample_passes;            // radix passes over the sample: 2 (prediction, 21 bits) or 3 (sampled-threshold mode)
  uint32_t dense_sel_tile;           // elements per tile of the dense selection (4096 .. 32768, by vector length)
  uint32_t dense_chunk_tiles;        // tiles per chunk of the dense compaction (1 .. 16, by vector length)
  uint32_t samp_tile;                // samples per tile of the sample selection (1024 for short samples, else 4096)
  uint64_t k_total;
  // zeroed region
  Ctl* ctl;
  ScopeState* state;
  unsigned long long* hist;          // [n_scopes][kHistBinsPerScope]
  double* sums;                      // [n_pairs][2]
  unsigned long long* cnts;          // [n_pairs][2]
  uint64_t* desc_emit;               // [tiles(L_EMIT)]
  uint64_t* desc_cand;               // [tiles(L_CAND)][2]
  uint64_t* desc_dcomp;              // [tiles(L_DCOMP)][2]
  // uploaded tables
  const ScopeDesc* scopes;           // [n_scopes]
  const uint32_t* tile0[L_COUNT];    // [n_scopes + 1] first tile of each scope per launch kind
  const uint64_t* samp_off;          // [n_scopes + 1]
  const uint64_t* layer_off;         // [n_layers + 1]
  const uint64_t* shard_off;         // [n_shards + 1]
  const uint64_t* pair_off;          // [n_layers + 1] first (mu+, mu-) pair of each layer
  const uint32_t* layer_cols;        // [n_layers] columns per layer (1 unless column-means mode)
  uint64_t n_pairs;                  // pairs in total
  // buffers
  void* cta_agg;                     // [grid] per-CTA survivor counts of the kernel that selects and compacts in one launch
  float* samp_val;
  uint32_t* cand_idx;
  float* cand_val;
  // outputs
  uint32_t* out_idx;
  float* out_val;
  uint32_t* out_shard_cnt_off;
  uint32_t* out_tau;
  float* out_means;
};

// ---------------------------------------------------------------- programmatic dependent launches
// A kernel launched with launch_dependent() may be brought onto the GPU while the kernel before it in the stream is
// still running - from the moment all CTAs of that kernel have called pdl_trigger() (or ended) - so that its launch
// latency is spent then and not after.  It must call pdl_wait() before it reads or writes anything the earlier
// kernels of the stream touch: that returns when the kernel before it has completed and its writes are visible.
// Where the kernel before it does not trigger, or is no kernel at all, the launch is an ordinary one.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                    Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  static std::atomic<int> refused{0};                        // a driver that does not take the attribute: ordinary launches
  if (!refused.load(std::memory_order_relaxed)) {
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, args...);
    if (e != cudaErrorNotSupported && e != cudaErrorInvalidValue) return e;
    (void)cudaGetLastError();
    refused.store(1, std::memory_order_relaxed);
  }
  cfg.attrs = nullptr;
  cfg.numAttrs = 0;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// ---------------------------------------------------------------- device helpers
__device__ __forceinline__ uint32_t lane_id() { return threadIdx.x & 31u; }
__device__ __forceinline__ uint32_t lanemask_lt() {
  uint32_t m;
  asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
  return m;
}
__device__ __forceinline__ uint64_t pack_desc(uint64_t flag, uint64_t value) { return (value << 2) | flag; }
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// True when a wait that began at t0 (global_timer_ns) and has polled `spins` times should give up.
__device__ __forceinline__ bool wait_expired(uint32_t spins, uint32_t spin_limit, uint64_t t0, uint64_t budget_ns) {
  return spins > spin_limit && (budget_ns == 0 || global_timer_ns() - t0 > budget_ns);
}

// ---------------------------------------------------------------- mbarriers and bulk asynchronous copies
// (the untiled form of the TMA engine's copies: whole kilobytes per request, completion counted in bytes on an
// mbarrier in shared memory; both addresses 16-byte aligned, the size a multiple of 16)
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* b, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* b) {
  asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.shared::cta.b64 st, [%0];\n\t}" ::"r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* b, uint32_t bytes) {
  asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n\t}" ::"r"(smem_u32(b)), "r"(bytes)
               : "memory");
}
// Announces `bytes` of copies on b's current phase without arriving (the arrive follows separately).
__device__ __forceinline__ void mbar_expect_tx(uint64_t* b, uint32_t bytes) {
  asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* b, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok)
               : "r"(smem_u32(b)), "r"(parity)
               : "memory");
  return ok != 0u;
}
// Global -> shared bulk copy of `bytes` (a multiple of 16; both addresses 16-byte aligned), counted on mbarrier b.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* b) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(b))
               : "memory");
}

// Waits until the phase of parity `parity` of b has completed.  Gives up (false) when the CTA's abort flag is up or
// after kWaitBudgetNs.
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity, const volatile int* abort,
                                          uint64_t budget_ns = kWaitBudgetNs) {
  uint32_t spins = 0;
  uint64_t t0 = 0;
  while (!mbar_try_wait(b, parity)) {
    ++spins;
    if (spins == 32u) t0 = global_timer_ns();
    if (spins > 32u && (spins & 31u) == 0u) {
      if (*abort) return false;
      if (global_timer_ns() - t0 > budget_ns) return false;
    }
  }
  return true;
}


// Copy of the small per-call tables in shared memory: scope descriptors and the tile -> scope table
// of one launch kind.  With few scopes (the usual case) every later lookup is a shared-memory read
// instead of a chain of dependent global loads.
struct SmemTables {
  ScopeDesc scopes[kSmemScopes];
  uint32_t tile0[kSmemScopes + 1];
};

// Most scopes for which the kernels over the candidate lists number only the tiles that hold
// candidates (a table of this many counters in shared memory).
constexpr uint32_t kVtScopes = 2048;

// In-place inclusive prefix sum of a[0 .. n) in shared memory, by a whole CTA of kThreads threads.
// The caller synchronises between filling a[] and the call; the result is visible to all on return.
__device__ __forceinline__ void block_inclusive_scan(uint32_t* a, uint32_t n) {
  __shared__ uint32_t s_scan_warp[kThreads / 32];
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const uint32_t per = (n + kThreads - 1) / kThreads;
  const uint32_t b = tid * per < n ? tid * per : n;
  const uint32_t e = b + per < n ? b + per : n;
  uint32_t sum = 0;
  for (uint32_t i = b; i < e; ++i) sum += a[i];
  uint32_t inc = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
    if ((int)lane >= o) inc += y;
  }
  if (lane == 31u) s_scan_warp[warp] = inc;
  __syncthreads();
  uint32_t run = inc - sum;
  for (uint32_t w = 0; w < warp; ++w) run += s_scan_warp[w];
  for (uint32_t i = b; i < e; ++i) {
    run += a[i];
    a[i] = run;
  }
  __syncthreads();
}

// Number of entries of the ascending table base[0 .. count) that are <= t, counted by the whole CTA
// in one round of loads (a binary search would be a chain of dependent global loads).
__device__ __forceinline__ uint32_t block_count_le(const uint32_t* base, uint32_t count, uint32_t t) {
  __shared__ uint32_t s_cnt;
  if (threadIdx.x == 0) s_cnt = 0;
  __syncthreads();
  uint32_t c = 0;
  for (uint32_t i = threadIdx.x; i < count; i += blockDim.x) c += base[i] <= t ? 1u : 0u;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xFFFFFFFFu, c, o);
  if ((threadIdx.x & 31u) == 0 && c) atomicAdd(&s_cnt, c);
  __syncthreads();
  const uint32_t r = s_cnt;
  __syncthreads();
  return r;
}

// Called by all threads of a CTA; the caller synchronises before using the result.  Returns the
// tables to use: the shared copy when the scopes fit, else the global ones.
__device__ __forceinline__ void load_tables(const DevTables& T, int launch_kind, SmemTables* sm,
                                            const ScopeDesc** scopes, const uint32_t** tile0) {
  if (T.n_scopes <= kSmemScopes) {
    const uint32_t words = T.n_scopes * (uint32_t)(sizeof(ScopeDesc) / 8);
    const uint64_t* src = reinterpret_cast<const uint64_t*>(T.scopes);
    uint64_t* dst = reinterpret_cast<uint64_t*>(sm->scopes);
    for (uint32_t i = threadIdx.x; i < words; i += blockDim.x) dst[i] = src[i];
    for (uint32_t i = threadIdx.x; i <= T.n_scopes; i += blockDim.x) sm->tile0[i] = T.tile0[launch_kind][i];
    *scopes = sm->scopes;
    *tile0 = sm->tile0;
  } else {
    *scopes = T.scopes;
    *tile0 = T.tile0[launch_kind];
  }
}

// Largest s in [0, n_scopes) with tile0[s] <= t (tile0 has n_scopes + 1 entries, ascending; scopes
// without tiles repeat their successor's value, so the scope found is the one that owns tile t).
__device__ __forceinline__ uint32_t scope_of_tile(const uint32_t* __restrict__ tile0, uint32_t n_scopes, uint32_t t) {
  uint32_t lo = 0, hi = n_scopes;  // invariant: tile0[lo] <= t < tile0[hi]
  while (hi - lo > 1) {
    uint32_t mid = (lo + hi) >> 1;
    if (tile0[mid] <= t) lo = mid; else hi = mid;
  }
  return lo;
}

// Largest l in [0, count) with off[l] <= x, for ascending off[0..count] with off[0] <= x < off[count];
// entries that repeat (empty ranges) resolve to the last one, i.e. the non-empty range holding x.
__device__ __forceinline__ uint32_t range_of(const uint64_t* __restrict__ off, uint32_t count, uint64_t x) {
  uint32_t lo = 0, hi = count;
  while (hi - lo > 1) {
    uint32_t mid = (lo + hi) >> 1;
    if (off[mid] <= x) lo = mid; else hi = mid;
  }
  return lo;
}

// The (mu+, mu-) pair an index belongs to: its layer, or its layer and column (row-major layers).
__device__ __forceinline__ uint64_t pair_of(const uint64_t* __restrict__ layer_off, const uint64_t* __restrict__ pair_off,
                                            const uint32_t* __restrict__ layer_cols, uint32_t n_layers, uint64_t idx) {
  const uint32_t l = range_of(layer_off, n_layers, idx);
  const uint32_t cols = layer_cols[l];
  return pair_off[l] + (cols > 1 ? (idx - layer_off[l]) % cols : 0ull);
}

// Internal bit of DevTables::flags (never passed by a caller): the lower bounds of this call come from a histogram
// over the dense vector (gd_dense.cu), not from a sample; its scopes count as selected densely in the statistics.
constexpr uint32_t kFlagDenseBound = 1u << 31;

// True when the scope's result comes from the candidate list the fused pass emitted: the
// prediction was a valid lower bound (at least k candidates) and the list did not overflow.
__device__ __forceinline__ bool predicted_ok(const DevTables& T, const ScopeDesc& d, const ScopeState& st) {
  if (T.flags & GD_FLAG_NO_PREDICTION) return false;
  uint64_t m = st.cand_count;
  return m >= d.k && m <= d.cand_cap;
}

// Smallest key a candidate of the fused pass can have: the predicted lower bound, but never 0 (zeros are never
// candidates).  The candidates' first histogram counts D = key - this.
__device__ __forceinline__ uint32_t candidate_base_key(uint32_t tau_lo) { return tau_lo == 0u ? 1u : tau_lo; }
__device__ __forceinline__ uint32_t fine_bin(uint32_t key, uint32_t base) {
  const uint32_t b = (key - base) >> kFineShift;
  return b < kFineTop ? b : kFineTop;
}

// True when the fused pass writes +0 over the entries it expects to be kept (ScopeState::tau_hi).  Not
// with quantisation-error feedback (the kept slots must hold v until the decode table exists), not
// without a prediction.  (Sampled-threshold mode has its own, simpler form: every candidate is kept.)
__device__ __forceinline__ bool early_zero_enabled(const DevTables& T) {
  return (T.flags & (GD_FLAG_NO_PREDICTION | GD_FLAG_SAMPLED_THRESHOLD | GD_FLAG_QUANT_ERROR_FEEDBACK |
                     GD_FLAG_NO_EARLY_ZERO)) == 0u;
}

// The small host-built tables of a call travel to the device as a kernel argument.
struct SetupBlob {
  unsigned char bytes[kSetupBlobBytes];
};

// What lets the pipelined fused pass start before the setup-and-predict launch has ended: the tables in its own
// argument, and where that launch marks (with the call's number) the scopes whose predictions are final and the CTAs
// that have cleared their part of the control region.
struct EmitEarly {
  const void* tables_src;        // host image of the tables (at most kSetupBlobBytes)
  size_t tables_bytes, scopes_off, tile0_emit_off;
  const uint32_t* ready;         // [kSmemScopes]
  const uint32_t* cleared;       // [clearing_ctas]
  uint32_t call, clearing_ctas;
};
// Host-side launchers of the kernel groups (one per .cu file); `tiles` is indexed by Launch.
cudaError_t upload_by_launches(void* dst, const void* src, size_t bytes, cudaStream_t stream);
cudaError_t launch_setup(void* tables_dst, const void* tables_src, size_t tables_bytes, void* zero_dst, size_t zero_bytes,
                         cudaStream_t stream, bool src_is_pinned);
cudaError_t launch_setup_predict(const DevTables& T, uint32_t gather_ctas, uint32_t gather_tile, uint32_t* flags, void* tables_dst, const void* tables_src,
                                 size_t tables_bytes, void* zero_dst, size_t zero_bytes, size_t state_off, size_t scopes_off,
                                 size_t tile0_off, cudaStream_t stream, uint32_t* call_out, uint32_t* clearing_ctas_out);
cudaError_t launch_sample_select(const DevTables& T, const uint32_t* tiles, cudaStream_t stream);
cudaError_t launch_add_emit(const DevTables& T, const uint32_t* tiles, cudaStream_t stream, const EmitEarly* early = nullptr);
cudaError_t launch_candidate_select(const DevTables& T, const uint32_t* tiles, cudaStream_t stream);
cudaError_t launch_dense_select(const DevTables& T, const uint32_t* tiles, cudaStream_t stream);
cudaError_t launch_compact(const DevTables& T, const uint32_t* tiles, bool dense, bool finalize, cudaStream_t stream);
cudaError_t launch_finalize(const DevTables& T, cudaStream_t stream);
cudaError_t launch_means(const DevTables& T, cudaStream_t stream);
cudaError_t launch_feedback(const DevTables& T, cudaStream_t stream);
cudaError_t launch_pack_sampled(const DevTables& T, const uint32_t* tiles, cudaStream_t stream);
cudaError_t launch_select_compact(const DevTables& T, const uint32_t* tiles, uint64_t cand_total, cudaStream_t stream);
cudaError_t launch_dense_bound(const DevTables& T, const uint32_t* tiles, cudaStream_t stream);
bool add_emit_pipe_takes(const DevTables& T);        // the pipelined fused pass (gd_emit_pipe.cu) can take the call
cudaError_t launch_add_emit_pipe(const DevTables& T, const uint32_t* tiles, cudaStream_t stream, const EmitEarly* early);
cudaError_t launch_dense_fused(const DevTables& T, uint64_t dense_units, cudaStream_t stream, void* tables_dst,
                               const void* tables_src, size_t tables_bytes, void* zero_dst, size_t zero_bytes);
uint64_t dense_fused_capacity();   // how many 1024-element units launch_dense_fused takes on the current device (0: none)
cudaError_t launch_bounded_wait_selftest(void* workspace, uint32_t spin_limit, cudaStream_t stream);
cudaError_t launch_mbar_wait_selftest(void* workspace, uint64_t budget_ns, cudaStream_t stream);   // after the former: the workspace is prepared
int sm_count();   // multiprocessors of the current device (148 if it cannot be asked)
// A small per-device cache of one int (0 = not known yet), for values that belong to the device a call runs on:
// multiprocessor counts, how many CTAs of a kernel fit on one of them.  Devices beyond kMaxDevices are not cached.
constexpr int kMaxDevices = 64;
struct PerDeviceInt {
  std::atomic<int> v[kMaxDevices];
  // value for the current device, or 0; *dev_out: the device ordinal, or -1 if it cannot be cached
  int get(int* dev_out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { *dev_out = -1; return 0; }
    *dev_out = dev;
    return v[dev].load(std::memory_order_relaxed);
  }
  void set(int dev, int value) { if (dev >= 0) v[dev].store(value, std::memory_order_relaxed); }
};

// Measurement hooks (gd_api.cu): count a kernel launch; record an event of the pair around the fused pass.
void note_launches(uint32_t count);
// Kernel tags of the measurement hooks, in the order a step launches them.
enum ProfileTag : uint32_t { PT_SETUP = 0, PT_PACK_SAMPLED = 9, PT_MEANS = 10, PT_SAMPLE_SELECT = 1, PT_ADD_EMIT = 2, PT_DENSE_SELECT = 3, PT_DENSE_COMPACT = 4,
                             PT_CAND_SELECT = 5, PT_CAND_COMPACT = 6, PT_FINALIZE = 7, PT_APPLY = 8, PT_FEEDBACK = 11,
                             PT_CAND_SELECT_COMPACT = 12, PT_SETUP_PREDICT = 13,
                             PT_DENSE_HIST = 14, PT_DENSE_FIND = 15, PT_DENSE_FUSED = 16 };
void profile_mark(cudaStream_t stream, bool begin, uint32_t tag);
struct ProfileScope {   // records an event pair around the launches made during its lifetime
  cudaStream_t stream;
  uint32_t tag;
  ProfileScope(cudaStream_t s, uint32_t t) : stream(s), tag(t) { profile_mark(stream, true, tag); }
  ~ProfileScope() { profile_mark(stream, false, tag); }
};

}  // namespace gd
