// Everything gd_compress does after the fused full pass, in ONE cooperative launch: the exact threshold
// selection among the candidates the pass emitted (Algorithm 1, the threshold-selection step) and the
// survivor compaction (Algorithm 1, steps 3-5), followed by the end of the call (thresholds, shard
// offsets of Section 3, the means of Section 5.4).
//
// The candidate lists of all scopes, laid end to end, are cut into one contiguous share per CTA (in
// units of kSub entries).  A CTA reads its share once, keeps the values in shared memory, and then
//   coarse   histograms its entries' keys in a window of 2046 bins of 2^11 keys around the sample's
//            estimate of the threshold (one bin for everything below the window, one for everything
//            above), adds its bins to the scope's global histogram, meets the grid at a barrier and
//            walks the finished histogram itself: the bin that holds the k-th largest key, the keys
//            above it;
//   refine   the same for the low 11 bits among the entries of that bin: after the second barrier
//            the walk gives the threshold key, the number of keys above it, the tie quota;
//   count    counts, in its share, the keys above and equal to the threshold and publishes the totals
//            of its last scope; a third barrier;
//   place    adds up the totals of the CTAs before it that end in the scope its share begins in
//            (shares are contiguous, so these are exactly the CTAs holding the scope's earlier
//            entries) and writes its survivors to their final, index-ordered slots.
// If some scope's bin is the first or the last one (its threshold lies outside the window: the
// estimate was far off, rare), the grid learns of it at the second barrier and selects with three
// plain radix passes (11 + 10 + 10 bits of the key) instead; GD_FLAG_PLAIN_RADIX forces that path.
// The loops over entries are kept rolled: every CTA runs each of them once or twice, so unrolled code
// would be paid for in instruction fetches, not saved in issue slots.  Used when the call has at most kSmemScopes
// scopes; models with more tensors than that run the two separate kernels.
#include <atomic>
#include <cstring>
#include <mutex>

#include "gd_compact_body.cuh"
#include <cooperative_groups.h>

#include "gd_select_body.cuh"

namespace gd {

namespace {

constexpr uint32_t kSub = 1024;     // entries per unit of the partition of the lists over the CTAs
#ifndef GD_K2_STAGE
#define GD_K2_STAGE 8192
#endif
#ifndef GD_K2_CTAS
#define GD_K2_CTAS 2
#endif
constexpr uint32_t kStage = GD_K2_STAGE;   // entries of a share kept in shared memory; the rest is read again from L2
constexpr int kCtasPerSm = GD_K2_CTAS;     // co-resident CTAs per SM the kernel is built for
constexpr int kRounds = kTile / kThreads;   // 16 entries per thread and block of kTile entries
constexpr uint32_t kWinBins = kRadixBins0 - 2u;   // fine bins of the window; bin 0: below it, bin 2047: above it

// Debug builds (-DGD_PHASE_STAMPS) leave, in the unused tail of the control block, the time at which the last CTA
// passed each phase boundary.
#ifdef GD_PHASE_STAMPS
#define GD_STAMP(i)                                                                                                      \
  do {                                                                                                                   \
    if (threadIdx.x == 0) atomicMax(reinterpret_cast<unsigned long long*>(T.ctl) + 12 + (i), global_timer_ns());         \
  } while (0)
#else
#define GD_STAMP(i) do { } while (0)
#endif

struct Shared {
  uint32_t stage[kStage];        // value bits of the share's first kStage entries
  uint32_t idx[kStage];          // their positions in the gradient
  uint32_t hist[kRadixBins0];    // digit histogram of the scope being counted
};

__device__ __forceinline__ uint64_t min64(uint64_t a, uint64_t b) { return a < b ? a : b; }

// One contiguous piece of one scope's list inside a CTA's share.
struct Segment {
  uint32_t s;          // scope
  uint64_t beg, end;   // entries [beg, end) of the scope's list
  uint32_t sp0;        // position of entry `beg` inside the share (a multiple of kSub)
  bool first, last;    // first / last segment of the share
};

// The dense work of the scopes whose prediction failed (rare), taken over by this launch: selection over
// their dense range, a grid barrier, then their compaction.
__device__ __noinline__ bool dense_takeover(const DevTables& T, uint32_t dense_sel_tiles, uint32_t dense_chunks,
                                            unsigned char* smem) {
  select_dense_outlined<false>(T, dense_sel_tiles, *reinterpret_cast<SelectSmem<V_DENSE, false>*>(smem));
  uint32_t phase = 0;
  if (!grid_barrier(&T.ctl->barrier_mid, phase, T.ctl)) return false;
  if (__ldcg(&T.ctl->status) != GD_OK) return false;
  compact_dense_outlined(T, dense_chunks, *reinterpret_cast<CompactDenseSmem*>(smem));
  __syncthreads();                                           // the memory goes back to its usual use
  return true;
}

// (the dense work borrows the kernel's dynamic shared memory)
static_assert(sizeof(SelectSmem<V_DENSE, false>) <= sizeof(Shared) && sizeof(CompactDenseSmem) <= sizeof(Shared),
              "the dense selection and compaction borrow this kernel's shared memory");

// DENSE_IN = false: the entries are the candidate lists the fused pass left.  DENSE_IN = true (short vectors, which
// need no prediction): the "list" of a scope is its dense range itself - the kernel forms v = grad + residual as it
// loads its share, selects with the three plain radix passes, and writes the whole new residual (v where dropped,
// +0 where kept) as it places the survivors: add, select and compact of Algorithm 1 in one launch.
// What the kernel needs when it is also the start of the call (short vectors: no launch before it has cleared the
// control region or written the tables): the host-built tables, as a kernel argument, and the two regions.
struct CallStart {
  SetupBlob blob;
  uint4* tables_dst;
  uint4* zero_dst;
  uint64_t zero_vec;       // 16-byte words to clear (0: an earlier launch has started the call)
  uint32_t tables_vec;     // 16-byte words of tables
};
struct NoCallStart {};
template <bool DENSE_IN> struct StartOf { using type = NoCallStart; };
template <> struct StartOf<true> { using type = CallStart; };

template <bool DENSE_IN>
__global__ void __launch_bounds__(kThreads, kCtasPerSm) select_compact_kernel(const __grid_constant__ DevTables T,
                                                                      uint32_t dense_sel_tiles, uint32_t dense_chunks,
                                                                      const __grid_constant__ typename StartOf<DENSE_IN>::type start) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Shared& sm = *reinterpret_cast<Shared*>(smem_raw);
  __shared__ ScopeDesc s_scope[kSmemScopes];
  __shared__ uint64_t s_len[kSmemScopes];          // candidates of each scope that this launch handles (0: not its scope)
  __shared__ uint32_t s_wlo[kSmemScopes];          // lower edge of the scope's window of fine bins
  __shared__ uint32_t s_vt0[kSmemScopes + 1];      // units before each scope
  __shared__ SelRun s_run[kSmemScopes];            // where the walk down each scope's histograms stands ...
  __shared__ int s_level[kSmemScopes];             // ... and after how many of them
  __shared__ uint32_t s_cnt[kRounds * kWarps], s_tot;    // placement: keys above | equal << 16 per (round, warp)
  __shared__ unsigned long long s_pre[2];
  __shared__ uint32_t s_layer;
  __shared__ int s_single, s_last;
  __shared__ double s_red[kWarps][2];
  __shared__ uint32_t s_redc[kWarps][2];
  __shared__ alignas(8) uint64_t s_stage_bar;      // completion of the bulk copies that bring the share into shared memory
  __shared__ int s_no_abort;
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const uint32_t ltm = lanemask_lt();

  GD_STAMP(0);
  pdl_trigger();   // (the apply of the push, enqueued behind this kernel, may be brought onto the GPU from now on)
  if constexpr (DENSE_IN) {
    if (start.zero_vec != 0u) {
      // the start of the call, by the whole grid: clear the control region, write the tables, and meet (the runtime's
      // own grid barrier: the one in the control region is among the words being cleared)
      const uint64_t stride = (uint64_t)gridDim.x * kThreads, g0 = (uint64_t)blockIdx.x * kThreads + tid;
      for (uint64_t i = g0; i < start.zero_vec; i += stride) start.zero_dst[i] = make_uint4(0u, 0u, 0u, 0u);
      const uint4* src = reinterpret_cast<const uint4*>(start.blob.bytes);
      for (uint64_t i = g0; i < start.tables_vec; i += stride) start.tables_dst[i] = src[i];
      __threadfence();
      cooperative_groups::this_grid().sync();
    }
  }
  // ---- tables, lengths, partition.  Everything the start reads - the call's status, the scope descriptors, what the
  // earlier kernels left in the scopes' states - is asked for at once: one round trip to L2 instead of three.
  static_assert(kSmemScopes * (sizeof(ScopeDesc) / 8) <= 2 * kThreads, "two descriptor words per thread");
  const uint32_t words = T.n_scopes * (uint32_t)(sizeof(ScopeDesc) / 8);
  const uint64_t* src = reinterpret_cast<const uint64_t*>(T.scopes);
  const int call_status = T.ctl->status;             // set only by an earlier kernel of this call: uniform over the grid
  const uint32_t dense_needed = (!DENSE_IN && dense_sel_tiles != 0u) ? T.ctl->dense_needed : 0u;
  const uint64_t w0 = tid < words ? src[tid] : 0ull, w1 = tid + kThreads < words ? src[tid + kThreads] : 0ull;
  uint64_t x_count = 0;
  uint32_t x_tau_lo = 0, x_tau_hi = 0;
  if (tid < T.n_scopes) {
    const ScopeState* sx = T.state + tid;
    x_count = sx->cand_count; x_tau_lo = sx->tau_lo; x_tau_hi = sx->tau_hi;
  }
  if (call_status != GD_OK) return;
  if (dense_needed != 0u) {
    if (!dense_takeover(T, dense_sel_tiles, dense_chunks, smem_raw)) return;
    if (tid < T.n_scopes) {                          // (the takeover has rewritten the states of the scopes it took)
      const ScopeState* sx = T.state + tid;
      x_count = __ldcg(reinterpret_cast<const unsigned long long*>(&sx->cand_count));
      x_tau_lo = __ldcg(&sx->tau_lo); x_tau_hi = __ldcg(&sx->tau_hi);
    }
  }
  {
    uint64_t* dst = reinterpret_cast<uint64_t*>(s_scope);
    if (tid < words) dst[tid] = w0;
    if (tid + kThreads < words) dst[tid + kThreads] = w1;
    for (uint32_t i = tid; i < kSmemScopes; i += kThreads) s_level[i] = 0;
    if (tid == 0) {
      mbar_init(&s_stage_bar, 1u);
      s_no_abort = 0;
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    if (tid < T.n_scopes) {
      const uint32_t x = tid;
      const bool ok = !(T.flags & GD_FLAG_NO_PREDICTION) && x_count >= s_scope[x].k && x_count <= s_scope[x].cand_cap;   // predicted_ok()
      const uint64_t m = DENSE_IN ? s_scope[x].hi - s_scope[x].lo : (ok ? x_count : 0ull);
      s_len[x] = m;
      // the window of fine bins is centred on the sample's estimate of the threshold, but starts no lower than
      // the smallest key a candidate can have
      const uint32_t base = candidate_base_key(x_tau_lo), half = (kWinBins / 2u) << kFineShift;
      const uint32_t est = x_tau_hi;
      s_wlo[x] = (est > half && est - half > base) ? est - half : base;
      s_vt0[x + 1] = (uint32_t)((m + kSub - 1) / kSub);
    }
    if (tid == 0) s_vt0[0] = 0;
    __syncthreads();
    block_inclusive_scan(s_vt0 + 1, T.n_scopes);
  }
  const uint32_t total_units = s_vt0[T.n_scopes];
  const uint32_t per = (total_units + gridDim.x - 1) / gridDim.x;
  const uint32_t t_beg = min(blockIdx.x * per, total_units);
  const uint32_t t_end = min(t_beg + per, total_units);
  const uint32_t s_first = t_beg < t_end ? scope_of_tile(s_vt0, T.n_scopes, t_beg) : 0u;
  // The plain radix passes, should they be needed, use the scopes' sample histograms (the sample selection is
  // long finished): cleared here by the whole grid, used only after the second barrier.
  // (With dense input the plain passes start at once, in the histograms the start of the call has cleared.)
  constexpr int kPlainView = DENSE_IN ? V_CAND : V_SAMPLE;
  if (!DENSE_IN) {
    const uint64_t per_scope = 2048 + 1024 + 1024;
    const uint64_t total = (uint64_t)T.n_scopes * per_scope;
    for (uint64_t i = (uint64_t)blockIdx.x * kThreads + tid; i < total; i += (uint64_t)gridDim.x * kThreads)
      T.hist[(i / per_scope) * kHistBinsPerScope + (i % per_scope)] = 0ull;
  }

  const bool two_means = T.value_mode == GD_VALUES_TWO_MEANS || T.value_mode == GD_VALUES_COLUMN_MEANS;
  const bool packed = T.value_mode != GD_VALUES_FP32;
  const bool feedback = (T.flags & GD_FLAG_QUANT_ERROR_FEEDBACK) != 0;   // kept slots keep v for feedback_kernel
  const bool early = !DENSE_IN && early_zero_enabled(T);
  const bool plain = DENSE_IN || (T.flags & GD_FLAG_PLAIN_RADIX) != 0;
  uint4* agg = reinterpret_cast<uint4*>(T.cta_agg);   // two uint4 per CTA: {last scope, -, gt lo, gt hi}, {eq lo, eq hi, -, -}
  uint32_t phase = 0;
  GD_STAMP(1);

  // Calls f(segment) for every segment of this CTA's share, in list order (uniform over the CTA).
  auto for_segments = [&](auto&& f) {
    uint32_t s = s_first;
    for (uint32_t t = t_beg; t < t_end;) {
      while (t >= s_vt0[s + 1]) ++s;
      const uint32_t seg_t_end = min(t_end, s_vt0[s + 1]);
      Segment g;
      g.s = s;
      g.beg = (uint64_t)(t - s_vt0[s]) * kSub;
      g.end = min64((uint64_t)(seg_t_end - s_vt0[s]) * kSub, s_len[s]);
      g.sp0 = (t - t_beg) * kSub;
      g.first = t == t_beg;
      g.last = seg_t_end == t_end;
      f(g);
      t = seg_t_end;
    }
  };
  // Where the value bits of the block that starts at entry b0 of a scope's list (position sp inside the share) are
  // read from: shared memory if the block was staged, else the list itself.
  auto block_values = [&](const float* vals, uint64_t b0, uint32_t sp, uint32_t valid) -> const uint32_t* {
    return sp + valid <= kStage ? sm.stage + sp : reinterpret_cast<const uint32_t*>(vals + b0);
  };
  // Flushes the CTA's digit histogram into a scope's global one and clears it.
  auto flush_hist = [&](unsigned long long* gh, uint32_t nbins) {
    __syncthreads();
    for (uint32_t b = tid; b < nbins; b += kThreads) {
      const uint32_t c = sm.hist[b];
      if (c) { atomicAdd(gh + b, (unsigned long long)c); sm.hist[b] = 0; }
    }
    __syncthreads();
  };
  // Brings scope s's walk down the three plain radix histograms (kept in its sample slots) to `level` digits.
  auto plain_walk = [&](uint32_t s, int level) {
    SelRun run;
    int have = s_level[s];
    if (have > 0) run = s_run[s];
    else { run.prefix = 0; run.rank = s_scope[s].k; run.gt = 0; }
    __syncthreads();
    for (; have < level; ++have)
      run = next_digit(hist_of(T, s, kPlainView, have), have == 0 ? kRadixBits0 : 10, run, T.ctl);
    if (tid == 0) { s_run[s] = run; s_level[s] = level; }
    __syncthreads();
    return run;
  };

  // ---- the share into shared memory (values and positions); coarse histogram around the estimate
  for (uint32_t b = tid; b < kRadixBins0; b += kThreads) sm.hist[b] = 0;
  if (DENSE_IN) {
    // v = grad + residual (or grad - base for a pull) of the share, formed on the way into shared memory: batches of
    // 16 elements per thread, all loads of a batch in flight before the first add.  (The host gives this kernel only
    // vectors whose shares fit the stage.)
    const bool delta = T.delta_base != nullptr;
    const float* second = delta ? T.delta_base : T.residual;
    for_segments([&](const Segment& g) {
      const uint64_t lo = s_scope[g.s].lo;
      for (uint64_t b0 = g.beg; b0 < g.end; b0 += kTile) {
        const uint32_t valid = (uint32_t)min64(kTile, g.end - b0);
        const uint32_t sp = g.sp0 + (uint32_t)(b0 - g.beg);
        if (sp + valid > kStage) break;
        float gv[kRounds], rv[kRounds];
#pragma unroll
        for (int j = 0; j < kRounds; ++j) {
          const uint32_t o = (uint32_t)j * kThreads + tid;
          gv[j] = o < valid ? __ldcs(T.grad + lo + b0 + o) : 0.0f;
          rv[j] = o < valid ? second[lo + b0 + o] : 0.0f;
        }
#pragma unroll
        for (int j = 0; j < kRounds; ++j) {
          const uint32_t o = (uint32_t)j * kThreads + tid;
          if (o < valid) sm.stage[sp + o] = __float_as_uint(delta ? __fsub_rn(gv[j], rv[j]) : __fadd_rn(gv[j], rv[j]));
        }
      }
    });
  } else {
  // Bulk asynchronous copies from the lists straight into shared memory: one thread asks for every block of the
  // share - values and positions, up to 16 KB per request - and all of it is in flight at once, counted on one
  // mbarrier (as fast as copies of 16 bytes per thread, cp.async, in far fewer instructions: 4 us for a share of
  // 61 KB either way).  A bulk copy moves multiples of 16 bytes: the last entries of a block whose length is
  // no multiple of 4 are fetched with plain loads.  Nothing is written past a block's end: that part of the stage
  // belongs to the share's next segment.
  if (tid == 0) {
    uint32_t bytes = 0;
    for_segments([&](const Segment& g) {
      for (uint64_t b0 = g.beg; b0 < g.end; b0 += kTile) {
        const uint32_t valid = (uint32_t)min64(kTile, g.end - b0);
        if (g.sp0 + (uint32_t)(b0 - g.beg) + valid > kStage) break;
        bytes += 2u * 4u * (valid & ~3u);
      }
    });
    mbar_arrive_expect_tx(&s_stage_bar, bytes);
    for_segments([&](const Segment& g) {
      const uint32_t* vals = reinterpret_cast<const uint32_t*>(T.cand_val + s_scope[g.s].cand_base);
      const uint32_t* idxs = T.cand_idx + s_scope[g.s].cand_base;
      for (uint64_t b0 = g.beg; b0 < g.end; b0 += kTile) {
        const uint32_t valid = (uint32_t)min64(kTile, g.end - b0);
        const uint32_t sp = g.sp0 + (uint32_t)(b0 - g.beg);
        if (sp + valid > kStage) break;                      // the rest of the share is read from the lists every time
        const uint32_t whole = valid & ~3u;
        if (whole) {
          bulk_load(sm.stage + sp, vals + b0, 4u * whole, &s_stage_bar);
          bulk_load(sm.idx + sp, idxs + b0, 4u * whole, &s_stage_bar);
        }
      }
    });
  }
  for_segments([&](const Segment& g) {
    const uint32_t* vals = reinterpret_cast<const uint32_t*>(T.cand_val + s_scope[g.s].cand_base);
    const uint32_t* idxs = T.cand_idx + s_scope[g.s].cand_base;
    for (uint64_t b0 = g.beg; b0 < g.end; b0 += kTile) {
      const uint32_t valid = (uint32_t)min64(kTile, g.end - b0);
      const uint32_t sp = g.sp0 + (uint32_t)(b0 - g.beg);
      if (sp + valid > kStage) break;
      const uint32_t e = (valid & ~3u) + tid;
      if (e < valid) {
        sm.stage[sp + e] = __ldcg(vals + b0 + e);
        sm.idx[sp + e] = __ldcg(idxs + b0 + e);
      }
    }
  });
  if (!mbar_wait(&s_stage_bar, 0u, &s_no_abort)) {
    if (tid == 0) atomicCAS(&T.ctl->status, (int)GD_OK, (int)GD_ERR_DEVICE_TIMEOUT);
    return;
  }
  }
  __syncthreads();
  if (!plain) {
    for_segments([&](const Segment& g) {
      const float* vals = T.cand_val + s_scope[g.s].cand_base;
      const uint32_t wlo = s_wlo[g.s];
      uint32_t below = 0, above = 0;                         // this thread's entries outside the window
      for (uint64_t b0 = g.beg; b0 < g.end; b0 += kTile) {
        const uint32_t valid = (uint32_t)min64(kTile, g.end - b0);
        const uint32_t* src = block_values(vals, b0, g.sp0 + (uint32_t)(b0 - g.beg), valid);
#pragma unroll 4
        for (uint32_t o = tid; o < valid; o += kThreads) {
          const uint32_t key = src[o] & kAbsMask;
          if (key < wlo) ++below;
          else {
            const uint32_t bin = (key - wlo) >> kFineShift;
            if (bin < kWinBins) atomicAdd(&sm.hist[1u + bin], 1u); else ++above;
          }
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        below += __shfl_xor_sync(0xFFFFFFFFu, below, o);
        above += __shfl_xor_sync(0xFFFFFFFFu, above, o);
      }
      if (lane == 0 && below) atomicAdd(&sm.hist[0], below);
      if (lane == 0 && above) atomicAdd(&sm.hist[kRadixBins0 - 1u], above);
      flush_hist(hist_of(T, g.s, V_CAND, 0), kRadixBins0);
    });
  }
  GD_STAMP(2);
  if (!DENSE_IN && !grid_barrier(&T.ctl->barrier[V_CAND], phase, T.ctl)) return;   // (dense input: nothing to wait for yet)
  GD_STAMP(3);

  // ---- the bin that holds each scope's threshold; refine: the low 11 bits among the entries of that bin
  bool outside = plain;                                      // some scope needs the plain radix passes
  if (!plain) {
    for_segments([&](const Segment& g) {
      SelRun run;
      run.prefix = 0; run.rank = s_scope[g.s].k; run.gt = 0;
      __syncthreads();
      run = next_digit(hist_of(T, g.s, V_CAND, 0), kRadixBits0, run, T.ctl);
      if (tid == 0) { s_run[g.s] = run; s_level[g.s] = 1; }
      __syncthreads();
      const uint32_t bin = run.prefix;
      if (bin == 0u || bin == kRadixBins0 - 1u) { outside = true; return; }   // (uniform: a property of the scope)
      const float* vals = T.cand_val + s_scope[g.s].cand_base;
      const uint32_t lo = s_wlo[g.s] + ((bin - 1u) << kFineShift);            // keys [lo, lo + 2^11) are the bin
      for (uint64_t b0 = g.beg; b0 < g.end; b0 += kTile) {
        const uint32_t valid = (uint32_t)min64(kTile, g.end - b0);
        const uint32_t* src = block_values(vals, b0, g.sp0 + (uint32_t)(b0 - g.beg), valid);
#pragma unroll 4
        for (uint32_t o = tid; o < valid; o += kThreads) {
          const uint32_t dd = (src[o] & kAbsMask) - lo;                       // (wraps for keys below the bin)
          if (dd < (1u << kFineShift)) atomicAdd(&sm.hist[dd], 1u);
        }
      }
      flush_hist(hist_of(T, g.s, V_CAND, 1), 1u << kFineShift);   // (the second and third slots together: 2048 bins)
    });
  }
  if (outside && tid == 0) atomicOr(&T.ctl->generic_needed, 1u);
  GD_STAMP(4);
  if (!DENSE_IN && !grid_barrier(&T.ctl->barrier[V_CAND], phase, T.ctl)) return;
  GD_STAMP(5);

  if (!DENSE_IN && __ldcg(&T.ctl->generic_needed) == 0u) {
    // the threshold key = lower edge of the bin + the digit found in the refined histogram
    for_segments([&](const Segment& g) {
      if (s_level[g.s] != 1) return;
      SelRun run = s_run[g.s];
      const uint32_t bin = run.prefix;
      run.prefix = 0;
      __syncthreads();
      run = next_digit(hist_of(T, g.s, V_CAND, 1), kFineShift, run, T.ctl);
      run.prefix = s_wlo[g.s] + ((bin - 1u) << kFineShift) + run.prefix;
      if (tid == 0) { s_run[g.s] = run; s_level[g.s] = 3; }
      __syncthreads();
    });
  } else {
    // ---- three plain radix passes over the keys (11 + 10 + 10 bits), in the scopes' cleared sample histograms
    __syncthreads();
    for (uint32_t i = tid; i < kSmemScopes; i += kThreads) s_level[i] = 0;
    __syncthreads();
    for (int pass = 0; pass < 3; ++pass) {
      const int shift = pass == 0 ? kShift0 : (pass == 1 ? kShift1 : kShift2);
      const uint32_t dmask = (1u << (pass == 0 ? kRadixBits0 : 10)) - 1u;
      const int pshift = pass == 1 ? kShift0 : kShift1;     // shift that exposes the digits fixed so far
      for_segments([&](const Segment& g) {
        const float* vals = T.cand_val + s_scope[g.s].cand_base;
        const uint32_t prefix = plain_walk(g.s, pass).prefix;
        for (uint64_t b0 = g.beg; b0 < g.end; b0 += kTile) {
          const uint32_t valid = (uint32_t)min64(kTile, g.end - b0);
          const uint32_t* src = block_values(vals, b0, g.sp0 + (uint32_t)(b0 - g.beg), valid);
#pragma unroll 4
          for (uint32_t o = tid; o < valid; o += kThreads) {
            const uint32_t key = src[o] & kAbsMask;
            if (pass == 0 || (key >> pshift) == prefix) atomicAdd(&sm.hist[(key >> shift) & dmask], 1u);
          }
        }
        flush_hist(hist_of(T, g.s, kPlainView, pass), dmask + 1u);
      });
      if (!grid_barrier(&T.ctl->barrier[V_CAND], phase, T.ctl)) return;
    }
    for_segments([&](const Segment& g) { plain_walk(g.s, 3); });
  }
  GD_STAMP(6);

  // ---- thresholds of the scopes of this share go on record; counts of its last scope for the CTAs after it
  {
    uint32_t my_scope = 0xFFFFFFFFu;
    unsigned long long my_g = 0, my_e = 0;                   // (per thread; added up below)
    for_segments([&](const Segment& g) {
      const SelRun run = s_run[g.s];
      if (g.beg == 0 && tid == 0) {                          // the CTA that holds the scope's first entries
        ScopeState* st = T.state + g.s;
        st->tau = run.prefix; st->q = run.rank; st->gt = run.gt;
        if (DENSE_IN) st->used_dense = 1u;                   // (statistics: selected over the dense range)
      }
      if (!g.last) return;
      const float* vals = T.cand_val + s_scope[g.s].cand_base;
      const uint32_t tau = run.prefix;
      uint32_t cg = 0, ce = 0;
      for (uint64_t b0 = g.beg; b0 < g.end; b0 += kTile) {
        const uint32_t valid = (uint32_t)min64(kTile, g.end - b0);
        const uint32_t* src = block_values(vals, b0, g.sp0 + (uint32_t)(b0 - g.beg), valid);
#pragma unroll 4
        for (uint32_t o = tid; o < valid; o += kThreads) {
          const uint32_t key = src[o] & kAbsMask;
          cg += key > tau ? 1u : 0u;
          ce += key == tau ? 1u : 0u;
        }
      }
      my_g = cg; my_e = ce; my_scope = g.s;
    });
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      my_g += __shfl_xor_sync(0xFFFFFFFFu, my_g, o);
      my_e += __shfl_xor_sync(0xFFFFFFFFu, my_e, o);
    }
    __syncthreads();
    if (tid == 0) { s_pre[0] = 0; s_pre[1] = 0; }
    __syncthreads();
    if (lane == 0 && (my_g | my_e)) { atomicAdd(&s_pre[0], my_g); atomicAdd(&s_pre[1], my_e); }
    __syncthreads();
    if (tid == 0) {
      const unsigned long long tg = s_pre[0], te = s_pre[1];
      __stcg(agg + 2 * blockIdx.x, make_uint4(my_scope, 0u, (uint32_t)tg, (uint32_t)(tg >> 32)));
      __stcg(agg + 2 * blockIdx.x + 1, make_uint4((uint32_t)te, (uint32_t)(te >> 32), 0u, 0u));
    }
  }
  GD_STAMP(7);
  if (!grid_barrier(&T.ctl->barrier[V_CAND], phase, T.ctl)) return;
  GD_STAMP(8);

  // ---- placement
  for_segments([&](const Segment& g) {
    const uint32_t s = g.s;
    const ScopeDesc& d = s_scope[s];
    const SelRun run = s_run[s];
    const uint32_t tau = run.prefix;
    const uint64_t q = run.rank;
    // keys above / equal to tau among the scope's entries before this segment: the CTAs before this one whose
    // share ends in the same scope hold exactly those entries (only the first segment of a share can have any)
    uint64_t seg_g = 0, seg_e = 0;
    if (g.first && g.beg != 0) {
      unsigned long long pg = 0, pe = 0;
      for (uint32_t b = tid; b < blockIdx.x; b += kThreads) {
        const uint4 a0 = __ldcg(agg + 2 * b), a1 = __ldcg(agg + 2 * b + 1);
        if (a0.x == s) {
          pg += ((unsigned long long)a0.w << 32) | a0.z;
          pe += ((unsigned long long)a1.y << 32) | a1.x;
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        pg += __shfl_xor_sync(0xFFFFFFFFu, pg, o);
        pe += __shfl_xor_sync(0xFFFFFFFFu, pe, o);
      }
      __syncthreads();
      if (tid == 0) { s_pre[0] = 0; s_pre[1] = 0; }
      __syncthreads();
      if (lane == 0 && (pg | pe)) { atomicAdd(&s_pre[0], pg); atomicAdd(&s_pre[1], pe); }
      __syncthreads();
      seg_g = s_pre[0];
      seg_e = s_pre[1];
    }
    const ScopeState* st = T.state + s;
    // Entries with key > zthr had +0 written over their residual slot by the fused pass.  Kept ones need no
    // store then (unless some entry of the scope could not be treated so: early_bad); the few that are not
    // kept after all get v back.
    const uint32_t zthr = early ? st->tau_hi : 0xFFFFFFFFu;
    const bool skip_cleared = early && st->early_bad == 0u;
    const float* vals = T.cand_val + d.cand_base;

    for (uint64_t b0 = g.beg; b0 < g.end; b0 += kTile) {
      const uint32_t valid = (uint32_t)min64(kTile, g.end - b0);
      const uint32_t* tile_idx = T.cand_idx + d.cand_base + b0;
      const uint32_t sp = g.sp0 + (uint32_t)(b0 - g.beg);
      const uint32_t* src = block_values(vals, b0, sp, valid);
      const uint32_t* isrc = sp + valid <= kStage ? sm.idx + sp : tile_idx;   // the block's positions (lists)
      const uint64_t pos0 = d.lo + b0;                        // position of the block's first entry (dense input)
      __syncthreads();                                       // the previous block is done with the shared variables
      if (two_means && tid == 0) {
        const uint32_t l0 = range_of(T.layer_off, T.n_layers, DENSE_IN ? pos0 : (uint64_t)tile_idx[0]);
        const uint32_t l1 = range_of(T.layer_off, T.n_layers, DENSE_IN ? pos0 + valid - 1 : (uint64_t)tile_idx[valid - 1]);
        s_layer = (uint32_t)T.pair_off[l0];                  // the one pair of the block, if it has only one
        s_single = (l0 == l1 && T.layer_cols[l0] == 1u) ? 1 : 0;
      }
      // classification: round j covers entries [256 j, 256 j + 256), thread t its entry 256 j + t; only the rounds that
      // hold entries run.  Keys above / equal to tau per (round, warp), packed (a block has at most 4096 entries).
      const int rounds = (int)((valid + kThreads - 1) / kThreads);
      uint32_t gm = 0, em = 0, zm = 0;
#pragma unroll 4
      for (int j = 0; j < rounds; ++j) {
        const uint32_t o = (uint32_t)j * kThreads + tid;
        const bool in = o < valid;
        const uint32_t key = in ? (src[o] & kAbsMask) : 0u;
        const bool isgt = in && key > tau, iseq = in && key == tau;
        gm |= (isgt ? 1u : 0u) << j;
        em |= (iseq ? 1u : 0u) << j;
        zm |= (in && key > zthr ? 1u : 0u) << j;
        const uint32_t cg = __popc(__ballot_sync(0xFFFFFFFFu, isgt)), ce = __popc(__ballot_sync(0xFFFFFFFFu, iseq));
        if (lane == 0) s_cnt[j * kWarps + (int)warp] = cg | (ce << 16);
      }
      __syncthreads();
      if (warp == 0) {                                        // exclusive prefix over the (round, warp) counts, in that order
        constexpr int kPerLane = kRounds * kWarps / 32;       // 4
        uint32_t c[kPerLane], sum = 0;
#pragma unroll
        for (int u = 0; u < kPerLane; ++u) {
          const int e = (int)lane * kPerLane + u;
          c[u] = e < rounds * kWarps ? s_cnt[e] : 0u;
          sum += c[u];
        }
        uint32_t inc = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
          if ((int)lane >= o) inc += y;
        }
        uint32_t run = inc - sum;
#pragma unroll
        for (int u = 0; u < kPerLane; ++u) {
          s_cnt[(int)lane * kPerLane + u] = run;
          run += c[u];
        }
        if (lane == 31) s_tot = inc;
      }
      __syncthreads();
      const uint32_t tot_g = s_tot & 0xFFFFu, tot_e = s_tot >> 16;
      // Slot of an entry = (#above before it) + min(#ties before it, q); with seg_g / seg_e the counts before this
      // block that is  out_base + seg_g + min(seg_e, q) + (above before it in the block) + min(ties before it in
      // the block, q - min(seg_e, q)): one 64-bit base per block and 32-bit arithmetic per entry.
      const uint64_t tie_base = seg_e < q ? seg_e : q;
      const uint64_t q_left64 = q - tie_base;
      const uint32_t q_left = q_left64 < 0xFFFFu ? (uint32_t)q_left64 : 0xFFFFu;   // a block has at most 4096 entries
      const uint64_t slot0 = seg_g + tie_base;
      const uint64_t room64 = d.k > slot0 ? d.k - slot0 : 0;
      const uint32_t room = room64 < kTile ? (uint32_t)room64 : kTile;
      uint32_t* const oi = T.out_idx + d.out_base + slot0;
      float* const ov = T.out_val ? T.out_val + d.out_base + slot0 : nullptr;
      const bool single = two_means && s_single;
      const uint32_t tile_layer = two_means ? s_layer : 0u;
      double sum_p = 0.0, sum_n = 0.0;
      uint32_t cnt_p = 0, cnt_n = 0;
      bool bad = false;
#pragma unroll 1
      for (int j = 0; j < rounds; ++j) {
        const bool isgt = (gm >> j) & 1u, iseq = (em >> j) & 1u, cleared = (zm >> j) & 1u;
        const uint32_t mg = __ballot_sync(0xFFFFFFFFu, isgt), me = __ballot_sync(0xFFFFFFFFu, iseq);
        const uint32_t o = (uint32_t)j * kThreads + tid;
        if (DENSE_IN ? o < valid : (isgt || iseq || cleared)) {
          const uint32_t before = s_cnt[j * kWarps + (int)warp];          // in the block, before this warp's round
          const uint32_t rg = before & 0xFFFFu, re = before >> 16;
          const uint32_t eb = re + __popc(me & ltm);
          const uint64_t idx = DENSE_IN ? pos0 + o : (uint64_t)isrc[o];
          const uint32_t b = src[o];
          const bool keep = isgt || (iseq && eb < q_left);
          // dense input: this is where the new residual is written, every element of it (v where dropped, +0 where
          // kept, v for kept entries whose quantisation error is fed back later)
          if (DENSE_IN && idx < T.n) T.residual[idx] = (keep && !feedback) ? 0.0f : __uint_as_float(b);
          if (keep) {
            const uint32_t pos = rg + __popc(mg & ltm) + (eb < q_left ? eb : q_left);
            if (pos < room && idx < T.n) {
              if (!DENSE_IN && !feedback && !(skip_cleared && cleared)) T.residual[idx] = 0.0f;
              if (packed) {
                const uint32_t sgn = b >> 31;
                oi[pos] = (uint32_t)idx | (sgn << 31);
                const double xv = (double)__uint_as_float(b);
                if (!two_means) {
                  // threshold mode: the value is implied by the scope's tau
                } else if (single) {
                  if (sgn) { sum_n += xv; ++cnt_n; } else { sum_p += xv; ++cnt_p; }
                } else {
                  const uint64_t pr = pair_of(T.layer_off, T.pair_off, T.layer_cols, T.n_layers, idx);
                  atomicAdd(T.sums + 2 * pr + sgn, xv);
                  atomicAdd(T.cnts + 2 * pr + sgn, 1ull);
                }
              } else {
                oi[pos] = (uint32_t)idx;
                ov[pos] = __uint_as_float(b);
                if (T.delta_base) T.delta_base[idx] = __fadd_rn(T.delta_base[idx], __uint_as_float(b));
              }
            } else {
              bad = true;
            }
          } else if (cleared && idx < T.n) {
            // cleared early but not kept after all (the estimate was below tau, or a tie beyond the quota)
            T.residual[idx] = __uint_as_float(b);
          }
        }
      }
      if (bad) atomicCAS(&T.ctl->status, (int)GD_OK, (int)GD_ERR_INTERNAL);
      if (single) {   // uniform over the CTA
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          sum_p += __shfl_xor_sync(0xFFFFFFFFu, sum_p, o);
          sum_n += __shfl_xor_sync(0xFFFFFFFFu, sum_n, o);
          cnt_p += __shfl_xor_sync(0xFFFFFFFFu, cnt_p, o);
          cnt_n += __shfl_xor_sync(0xFFFFFFFFu, cnt_n, o);
        }
        if (lane == 0) { s_red[warp][0] = sum_p; s_red[warp][1] = sum_n; s_redc[warp][0] = cnt_p; s_redc[warp][1] = cnt_n; }
        __syncthreads();
        if (tid < 2) {
          double sx = 0.0;
          unsigned long long cx = 0;
          for (int w = 0; w < kWarps; ++w) { sx += s_red[w][tid]; cx += s_redc[w][tid]; }
          if (cx) {
            atomicAdd(T.sums + 2 * (size_t)tile_layer + tid, sx);
            atomicAdd(T.cnts + 2 * (size_t)tile_layer + tid, cx);
          }
        }
      }
      seg_g += tot_g;
      seg_e += tot_e;
    }
  });
  GD_STAMP(9);

  // ---- the last CTA to leave finishes the call
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(&T.ctl->compact_done[0], 1u) == gridDim.x - 1u) ? 1 : 0;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  finalize_call(T, T.k_total);
}

}  // namespace


namespace {

// Co-resident CTAs of the kernel per SM on the current device, asked once per device (with the kernel's shared-memory
// attribute set on the way); *dev receives the device.
template <bool DENSE_IN>
cudaError_t resident_ctas(int* resident_out, int* dev_out) {
  static PerDeviceInt resident_of;                         // (0: not asked yet)
  int dev = -1;
  const size_t smem = sizeof(Shared);
  int resident = resident_of.get(&dev);
  if (dev < 0) return cudaErrorInvalidDevice;              // (the shared-memory attribute below is per device)
  if (resident == 0) {
    cudaError_t e = cudaFuncSetAttribute(select_compact_kernel<DENSE_IN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int r = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&r, select_compact_kernel<DENSE_IN>, kThreads, smem);
    if (e != cudaSuccess) return e;
    if (r <= 0) return cudaErrorLaunchFailure;
    resident = r;
    resident_of.set(dev, r);
  }
  *resident_out = resident;
  *dev_out = dev;
  return cudaSuccess;
}

template <bool DENSE_IN>
cudaError_t launch_impl(const DevTables& T, uint64_t units, uint32_t dsel, uint32_t dchunks, uint32_t tag, cudaStream_t stream,
                        const typename StartOf<DENSE_IN>::type& start) {
  ProfileScope prof(stream, tag);
  const size_t smem = sizeof(Shared);
  int resident = 0, dev = -1;
  cudaError_t er = resident_ctas<DENSE_IN>(&resident, &dev);
  if (er != cudaSuccess) return er;
  const uint32_t per_sm = resident < kCtasPerSm ? (uint32_t)resident : (uint32_t)kCtasPerSm;
  uint32_t grid = (uint32_t)sm_count() * per_sm;
  if (units < 1) units = 1;
  if (grid > units) grid = (uint32_t)units;                // no more CTAs than units of work
  if (grid > kSelectCompactMaxGrid) grid = kSelectCompactMaxGrid;
  if (DENSE_IN && (units + grid - 1) / grid > kStage / kSub) return cudaErrorInvalidConfiguration;   // a share must fit the stage
  DevTables Tc = T;
  void* args[] = {(void*)&Tc, (void*)&dsel, (void*)&dchunks, (void*)&start};
  cudaError_t e = cudaLaunchCooperativeKernel((const void*)select_compact_kernel<DENSE_IN>, dim3(grid), dim3(kThreads), args,
                                              smem, stream);
  if (e != cudaSuccess) return e;
  note_launches(1);
  return cudaSuccess;
}

}  // namespace

cudaError_t launch_select_compact(const DevTables& T, const uint32_t* tiles, uint64_t cand_total, cudaStream_t stream) {
  // units of work: the lists' capacity - or the dense tiles this launch may have to take over, if there are more
  uint64_t units = (cand_total + kSub - 1) / kSub;
  if (units < tiles[L_DSEL]) units = tiles[L_DSEL];
  return launch_impl<false>(T, units, tiles[L_DSEL], tiles[L_DCOMP], PT_CAND_SELECT_COMPACT, stream, NoCallStart{});
}

// Short vectors: residual add, exact selection and compaction over the dense range itself, in one launch.
// dense_units: the scopes' lengths in units of 1024 elements, summed.
// tables_src != NULL: the launch is also the start of the call - it clears zero_bytes at zero_dst and writes the
// tables_bytes (at most kSetupBlobBytes) of host-built tables to tables_dst before anything else.
cudaError_t launch_dense_fused(const DevTables& T, uint64_t dense_units, cudaStream_t stream, void* tables_dst,
                               const void* tables_src, size_t tables_bytes, void* zero_dst, size_t zero_bytes) {
  static CallStart start;                                    // (large: kept off the stack; filled under the lock below)
  static std::mutex start_mutex;
  std::lock_guard<std::mutex> lock(start_mutex);
  start.zero_vec = 0;
  start.tables_vec = 0;
  start.tables_dst = nullptr;
  start.zero_dst = nullptr;
  if (tables_src) {
    if (tables_bytes > kSetupBlobBytes) return cudaErrorInvalidValue;
    std::memcpy(start.blob.bytes, tables_src, tables_bytes);
    start.tables_dst = (uint4*)tables_dst;
    start.tables_vec = (uint32_t)(tables_bytes / 16);
    start.zero_dst = (uint4*)zero_dst;
    start.zero_vec = zero_bytes / 16;
  }
  return launch_impl<true>(T, dense_units, 0u, 0u, PT_DENSE_FUSED, stream, start);
}

// How many units launch_dense_fused can take on the current device: every CTA's share must fit its shared-memory
// stage.  0 if the kernel cannot run here.
uint64_t dense_fused_capacity() {
  int resident = 0, dev = -1;
  if (resident_ctas<true>(&resident, &dev) != cudaSuccess) { (void)cudaGetLastError(); return 0; }
  const uint64_t per_sm = resident < kCtasPerSm ? (uint64_t)resident : (uint64_t)kCtasPerSm;
  uint64_t grid = (uint64_t)sm_count() * per_sm;
  if (grid > kSelectCompactMaxGrid) grid = kSelectCompactMaxGrid;
  return grid * (kStage / kSub);
}

}  // namespace gd
