// The selection over the whole dense vector without a sample (GD_FLAG_NO_PREDICTION on long vectors):
// Algorithm 1's threshold-selection step, started from one histogram pass.
//
//   dense_hist   streams grad and residual once (8 bytes per element, nothing written), forms
//                v = grad + residual and counts the first 11 bits of |v| per scope;
//   dense_find   walks each scope's histogram: the bin that holds the k-th largest key.  Its lower edge
//                is an exact lower bound of the threshold, and the entries at or above it - at most k
//                plus one bin's worth - are exactly what the fused pass lists as candidates;
// after which the call continues like a predicted one (fused pass, selection among the candidates,
// compaction), with a bound that cannot fail.  The literal alternative - three histogram passes and a
// compaction pass over all n elements - is bound by shared-memory atomics at about 2.5 TB/s per pass.
//
// Only the upper tail matters, so the histogram pass skips what lies far below the largest key seen so
// far: a thread counts a key only if its bin is within kWindowBins of the largest bin it knows of (the
// scope's running maximum when its CTA started, raised by what the thread itself has seen).  Every
// such floor is at most the final floor, so the bins from (final maximum - kWindowBins) up are
// complete; dense_find checks that the k-th largest key lies there, and otherwise asks for the pass
// to be run once more without the window (a second launch that usually starts, looks at a flag and
// leaves).
#include <atomic>

#include "gd_select_body.cuh"

namespace gd {

namespace {

constexpr uint32_t kWindowBins = 64;   // 8 binades below the largest key (the first digit resolves an eighth of a binade)

template <bool FULL>
__global__ void __launch_bounds__(kThreads, 4) dense_hist_kernel(const __grid_constant__ DevTables T) {
  __shared__ uint32_t s_hist[kRadixBins0];
  __shared__ uint32_t s_max;
  __shared__ SmemTables s_tab;
  const uint32_t tid = threadIdx.x, lane = tid & 31u;
  if (FULL && T.ctl->hist_redo == 0u) return;
  const ScopeDesc* scopes;
  const uint32_t* tile0;
  load_tables(T, L_EMIT, &s_tab, &scopes, &tile0);
  for (uint32_t b = tid; b < kRadixBins0; b += kThreads) s_hist[b] = 0;
  if (tid == 0) s_max = 0;
  __syncthreads();
  const uint32_t t = blockIdx.x;
  const uint32_t s = T.n_scopes <= kSmemScopes ? scope_of_tile(tile0, T.n_scopes, t) : block_count_le(tile0, T.n_scopes, t) - 1u;
  const ScopeDesc& d = scopes[s];
  if (d.k == 0) return;                                   // nothing is kept: no threshold to find
  const uint64_t lo = d.lo, hi = d.hi;
  const uint64_t CH = (uint64_t)T.emit_chunk_tiles * kTile;
  const uint64_t cbase = (lo / CH + (t - tile0[s])) * CH;
  ScopeState* st = T.state + s;
  const bool delta = T.delta_base != nullptr;            // v = g - base instead of g + r
  const float* second = delta ? T.delta_base : T.residual;
  // bins below `floor` are not counted
  uint32_t top = FULL ? 0u : __ldcg(&st->top_bin_max);
  uint32_t floor_bin = top > kWindowBins ? top - kWindowBins : 0u;
  auto count = [&](float x) {
    const uint32_t bin = (__float_as_uint(x) & kAbsMask) >> kShift0;
    if (bin >= floor_bin) {
      atomicAdd(&s_hist[bin], 1u);
      if (!FULL && bin > top) { top = bin; floor_bin = top > kWindowBins ? top - kWindowBins : 0u; }
    }
  };
  const int tiles = (int)T.emit_chunk_tiles;
#pragma unroll 1
  for (int i = 0; i < tiles; ++i) {
    const uint64_t base = cbase + (uint64_t)i * kTile;
    if (base >= lo && base + kTile <= hi) {
      const uint64_t e0 = base + (uint64_t)tid * 4u;
      float4 g4[4], r4[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) g4[j] = __ldcs(reinterpret_cast<const float4*>(T.grad + e0 + j * 1024));
#pragma unroll
      for (int j = 0; j < 4; ++j) r4[j] = __ldcs(reinterpret_cast<const float4*>(second + e0 + j * 1024));
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        count(delta ? __fsub_rn(g4[j].x, r4[j].x) : __fadd_rn(g4[j].x, r4[j].x));
        count(delta ? __fsub_rn(g4[j].y, r4[j].y) : __fadd_rn(g4[j].y, r4[j].y));
        count(delta ? __fsub_rn(g4[j].z, r4[j].z) : __fadd_rn(g4[j].z, r4[j].z));
        count(delta ? __fsub_rn(g4[j].w, r4[j].w) : __fadd_rn(g4[j].w, r4[j].w));
      }
    } else if (base < hi && base + kTile > lo) {          // tile cut by the scope (or by the end of the vector)
      for (uint32_t o = tid; o < kTile; o += kThreads) {
        const uint64_t e = base + o;
        if (e >= lo && e < hi) count(delta ? __fsub_rn(__ldg(T.grad + e), second[e]) : __fadd_rn(__ldg(T.grad + e), second[e]));
      }
    }
  }
  if (!FULL) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) top = max(top, __shfl_xor_sync(0xFFFFFFFFu, top, o));
    if (lane == 0) atomicMax(&s_max, top);
  }
  __syncthreads();
  unsigned long long* gh = T.hist + (size_t)s * kHistBinsPerScope + (FULL ? 2048u : 0u);   // the scope's sample slots
  for (uint32_t b = tid; b < kRadixBins0; b += kThreads) {
    const uint32_t c = s_hist[b];
    if (c) atomicAdd(gh + b, (unsigned long long)c);
  }
  if (!FULL && tid == 0) atomicMax(&st->top_bin_max, s_max);
}

// One CTA per scope: the bin of the k-th largest key, from the histogram dense_hist left.
template <bool FULL>
__global__ void __launch_bounds__(kThreads) dense_find_kernel(const __grid_constant__ DevTables T) {
  __shared__ unsigned long long s_part[kWarps];
  __shared__ int s_valid;
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  pdl_trigger();   // (the fused pass is enqueued behind the second walk)
  if (FULL && T.ctl->hist_redo == 0u) return;
  const uint32_t s = blockIdx.x;
  const ScopeDesc& d = T.scopes[s];
  ScopeState* st = T.state + s;
  if (d.k == 0) return;
  const unsigned long long* gh = T.hist + (size_t)s * kHistBinsPerScope + (FULL ? 2048u : 0u);
  const uint32_t top = FULL ? 0u : __ldcg(&st->top_bin_max);
  const uint32_t floor_bin = top > kWindowBins ? top - kWindowBins : 0u;
  // the histogram is complete from floor_bin up: it is usable if those bins hold at least k keys
  unsigned long long part = 0;
  for (uint32_t b = floor_bin + tid; b < kRadixBins0; b += kThreads) part += __ldcg(gh + b);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, o);
  if (lane == 0) s_part[warp] = part;
  __syncthreads();
  if (tid == 0) {
    unsigned long long tot = 0;
    for (int w = 0; w < kWarps; ++w) tot += s_part[w];
    s_valid = tot >= d.k ? 1 : 0;
    if (!s_valid) {
      if (FULL) atomicCAS(&T.ctl->status, (int)GD_OK, (int)GD_ERR_INTERNAL);   // the full histogram counts every key
      else atomicOr(&T.ctl->hist_redo, 1u);
    }
  }
  __syncthreads();
  if (!s_valid) return;
  SelRun run;
  run.prefix = 0; run.rank = d.k; run.gt = 0;
  run = next_digit(gh, kRadixBits0, run, T.ctl);
  if (tid == 0) {
    st->tau_lo = run.prefix << kShift0;                    // lower edge of the bin: an exact lower bound of the threshold
    st->tau_hi = st->tau_lo;                               // (where the selection among the candidates centres its window;
                                                           // nothing is cleared early in this mode)
  }
}

}  // namespace

// Histogram pass and walk, then - enqueued always, run only if some scope's window missed - once more without
// the window.  `tiles` is indexed by Launch.
cudaError_t launch_dense_bound(const DevTables& T, const uint32_t* tiles, cudaStream_t stream) {
  if (!tiles[L_EMIT]) return cudaSuccess;
  {
    ProfileScope prof(stream, PT_DENSE_HIST);
    dense_hist_kernel<false><<<tiles[L_EMIT], kThreads, 0, stream>>>(T);
    GD_LAUNCH_CHECK();
  }
  {
    ProfileScope prof(stream, PT_DENSE_FIND);
    dense_find_kernel<false><<<T.n_scopes, kThreads, 0, stream>>>(T);
    GD_LAUNCH_CHECK();
  }
  {
    ProfileScope prof(stream, PT_DENSE_HIST);
    dense_hist_kernel<true><<<tiles[L_EMIT], kThreads, 0, stream>>>(T);
    GD_LAUNCH_CHECK();
  }
  {
    ProfileScope prof(stream, PT_DENSE_FIND);
    dense_find_kernel<true><<<T.n_scopes, kThreads, 0, stream>>>(T);
    GD_LAUNCH_CHECK();
  }
  return cudaSuccess;
}

}  // namespace gd
