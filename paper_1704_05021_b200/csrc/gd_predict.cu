// Start of a gd_compress call and the prediction of every scope's threshold, in one ordinary launch.
//
// The fused full pass needs, per scope, a lower bound tau_lo of the threshold key (entries at or above
// it become candidates) and an estimate tau_hi of the threshold itself (entries above it have their
// residual slot cleared in the stream).  Both are order statistics of a small stratified sample of
// v = grad + residual (Algorithm 1's threshold-selection step, run on a sample; the result of the call
// never depends on it).  When every scope's sample is at most kLocalSampleMax values, the sample is
// gathered in tiles of 256 to 1024 by CTAs spread over the whole GPU (one SM keeps too few scattered reads in
// flight), and the CTA that finishes a scope's gather last selects both ranks by itself, in a
// shared-memory histogram, with two radix passes over the gathered values (11 + 10 bits: the
// prediction needs 21 bits only) - no global histogram, no grid barrier.  Every CTA marks its tile with
// the call's number when it is done and then looks at the scope's other marks: whoever sees all of
// them selects (the CTA whose mark lands last always does; if two see it at once both write the same
// prediction), so nothing needs clearing and nothing waits.  The
// remaining CTAs of the same launch clear the call's control region and write the host-built tables
// behind it, which otherwise is a launch of its own.  Larger samples (one scope of hundreds of
// millions of elements) take the cooperative selection in gd_select.cu.
#include <atomic>
#include <chrono>
#include <cstring>

#include "gd_select_body.cuh"

namespace gd {

namespace {

constexpr int kPredictThreads = 1024;
constexpr int kPredictWarps = kPredictThreads / 32;
constexpr size_t kKeysBytes = sizeof(uint32_t) * kLocalSampleMax;   // dynamic shared memory: one scope's whole sample

// For each of `count` ranks (1-based, from the largest key down): the bin of hist[0 .. nbins) that holds it and
// the number of keys in the bins above that bin.  nbins is 1024 or 2048; run by the whole CTA.
__device__ void find_ranks(const uint32_t* hist, uint32_t nbins, const uint32_t* ranks, int count, uint32_t* bin_out,
                           uint32_t* above_out) {
  __shared__ uint32_t s_wsum[kPredictWarps];
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const uint32_t per = nbins / kPredictThreads;           // 1 or 2 bins per thread, from the top bin down
  const uint32_t top = nbins - 1u - tid * per;
  const uint32_t c0 = hist[top], c1 = per == 2u ? hist[top - 1u] : 0u;
  const uint32_t sum = c0 + c1;
  uint32_t inc = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
    if ((int)lane >= o) inc += y;
  }
  __syncthreads();                                        // the scratch is free again
  if (lane == 31u) s_wsum[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    uint32_t v = s_wsum[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, v, o);
      if ((int)lane >= o) v += y;
    }
    s_wsum[lane] = v;
  }
  __syncthreads();
  const uint32_t above = inc - sum + (warp ? s_wsum[warp - 1u] : 0u);
  for (int r = 0; r < count; ++r) {
    const uint32_t rank = ranks[r];
    if (above < rank && rank <= above + c0) { bin_out[r] = top; above_out[r] = above; }
    else if (per == 2u && above + c0 < rank && rank <= above + sum) { bin_out[r] = top - 1u; above_out[r] = above + c0; }
  }
  __syncthreads();
}

__global__ void __launch_bounds__(kPredictThreads, 1)
setup_predict_kernel(const __grid_constant__ DevTables T, const __grid_constant__ SetupBlob blob, uint32_t gather_ctas,
                     uint32_t gather_tile, uint32_t call, uint32_t* flags, uint4* tables_dst, uint32_t tables_vec, uint4* zero_dst, uint64_t zero_vec,
                     uint64_t state_vec_beg, uint64_t state_vec_end, uint32_t scopes_off, uint32_t tile0_off) {
  extern __shared__ __align__(16) unsigned char smem_keys[];   // the scope's sample, for the CTA that finishes the scope
  __shared__ uint32_t s_hist[kRadixBins0];
  __shared__ uint32_t s_bin[2], s_above[2], s_rank[2];
  __shared__ int s_is_last;
  const uint32_t tid = threadIdx.x, lane = tid & 31u;
  const ScopeDesc* scopes = reinterpret_cast<const ScopeDesc*>(blob.bytes + scopes_off);
  pdl_trigger();   // the fused pass, enqueued behind this kernel, may be brought onto the GPU from now on
  pdl_wait();      // (this kernel itself may have been: nothing is read or written before the stream's earlier kernels are done)

  if (blockIdx.x >= gather_ctas) {
    // ---- the start of the call: clear the control region (the scope states are cleared by the CTAs that fill them
    // in; those of scopes without a sample here), write the tables
    const uint64_t z = blockIdx.x - gather_ctas, nz = gridDim.x - gather_ctas;
    const uint64_t stride = nz * kPredictThreads;
    for (uint64_t i = z * kPredictThreads + tid; i < zero_vec; i += stride)
      if (i < state_vec_beg || i >= state_vec_end) zero_dst[i] = make_uint4(0u, 0u, 0u, 0u);
    const uint4* src = reinterpret_cast<const uint4*>(blob.bytes);
    for (uint64_t i = z * kPredictThreads + tid; i < tables_vec; i += stride) tables_dst[i] = src[i];
    // Marks for the fused pass, which may be running already (it is a programmatic dependent of this launch and, with
    // its tables in its own argument, does not wait for this grid to end): one per scope whose prediction is final -
    // here the scopes without a sample - and one per CTA that has done its part of the clearing.
    uint32_t* ready = flags + gather_ctas;
    uint32_t* cleared = ready + kSmemScopes;
    if (z == 0) {
      for (uint32_t x = tid; x < T.n_scopes; x += kPredictThreads) {
        if (scopes[x].samp_m == 0) {
          uint4* p = reinterpret_cast<uint4*>(T.state + x);
          static_assert(sizeof(ScopeState) == 48, "three 16-byte stores clear one scope state");
          p[0] = make_uint4(0u, 0u, 0u, 0u); p[1] = p[0]; p[2] = p[0];
          __threadfence();
          if (x < kSmemScopes) __stcg(ready + x, call);
        }
      }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0 && z < kStartMarks) __stcg(cleared + z, call);
    return;
  }

  // ---- one tile of one scope's sample
  const uint32_t kGather = gather_tile;                    // samples per tile (256, 512 or 1024): one per thread
  const uint32_t* tile0 = reinterpret_cast<const uint32_t*>(blob.bytes + tile0_off);
  const uint32_t s = scope_of_tile(tile0, T.n_scopes, blockIdx.x);
  const uint32_t first = tile0[s], lt = blockIdx.x - first, n_tiles = tile0[s + 1] - first;
  const ScopeDesc d = scopes[s];
  ScopeState* st = T.state + s;
  const uint32_t m = (uint32_t)d.samp_m;
  if (lt == 0 && tid == 0) {
    // everything but the prediction, which is written by the CTA that finishes the scope
    st->cand_count = 0; st->tau = 0; st->q = 0; st->gt = 0; st->early_bad = 0; st->used_dense = 0; st->top_bin_max = 0;
  }
  if (tid < kGather) {
    const uint32_t li = lt * kGather + tid;
    if (li < m) __stcg(T.samp_val + d.samp_base + li, sample_value(T, d, s, li));
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    __stcg(flags + blockIdx.x, call);
    __threadfence();
  }
  __syncthreads();
  {
    int all = 1;
    for (uint32_t x = tid; x < n_tiles; x += kPredictThreads) all &= __ldcg(flags + first + x) == call ? 1 : 0;
    s_is_last = 1;
    __syncthreads();
    if (!all) s_is_last = 0;
    __syncthreads();
  }
#ifdef GD_PHASE_STAMPS
  if (tid == 0) atomicMax(reinterpret_cast<unsigned long long*>(T.ctl) + 22, global_timer_ns());
#endif
  if (!s_is_last) return;
  __threadfence();

  // ---- the scope's sample is complete: select both ranks
  const float* vals = T.samp_val + d.samp_base;
  for (uint32_t b = tid; b < kRadixBins0; b += kPredictThreads) s_hist[b] = 0;
  if (tid == 0) {
    s_rank[0] = (uint32_t)d.samp_rank;                     // the lower bound (a rank with a safety margin) ...
    s_rank[1] = (uint32_t)rank_hi_of(d);                   // ... and the estimate of the threshold itself
  }
  __syncthreads();
  // The whole sample into shared memory (at most 32 keys per thread: 128 KB), eight loads per thread in flight at a
  // time.  The loops below are rolled on purpose: this code runs once per call, after the fused pass of the call
  // before has swept the L2, so every instruction line is fetched from DRAM - unrolled 32 times with the keys in
  // registers, the same selection took 9 us, most of it instruction fetches; rolled, 6 us.
  constexpr int kKeys = 32;
  const uint32_t* keys = reinterpret_cast<const uint32_t*>(smem_keys);
  uint32_t zeros = 0;                                      // samples that are +-0: counted privately
  {
    constexpr int kBatch = 8;                               // loads per thread in flight at a time
    uint32_t* wkeys = reinterpret_cast<uint32_t*>(smem_keys);
    for (uint32_t li0 = tid; li0 < m; li0 += kBatch * kPredictThreads) {
      uint32_t w[kBatch];
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        const uint32_t li = li0 + (uint32_t)u * kPredictThreads;
        w[u] = li < m ? __float_as_uint(__ldcg(vals + li)) : 0u;
      }
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        const uint32_t li = li0 + (uint32_t)u * kPredictThreads;
        if (li < m) {
          wkeys[li] = w[u];
          // first digit: counted as the keys arrive
          const uint32_t key = w[u] & kAbsMask;
          if (key == 0u) ++zeros;
          else atomicAdd(&s_hist[key >> kShift0], 1u);
        }
      }
    }
  }
  const uint32_t per_thread = (m + kPredictThreads - 1u) / kPredictThreads;   // <= kKeys
  static_assert(kLocalSampleMax == (uint32_t)kKeys * kPredictThreads, "the shared-memory copy of the sample");
  const uint32_t zeros_mine = zeros;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) zeros += __shfl_xor_sync(0xFFFFFFFFu, zeros, o);
  if (lane == 0 && zeros) atomicAdd(&s_hist[0], zeros);
  __syncthreads();
  find_ranks(s_hist, kRadixBins0, s_rank, 2, s_bin, s_above);
  const uint32_t pa = s_bin[0], pb = s_bin[1];             // first digits of the two ranks
  const uint32_t ra = s_rank[0] - s_above[0], rb = s_rank[1] - s_above[1];   // ranks inside those bins
  __syncthreads();
  for (uint32_t b = tid; b < kRadixBins0; b += kPredictThreads) s_hist[b] = 0;
  if (tid == 0) { s_rank[0] = ra; s_rank[1] = rb; }
  __syncthreads();

  // second digit: the keys under the first rank's first digit in the lower half of the histogram, those under the
  // second rank's (if it differs) in the upper half
#pragma unroll 4
  for (uint32_t j = 0; j < per_thread; ++j) {
    const uint32_t li = j * kPredictThreads + tid;
    if (li < m) {
      const uint32_t key = keys[li] & kAbsMask;
      const uint32_t top = key >> kShift0, dig = (key >> kShift1) & 1023u;
      if (key == 0u) {}
      else if (top == pa) atomicAdd(&s_hist[dig], 1u);
      else if (top == pb) atomicAdd(&s_hist[1024u + dig], 1u);
    }
  }
  zeros = zeros_mine;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) zeros += __shfl_xor_sync(0xFFFFFFFFu, zeros, o);
  if (lane == 0 && zeros) {
    if (pa == 0u) atomicAdd(&s_hist[0], zeros);
    else if (pb == 0u) atomicAdd(&s_hist[1024u], zeros);
  }
  __syncthreads();
  uint32_t da, db;
  if (pa == pb) {
    find_ranks(s_hist, 1024u, s_rank, 2, s_bin, s_above);
    da = s_bin[0]; db = s_bin[1];
  } else {
    find_ranks(s_hist, 1024u, s_rank, 1, s_bin, s_above);
    da = s_bin[0];
    __syncthreads();
    find_ranks(s_hist + 1024, 1024u, s_rank + 1, 1, s_bin + 1, s_above + 1);
    db = s_bin[1];
  }
  if (tid == 0) {
    // lower edges of the 21-bit buckets
    st->tau_lo = ((pa << 10) | da) << kShift1;
    st->tau_hi = ((pb << 10) | db) << kShift1;
    __threadfence();
    if (s < kSmemScopes) __stcg(flags + gather_ctas + s, call);   // the scope's prediction is final (see the clearing CTAs)
#ifdef GD_PHASE_STAMPS
    atomicMax(reinterpret_cast<unsigned long long*>(T.ctl) + 23, global_timer_ns());
#endif
  }
}

}  // namespace

static_assert(kLocalSampleMax == 32u * kPredictThreads, "what one CTA keeps in shared memory: 32 keys per thread");

// gather_ctas: CTAs that gather the samples (the scopes' sample tiles of gather_tile values); flags: one word per such CTA; tables_src: the host image of the
// tables (at most kSetupBlobBytes); scopes_off, tile0_off: where the scope descriptors and the first sample tile of
// every scope start in it; state_off: where the scope states lie inside the region to clear.
cudaError_t launch_setup_predict(const DevTables& T, uint32_t gather_ctas, uint32_t gather_tile, uint32_t* flags,
                                 void* tables_dst,
                                 const void* tables_src, size_t tables_bytes, void* zero_dst, size_t zero_bytes, size_t state_off, size_t scopes_off,
                                 size_t tile0_off, cudaStream_t stream, uint32_t* call_out, uint32_t* clearing_ctas_out) {
  if (tables_bytes > kSetupBlobBytes) return cudaErrorInvalidValue;
  ProfileScope prof(stream, PT_SETUP_PREDICT);
  static PerDeviceInt configured;                          // the kernel's shared-memory attribute is per device
  int dev = -1;
  if (configured.get(&dev) == 0) {
    if (dev < 0) return cudaErrorInvalidDevice;
    cudaError_t e = cudaFuncSetAttribute(setup_predict_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kKeysBytes);
    if (e != cudaSuccess) return e;
    configured.set(dev, 1);
  }
  // The number of the call, which marks the finished sample tiles: starts at a value that differs from process to
  // process and does not repeat within one (for 2^32 calls).  A stale mark that happened to equal it would only make
  // a prediction start from an incomplete sample, and the prediction never affects results.
  static std::atomic<uint32_t> next_call{(uint32_t)std::chrono::steady_clock::now().time_since_epoch().count() | 1u};
  const uint32_t call = next_call.fetch_add(1u, std::memory_order_relaxed);
  SetupBlob blob;
  std::memcpy(blob.bytes, tables_src, tables_bytes);
  const uint64_t zero_vec = zero_bytes / 16;              // both regions are 256-byte aligned and padded
  uint64_t zero_ctas = (zero_vec + kPredictThreads * 4 - 1) / (kPredictThreads * 4);
  uint64_t cap = (uint64_t)sm_count();
  if (cap > kStartMarks) cap = kStartMarks;
  if (zero_ctas > cap) zero_ctas = cap;
  if (zero_ctas < 1) zero_ctas = 1;
  const uint64_t state_beg = state_off / 16;
  const uint64_t state_end = (state_off + sizeof(ScopeState) * (size_t)T.n_scopes + 15) / 16;
  const cudaError_t le = launch_dependent(setup_predict_kernel, dim3((unsigned)(gather_ctas + zero_ctas)), dim3(kPredictThreads), kKeysBytes, stream,
                                          T, blob, gather_ctas, gather_tile, call, flags, (uint4*)tables_dst, (uint32_t)(tables_bytes / 16),
                                          (uint4*)zero_dst, zero_vec, state_beg, state_end, (uint32_t)scopes_off, (uint32_t)tile0_off);
  if (le != cudaSuccess) return le;
  GD_LAUNCH_CHECK();
  *call_out = call;
  *clearing_ctas_out = (uint32_t)zero_ctas;
  return cudaSuccess;
}

}  // namespace gd
