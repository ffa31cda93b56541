// Survivor compaction of gd_compress (Algorithm 1, steps 3-5: mask, residual rewrite, sparse
// output), the two-means sums of Section 5.4, and the kernel that finishes a call (thresholds,
// shard offsets of Section 3, the means).
#include <atomic>

#include "gd_compact_body.cuh"

namespace gd {

namespace {

__global__ void __launch_bounds__(kThreads, 3) compact_dense_kernel(const __grid_constant__ DevTables T,
                                                                    uint32_t total_chunks, int do_finalize) {
  __shared__ CompactDenseSmem S;
  compact_dense_body(T, total_chunks, do_finalize, S);
}

// The compaction over the candidate lists also takes over, first, the compaction over the dense range of the
// scopes whose prediction failed (dense_chunks != 0; rare), so that no launch is spent on looking at a flag.
__global__ void __launch_bounds__(kThreads, 3) compact_kernel(const __grid_constant__ DevTables T, uint32_t total_tiles,
                                                              int do_finalize, uint32_t dense_chunks) {
  if (dense_chunks != 0u && T.ctl->dense_needed != 0u) {
    __shared__ CompactDenseSmem S;
    compact_dense_outlined(T, dense_chunks, S);
  }
  compact_cand_body(T, total_tiles, do_finalize);
}

// Sampled-threshold mode: the candidate lists ARE the survivors.  Copies every scope's list to its
// place in the output (scopes concatenated in index order), clears the survivors' residual slots
// unless the fused pass has done so already, and lets the last CTA finish the call with the survivor
// count found here.
__global__ void __launch_bounds__(kThreads) pack_sampled_kernel(const __grid_constant__ DevTables T) {
  __shared__ unsigned long long s_part[kWarps];
  __shared__ unsigned long long s_off;
  __shared__ int s_last;
  __shared__ SmemTables s_tab;
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const ScopeDesc* scopes;
  const uint32_t* tile0;
  load_tables(T, L_CAND, &s_tab, &scopes, &tile0);
  __syncthreads();
  const uint32_t t = blockIdx.x;
  const uint32_t s = scope_of_tile(tile0, T.n_scopes, t);
  const ScopeDesc& d = scopes[s];
  // survivors of the scopes before s (and, for the last CTA, of all scopes)
  auto count_before = [&](uint32_t upto) -> unsigned long long {
    unsigned long long part = 0;
    for (uint32_t x = tid; x < upto; x += kThreads) {
      const unsigned long long m = T.state[x].cand_count, c = scopes[x].cand_cap;
      part += m < c ? m : c;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, o);
    __syncthreads();
    if (lane == 0) s_part[warp] = part;
    __syncthreads();
    if (tid == 0) {
      unsigned long long tot = 0;
      for (int w = 0; w < kWarps; ++w) tot += s_part[w];
      s_off = tot;
    }
    __syncthreads();
    return s_off;
  };
  const bool cleared = !(T.flags & GD_FLAG_NO_EARLY_ZERO);   // the fused pass wrote +0 over every listed survivor's slot
  const unsigned long long m_all = T.state[s].cand_count;
  const uint64_t m = m_all < d.cand_cap ? m_all : d.cand_cap;
  const uint64_t beg = (uint64_t)(t - tile0[s]) * kTile;
  if (beg < m) {
    const uint64_t out_off = count_before(s);
    const uint64_t end = (beg + kTile < m) ? beg + kTile : m;
    uint32_t ib[16], vb[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const uint64_t i = beg + (uint64_t)j * kThreads + tid;
      ib[j] = i < end ? T.cand_idx[d.cand_base + i] : 0u;
      vb[j] = i < end ? __float_as_uint(T.cand_val[d.cand_base + i]) : 0u;
    }
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const uint64_t i = beg + (uint64_t)j * kThreads + tid;
      if (i < end && ib[j] < T.n && out_off + i < T.k_total) {
        T.out_idx[out_off + i] = ib[j];
        T.out_val[out_off + i] = __uint_as_float(vb[j]);
        if (!cleared) T.residual[ib[j]] = 0.0f;
        if (T.delta_base) T.delta_base[ib[j]] = __fadd_rn(T.delta_base[ib[j]], __uint_as_float(vb[j]));
      }
    }
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(&T.ctl->compact_done[0], 1u) == gridDim.x - 1u) ? 1 : 0;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  finalize_call(T, count_before(T.n_scopes));
}

// Divides the accumulated sums by their counts when there are too many pairs for the finishing CTA.
__global__ void __launch_bounds__(kThreads) means_kernel(const __grid_constant__ DevTables T) {
  const uint64_t stride = (uint64_t)gridDim.x * kThreads;
  for (uint64_t e = (uint64_t)blockIdx.x * kThreads + threadIdx.x; e < 2 * T.n_pairs; e += stride) {
    const unsigned long long c = T.cnts[e];
    T.out_means[e] = c ? (float)(T.sums[e] / (double)c) : 0.0f;
  }
}

// GD_FLAG_QUANT_ERROR_FEEDBACK: the compaction left v in the residual slots of the survivors; once the
// decode table (out_means) is final, every such slot becomes v minus the value its survivor decodes to.
__global__ void __launch_bounds__(kThreads) feedback_kernel(const __grid_constant__ DevTables T) {
  const uint64_t stride = (uint64_t)gridDim.x * kThreads;
  for (uint64_t j = (uint64_t)blockIdx.x * kThreads + threadIdx.x; j < T.k_total; j += stride) {
    const uint32_t w = T.out_idx[j];
    const uint64_t idx = w & kAbsMask;
    if (idx >= T.n) continue;
    const uint64_t pr = pair_of(T.layer_off, T.pair_off, T.layer_cols, T.n_layers, idx);
    T.residual[idx] = __fsub_rn(T.residual[idx], T.out_means[2 * pr + (w >> 31)]);
  }
}

// Self-test kernel of the bounded waits: tile 1 waits on tile 0, which nothing publishes; tile 2
// then meets the aborted tile 1.
__global__ void __launch_bounds__(32) bounded_wait_selftest_kernel(Ctl* ctl, uint4* desc, uint32_t spin_limit) {
  uint64_t ex_a, ex_b;
  const bool ok1 = tile_lookback(desc, 1, 0, 5, 0, ex_a, ex_b, ctl, spin_limit, 0);
  const bool ok2 = tile_lookback(desc, 2, 0, 7, 0, ex_a, ex_b, ctl, spin_limit, 0);
  if (lane_id() == 0) {
    ctl->n_scopes = ok1 ? 0u : 1u;
    ctl->n_scopes_predicted = ok2 ? 0u : 1u;
  }
}

}  // namespace

cudaError_t launch_bounded_wait_selftest(void* workspace, uint32_t spin_limit, cudaStream_t stream) {
  cudaError_t e = cudaMemsetAsync(workspace, 0, 512, stream);
  if (e != cudaSuccess) return e;
  bounded_wait_selftest_kernel<<<1, 32, 0, stream>>>((Ctl*)workspace, (uint4*)((unsigned char*)workspace + 256), spin_limit);
  GD_LAUNCH_CHECK();
  return cudaSuccess;
}

cudaError_t launch_finalize(const DevTables& T, cudaStream_t stream) {
  ProfileScope prof(stream, PT_FINALIZE);
  finalize_kernel<<<1, kThreads, 0, stream>>>(T);
  GD_LAUNCH_CHECK();
  return cudaSuccess;
}

cudaError_t launch_means(const DevTables& T, cudaStream_t stream) {
  ProfileScope prof(stream, PT_MEANS);
  uint64_t blocks = (2 * T.n_pairs + kThreads - 1) / kThreads;
  const uint64_t cap = (uint64_t)sm_count() * 8;
  if (blocks > cap) blocks = cap;
  means_kernel<<<(unsigned)blocks, kThreads, 0, stream>>>(T);
  GD_LAUNCH_CHECK();
  return cudaSuccess;
}

cudaError_t launch_feedback(const DevTables& T, cudaStream_t stream) {
  if (!T.k_total) return cudaSuccess;
  ProfileScope prof(stream, PT_FEEDBACK);
  uint64_t blocks = (T.k_total + kThreads - 1) / kThreads;
  const uint64_t cap = (uint64_t)sm_count() * 8;
  if (blocks > cap) blocks = cap;
  feedback_kernel<<<(unsigned)blocks, kThreads, 0, stream>>>(T);
  GD_LAUNCH_CHECK();
  return cudaSuccess;
}

cudaError_t launch_pack_sampled(const DevTables& T, const uint32_t* tiles, cudaStream_t stream) {
  if (!tiles[L_CAND]) return launch_finalize(T, stream);   // nothing can survive: finish with count 0
  ProfileScope prof(stream, PT_PACK_SAMPLED);
  pack_sampled_kernel<<<tiles[L_CAND], kThreads, 0, stream>>>(T);
  GD_LAUNCH_CHECK();
  return cudaSuccess;
}

// dense = true: the dense compaction alone (no prediction in this call).  dense = false: the compaction over the
// candidate lists, which also runs the dense one for scopes whose prediction failed.
cudaError_t launch_compact(const DevTables& T, const uint32_t* tiles, bool dense, bool finalize, cudaStream_t stream) {
  const uint32_t total = tiles[dense ? L_DCOMP : L_CAND];
  if (!total) return finalize ? launch_finalize(T, stream) : cudaSuccess;
  ProfileScope prof(stream, dense ? PT_DENSE_COMPACT : PT_CAND_COMPACT);
  // The kernels take tiles from a ticket until none is left: no more CTAs than are resident at once,
  // or the later ones would only start, find nothing and leave.
  static PerDeviceInt resident[2];                         // per kernel and device
  int dev = -1;
  int r = resident[dense ? 1 : 0].get(&dev);
  if (r == 0) {
    cudaError_t e = dense ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&r, compact_dense_kernel, kThreads, 0)
                          : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&r, compact_kernel, kThreads, 0);
    if (e != cudaSuccess || r <= 0) return cudaErrorLaunchFailure;
    resident[dense ? 1 : 0].set(dev, r);
  }
  const uint32_t cap = (uint32_t)sm_count() * (uint32_t)r;
  const uint32_t most = (!dense && tiles[L_DCOMP] > total) ? tiles[L_DCOMP] : total;   // it may take over the dense chunks
  const uint32_t grid = most < cap ? most : cap;
  if (dense)
    compact_dense_kernel<<<grid, kThreads, 0, stream>>>(T, total, finalize ? 1 : 0);
  else
    compact_kernel<<<grid, kThreads, 0, stream>>>(T, total, finalize ? 1 : 0, tiles[L_DCOMP]);
  GD_LAUNCH_CHECK();
  return cudaSuccess;
}

}  // namespace gd
