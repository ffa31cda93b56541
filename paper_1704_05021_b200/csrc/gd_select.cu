// Threshold selection of gd_compress (Algorithm 1, the threshold-selection step):
// an exact radix select on the bit pattern of |v|, run over three kinds of lists -
//   the sample   -> tau_lo, the predicted lower bound used by the fused pass,
//   the candidate list the fused pass emitted -> tau and the tie quota (the usual case),
//   the dense range itself -> the same, for scopes whose prediction failed.
//
// One cooperative launch does a whole selection: per pass every CTA histograms one digit of the
// 31-bit magnitude key (11 + 10 + 10 bits) over its share of the tiles, the grid meets at a
// barrier, and every CTA works out the next digit of the scopes it touches from the finished
// histogram.  The barrier is a counter in the workspace; its wait is bounded like every other wait.
#include <atomic>

#include "gd_select_body.cuh"

namespace gd {

namespace {

// One cooperative launch = one selection.  The selection over the candidate lists also takes over, first, the
// selection over the dense range of the scopes whose prediction failed (dense_tiles != 0): such scopes are rare,
// and two launches that start, look at a flag and leave cost every call about six microseconds.
template <int VIEW, bool MANY>
__global__ void __launch_bounds__(kThreads, (MANY && VIEW != V_DENSE) ? 2 : 4) select_kernel(const __grid_constant__ DevTables T, uint32_t total_tiles,
                                                                                             uint32_t dense_tiles) {
  __shared__ SelectSmem<VIEW, MANY> S;
  pdl_trigger();   // (the fused pass, enqueued behind the selection on the sample, may be brought onto the GPU from now on)
  if (VIEW == V_CAND) {
    // (the dense selection borrows this selection's shared memory, which is large enough: asserted below)
    if (dense_tiles != 0u && T.ctl->dense_needed != 0u)
      select_dense_outlined<MANY>(T, dense_tiles, *reinterpret_cast<SelectSmem<V_DENSE, MANY>*>(&S));
  }
  select_body<VIEW, MANY>(T, total_tiles, S);
}

static_assert(sizeof(SelectSmem<V_DENSE, false>) <= sizeof(SelectSmem<V_CAND, false>) &&
              sizeof(SelectSmem<V_DENSE, true>) <= sizeof(SelectSmem<V_CAND, true>), "the dense selection borrows the memory");

template <int VIEW, bool MANY>
cudaError_t launch_select_impl(const DevTables& T, uint32_t total_tiles, uint32_t dense_tiles, uint32_t ctas_per_sm,
                               cudaStream_t stream) {
  if (!total_tiles) return cudaSuccess;
  ProfileScope prof(stream, VIEW == V_SAMPLE ? PT_SAMPLE_SELECT : (VIEW == V_CAND ? PT_CAND_SELECT : PT_DENSE_SELECT));
  static PerDeviceInt cached;                              // co-resident CTAs per SM of this kernel, per device
  int dev = -1;
  int resident = cached.get(&dev);
  if (resident == 0) {
    int r = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&r, select_kernel<VIEW, MANY>, kThreads, 0) != cudaSuccess || r <= 0)
      return cudaErrorLaunchFailure;
    resident = r;
    cached.set(dev, r);
  }
  const uint32_t per_sm = ctas_per_sm < (uint32_t)resident ? ctas_per_sm : (uint32_t)resident;
  uint32_t grid = (uint32_t)sm_count() * per_sm;
  // no more CTAs than tiles - counting the dense tiles this launch may have to take over, so that the
  // rare dense selection is not left to the few CTAs a short candidate list would get
  const uint32_t most_tiles = total_tiles > dense_tiles ? total_tiles : dense_tiles;
  if (grid > most_tiles) grid = most_tiles;
  DevTables Tc = T;
  void* args[] = {(void*)&Tc, (void*)&total_tiles, (void*)&dense_tiles};
  cudaError_t e = cudaLaunchCooperativeKernel((const void*)select_kernel<VIEW, MANY>, dim3(grid), dim3(kThreads), args, 0, stream);
  if (e != cudaSuccess) return e;
  note_launches(1);
  return cudaSuccess;
}

template <int VIEW>
cudaError_t launch_select(const DevTables& T, uint32_t total_tiles, uint32_t dense_tiles, uint32_t ctas_per_sm,
                          cudaStream_t stream) {
  return T.n_scopes > kSmemScopes ? launch_select_impl<VIEW, true>(T, total_tiles, dense_tiles, ctas_per_sm, stream)
                                  : launch_select_impl<VIEW, false>(T, total_tiles, dense_tiles, ctas_per_sm, stream);
}

}  // namespace

cudaError_t launch_sample_select(const DevTables& T, const uint32_t* tiles, cudaStream_t stream) {
  return launch_select<V_SAMPLE>(T, tiles[L_SAMP], 0u, 2, stream);
}

cudaError_t launch_candidate_select(const DevTables& T, const uint32_t* tiles, cudaStream_t stream) {
  return launch_select<V_CAND>(T, tiles[L_CAND], tiles[L_DSEL], 2, stream);   // and the dense selection, if needed
}

cudaError_t launch_dense_select(const DevTables& T, const uint32_t* tiles, cudaStream_t stream) {
  return launch_select<V_DENSE>(T, tiles[L_DSEL], 0u, 8, stream);
}

}  // namespace gd
