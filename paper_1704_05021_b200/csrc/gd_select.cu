// Threshold selection of gd_compress (Algorithm 1, "Select threshold: R% of |grad| is smaller"):
// an exact radix select on the bit pattern of |v|, run over three kinds of lists -
//   the sample   -> tau_lo, the predicted lower bound used by the fused pass,
//   the candidate list the fused pass emitted -> tau and the tie quota (the usual case),
//   the dense range itself -> the same, for scopes whose prediction failed.
#include "gd_internal.cuh"

namespace gd {

namespace {

__device__ __forceinline__ uint32_t mix32(uint32_t x) {
  x ^= x >> 16; x *= 0x7FEB352Du; x ^= x >> 15; x *= 0x846CA68Bu; x ^= x >> 16;
  return x;
}

// One thread per sample: stratum li of scope s covers [a, b) of the scope and one position inside
// it is read.  The sample only steers the prediction; any sample gives the same final result.
__global__ void __launch_bounds__(kThreads) sample_gather_kernel(const __grid_constant__ DevTables T,
                                                                 uint64_t samp_total) {
  const uint64_t i = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
  if (i >= samp_total) return;
  const uint32_t s = range_of(T.samp_off, T.n_scopes, i);
  const ScopeDesc& d = T.scopes[s];
  const uint64_t li = i - d.samp_base;
  const uint64_t ns = d.hi - d.lo, m = d.samp_m;
  const uint64_t a = (li * ns) / m, b = ((li + 1) * ns) / m;
  const uint64_t width = b - a;
  uint64_t pos = d.lo + a;
  if (width > 1) pos += mix32((uint32_t)li * 0x9E3779B9u + s) % width;
  T.samp_val[i] = __fadd_rn(__ldg(T.grad + pos), T.residual[pos]);
}

// One pass histograms one digit of the 31-bit magnitude key among the elements that match the
// digits fixed so far; the last CTA of a scope to finish turns the histogram into the next digit.
// After three passes (11 + 10 + 10 bits) the state holds the rank-th largest key, the number of
// keys above it and how many keys equal to it belong to the top `rank`.
template <int VIEW>
__global__ void __launch_bounds__(kThreads) select_pass_kernel(const __grid_constant__ DevTables T, int pass,
                                                               uint32_t total_tiles) {
  constexpr int LK = VIEW == V_SAMPLE ? L_SAMP : (VIEW == V_CAND ? L_CAND : L_DSEL);
  constexpr uint32_t TILE = VIEW == V_DENSE ? kDenseSelTile : kTile;
  __shared__ uint32_t sh[kRadixBins0];
  __shared__ unsigned long long s_warp[kWarps];
  __shared__ int s_last;
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  if (T.ctl->status != GD_OK) return;   // set only by an earlier kernel of this call
  if (VIEW == V_DENSE && !(T.flags & GD_FLAG_NO_PREDICTION) && T.ctl->dense_needed == 0u) return;
  const uint32_t* tile0 = T.tile0[LK];
  const int shift = pass == 0 ? kShift0 : (pass == 1 ? kShift1 : kShift2);
  const int bits = pass == 0 ? kRadixBits0 : 10;
  const uint32_t nbins = 1u << bits;
  const int pshift = pass == 1 ? kShift0 : kShift1;   // shift that exposes the digits fixed so far

  for (uint32_t t = blockIdx.x; t < total_tiles; t += gridDim.x) {
    const uint32_t s = scope_of_tile(tile0, T.n_scopes, t);
    const ScopeDesc& d = T.scopes[s];
    ScopeState* st = T.state + s;
    const uint32_t first = __ldg(tile0 + s), ntiles = __ldg(tile0 + s + 1) - first;
    const uint32_t lt = t - first;

    uint64_t len, rank;
    const float* vals;
    if (VIEW == V_SAMPLE) {
      len = d.samp_m; vals = T.samp_val + d.samp_base; rank = d.samp_rank;
    } else if (VIEW == V_CAND) {
      if (!predicted_ok(T, d, *st)) continue;
      len = st->cand_count; vals = T.cand_val + d.cand_base; rank = d.k;
    } else {
      if (predicted_ok(T, d, *st)) continue;
      len = d.hi - d.lo; vals = T.residual + d.lo; rank = d.k;
    }
    uint32_t prefix = 0;
    uint64_t gt = 0;
    if (pass > 0) { prefix = st->sel[VIEW].prefix; rank = st->sel[VIEW].rank; gt = st->sel[VIEW].gt; }

    __syncthreads();                       // previous iteration is done with sh / s_last
    for (uint32_t b = tid; b < nbins; b += kThreads) sh[b] = 0;
    __syncthreads();
    const uint64_t beg = (uint64_t)lt * TILE;
    const uint64_t end = (beg + TILE < len) ? beg + TILE : len;
    for (uint64_t i0 = beg + (tid & ~31u); i0 < end; i0 += kThreads) {   // warp-uniform trip count
      const uint64_t i = i0 + lane;
      uint32_t digit = 0xFFFFFFFFu;                                      // "does not count"
      if (i < end) {
        const uint32_t key = __float_as_uint(vals[i]) & kAbsMask;
        if (pass == 0 || (key >> pshift) == prefix) digit = (key >> shift) & (nbins - 1u);
      }
      const uint32_t d0 = __shfl_sync(0xFFFFFFFFu, digit, 0);
      if (__all_sync(0xFFFFFFFFu, digit == d0)) {        // whole warp in one bin: one add
        if (lane == 0 && d0 != 0xFFFFFFFFu) atomicAdd(&sh[d0], 32u);
      } else if (digit != 0xFFFFFFFFu) {
        atomicAdd(&sh[digit], 1u);
      }
    }
    __syncthreads();
    unsigned long long* ghist = T.hist + (size_t)s * kRadixBins0;
    for (uint32_t b = tid; b < nbins; b += kThreads) {
      const uint32_t c = sh[b];
      if (c) atomicAdd(ghist + b, (unsigned long long)c);
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(&st->done[VIEW][pass], 1u) == ntiles - 1u) ? 1 : 0;
    __syncthreads();
    if (!s_last) continue;
    __threadfence();

    // Last CTA of the scope: thread x owns the bins [top - C + 1, top], top = nbins - 1 - x * C.
    const uint32_t C = nbins / kThreads;
    const uint32_t top = nbins - 1u - tid * C;
    unsigned long long cs = 0;
    for (uint32_t j = 0; j < C; ++j) cs += __ldcg(ghist + top - j);
    unsigned long long inc = cs;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
      if ((int)lane >= o) inc += y;
    }
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    unsigned long long above = inc - cs;
    for (uint32_t w = 0; w < warp; ++w) above += s_warp[w];
    if (tid == kThreads - 1 && above + cs < rank) atomicCAS(&T.ctl->status, (int)GD_OK, (int)GD_ERR_INTERNAL);
    const bool owner = rank == 0 ? (tid == 0) : (above < rank && rank <= above + cs);
    if (owner) {
      uint32_t digit = nbins - 1u;
      unsigned long long acc = 0;
      if (rank != 0) {
        acc = above;
        for (uint32_t j = 0; j < C; ++j) {
          const unsigned long long c = __ldcg(ghist + top - j);
          if (acc + c >= rank) { digit = top - j; break; }
          acc += c;
        }
      }
      const uint32_t nprefix = (prefix << bits) | digit;
      const uint64_t nrank = rank - acc, ngt = gt + acc;
      st->sel[VIEW].prefix = nprefix;
      st->sel[VIEW].rank = nrank;
      st->sel[VIEW].gt = ngt;
      if (pass == 2) {
        if (VIEW == V_SAMPLE) {
          st->tau_lo = nprefix;
        } else {
          st->tau = nprefix; st->q = nrank; st->gt = ngt;
          if (VIEW == V_DENSE) st->used_dense = 1u;
        }
      }
    }
    __syncthreads();
    for (uint32_t b = tid; b < nbins; b += kThreads) ghist[b] = 0ull;   // ready for the next pass
  }
}

}  // namespace

cudaError_t launch_sample_select(const DevTables& T, const uint32_t* tiles, uint64_t samp_total, cudaStream_t stream) {
  if (!samp_total) return cudaSuccess;
  const uint32_t blocks = (uint32_t)((samp_total + kThreads - 1) / kThreads);
  sample_gather_kernel<<<blocks, kThreads, 0, stream>>>(T, samp_total);
  GD_LAUNCH_CHECK();
  for (int pass = 0; pass < 3; ++pass) {
    select_pass_kernel<V_SAMPLE><<<tiles[L_SAMP], kThreads, 0, stream>>>(T, pass, tiles[L_SAMP]);
    GD_LAUNCH_CHECK();
  }
  return cudaSuccess;
}

cudaError_t launch_candidate_select(const DevTables& T, const uint32_t* tiles, cudaStream_t stream) {
  if (!tiles[L_CAND]) return cudaSuccess;
  for (int pass = 0; pass < 3; ++pass) {
    select_pass_kernel<V_CAND><<<tiles[L_CAND], kThreads, 0, stream>>>(T, pass, tiles[L_CAND]);
    GD_LAUNCH_CHECK();
  }
  return cudaSuccess;
}

cudaError_t launch_dense_select(const DevTables& T, const uint32_t* tiles, cudaStream_t stream) {
  if (!tiles[L_DSEL]) return cudaSuccess;
  const uint32_t cap = (uint32_t)sm_count() * 8u;
  const uint32_t grid = tiles[L_DSEL] < cap ? tiles[L_DSEL] : cap;
  for (int pass = 0; pass < 3; ++pass) {
    select_pass_kernel<V_DENSE><<<grid, kThreads, 0, stream>>>(T, pass, tiles[L_DSEL]);
    GD_LAUNCH_CHECK();
  }
  return cudaSuccess;
}

}  // namespace gd
