// Kernels of gd_compress: Algorithm 1 (GradDrop) of Aji & Heafield 2017 on one flat fp32 gradient.
//
// Pipeline, all on the caller's stream, no host round trip:
//   sample_gather        v = g + r at a stratified sample of positions (prediction only)
//   select_pass<SAMPLE>  x3: exact radix select of the predicted lower bound tau_lo on the sample
//   add_emit             the one full pass: r <- g + r (Alg. 1 step 1), and every entry with
//                        |v| >= tau_lo is appended, in index order, to a candidate list through a
//                        single-pass decoupled look-back scan
//   select_pass<CAND>    x3: exact radix select (31-bit |v| key, 11+10+10 bits) of the k-th largest
//                        key among the candidates -> tau, number of ties kept   (Alg. 1 step 2)
//   compact<CAND>        survivors (key > tau, plus the first q ties) -> out_idx/out_val in index
//                        order, residual slot <- +0 (Alg. 1 steps 3-5), two-means partial sums
//   select_pass<DENSE>, compact<DENSE>: the same two steps over the whole dense range, run only
//                        for scopes whose prediction failed (fewer than k candidates, or more
//                        than the list holds); they exit at once otherwise
//   finalize             thresholds, shard offsets (Section 3), the two means (Section 5.4)
//
// The prediction never changes the result: a scope either has at least k candidates, in which
// case the k largest keys and all their ties are in the list, or it is redone densely.
#include "gd_internal.cuh"

namespace gd {

// ---------------------------------------------------------------- 128-bit look-back descriptors
// One descriptor per tile: {flag:2 | count_a:62, count_b:64}, written and read as one 128-bit
// access so that flag and both counts are always seen together.
__device__ __forceinline__ void st_desc(uint4* p, uint64_t lo, uint64_t hi) {
  asm volatile("{\n\t.reg .b128 t;\n\tmov.b128 t, {%1, %2};\n\tst.relaxed.gpu.global.b128 [%0], t;\n\t}"
               ::"l"(p), "l"(lo), "l"(hi) : "memory");
}
__device__ __forceinline__ void ld_desc(const uint4* p, uint64_t& lo, uint64_t& hi) {
  asm volatile("{\n\t.reg .b128 t;\n\tld.relaxed.gpu.global.b128 t, [%2];\n\tmov.b128 {%0, %1}, t;\n\t}"
               : "=l"(lo), "=l"(hi) : "l"(p) : "memory");
}

__device__ __forceinline__ uint64_t warp_sum(uint64_t x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
  return x;
}

// Decoupled look-back over the tiles [first, t) of one scope, run by one full warp.  Publishes this
// tile's totals, waits (bounded) for its predecessors and returns the exclusive prefixes.  A wait
// that runs out marks the tile aborted, records GD_ERR_DEVICE_TIMEOUT and returns false; tiles
// that meet an aborted predecessor abort too, so nothing waits on a tile that gave up.
__device__ bool tile_lookback(uint4* desc, uint32_t t, uint32_t first, uint64_t tot_a, uint64_t tot_b,
                              uint64_t& ex_a, uint64_t& ex_b, Ctl* ctl) {
  const uint32_t lane = lane_id();
  ex_a = 0;
  ex_b = 0;
  if (t == first) {
    if (lane == 0) st_desc(desc + t, pack_desc(F_PREFIX, tot_a), tot_b);
    return true;
  }
  if (lane == 0) st_desc(desc + t, pack_desc(F_AGG, tot_a), tot_b);
  bool ok = true;
  int64_t cur = (int64_t)t - 1;
  for (;;) {
    const int64_t my = cur - (int64_t)lane;
    const bool real = my >= (int64_t)first;      // lanes before the scope's first tile act as a zero prefix
    uint64_t lo = pack_desc(F_PREFIX, 0), hi = 0;
    uint32_t nearest = 32, flag = F_PREFIX, spins = 0;
    for (;;) {
      if (real) ld_desc(desc + my, lo, hi);
      flag = (uint32_t)(lo & 3u);
      const uint32_t stop = __ballot_sync(0xFFFFFFFFu, flag >= F_PREFIX);
      const uint32_t inv = __ballot_sync(0xFFFFFFFFu, flag == F_INVALID);
      nearest = stop ? (uint32_t)__ffs((int)stop) - 1u : 32u;
      const uint32_t need = nearest >= 32u ? 0xFFFFFFFFu : ((1u << nearest) - 1u);
      if ((inv & need) == 0u) break;
      if (++spins > kLookbackSpinLimit) { ok = false; break; }
      if (spins > 8) __nanosleep(64);
    }
    if (!ok) break;
    const bool take = lane <= nearest;
    ex_a += warp_sum(take ? (lo >> 2) : 0ull);
    ex_b += warp_sum(take ? hi : 0ull);
    if (nearest < 32u) {
      const uint32_t ab = __ballot_sync(0xFFFFFFFFu, flag == F_ABORT);
      if ((ab >> nearest) & 1u) ok = false;
      break;
    }
    cur -= 32;
  }
  if (lane == 0) {
    if (ok) {
      st_desc(desc + t, pack_desc(F_PREFIX, ex_a + tot_a), ex_b + tot_b);
    } else {
      st_desc(desc + t, pack_desc(F_ABORT, 0), 0);
      atomicCAS(&ctl->status, (int)GD_OK, (int)GD_ERR_DEVICE_TIMEOUT);
    }
  }
  return ok;
}

// ---------------------------------------------------------------- sample for the prediction
__device__ __forceinline__ uint32_t mix32(uint32_t x) {
  x ^= x >> 16; x *= 0x7FEB352Du; x ^= x >> 15; x *= 0x846CA68Bu; x ^= x >> 16;
  return x;
}

// One thread per sample: stratum li of scope s covers [a, b) of the scope, one position inside it is
// read.  The sample only steers the prediction of tau_lo; any sample gives the same final result.
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

// ---------------------------------------------------------------- the fused full pass
// Tiles are aligned to kTile elements of the flat vector; a tile that straddles a scope boundary is
// processed once per scope, each pass touching only its own scope's elements.  Inside a tile, warp w
// owns 512 consecutive elements and reads them as four rounds of 128-bit loads (lane l, round j ->
// elements w*512 + j*128 + l*4 .. +3), so candidate order inside the warp is (round, lane, component).
__global__ void __launch_bounds__(kThreads, 4) add_emit_kernel(const __grid_constant__ DevTables T) {
  __shared__ uint32_t s_tile;
  __shared__ uint32_t s_wtot[kWarps];
  __shared__ uint64_t s_excl;
  __shared__ int s_ok;
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  if (tid == 0) s_tile = atomicAdd(&T.ctl->ticket[L_EMIT], 1u);
  __syncthreads();
  const uint32_t t = s_tile;
  const uint32_t* tile0 = T.tile0[L_EMIT];
  const uint32_t s = scope_of_tile(tile0, T.n_scopes, t);
  const ScopeDesc& d = T.scopes[s];
  const uint64_t lo = d.lo, hi = d.hi;
  const uint32_t first = __ldg(tile0 + s), ntiles = __ldg(tile0 + s + 1) - first;
  const uint32_t lt = t - first;
  const uint64_t base = (lo / kTile + lt) * (uint64_t)kTile;
  const uint32_t tau_lo = ((T.flags & GD_FLAG_NO_PREDICTION) || d.k == 0) ? 0xFFFFFFFFu : T.state[s].tau_lo;
  const uint64_t wbase = base + (uint64_t)warp * 512u + lane * 4u;

  float v[16];
  uint32_t cmask = 0;
  if (base >= lo && base + kTile <= hi) {
    float4 g4[4], r4[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) g4[j] = __ldcs(reinterpret_cast<const float4*>(T.grad + wbase + j * 128));
#pragma unroll
    for (int j = 0; j < 4; ++j) r4[j] = *reinterpret_cast<const float4*>(T.residual + wbase + j * 128);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float4 x;
      x.x = __fadd_rn(g4[j].x, r4[j].x);
      x.y = __fadd_rn(g4[j].y, r4[j].y);
      x.z = __fadd_rn(g4[j].z, r4[j].z);
      x.w = __fadd_rn(g4[j].w, r4[j].w);
      *reinterpret_cast<float4*>(T.residual + wbase + j * 128) = x;
      v[4 * j + 0] = x.x; v[4 * j + 1] = x.y; v[4 * j + 2] = x.z; v[4 * j + 3] = x.w;
    }
#pragma unroll
    for (int e = 0; e < 16; ++e)
      cmask |= ((__float_as_uint(v[e]) & kAbsMask) >= tau_lo ? 1u : 0u) << e;
  } else {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const uint64_t i = wbase + j * 128 + c;
        float x = 0.f;
        if (i >= lo && i < hi) {
          x = __fadd_rn(__ldg(T.grad + i), T.residual[i]);
          T.residual[i] = x;
          cmask |= ((__float_as_uint(x) & kAbsMask) >= tau_lo ? 1u : 0u) << (4 * j + c);
        }
        v[4 * j + c] = x;
      }
    }
  }

  // ranks inside the warp
  const uint32_t ltm = lanemask_lt();
  uint32_t wtotal = 0, rnd_off[4], before[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const uint32_t f = (cmask >> (4 * j)) & 15u;
    rnd_off[j] = wtotal;
    before[j] = 0;
    if (__any_sync(0xFFFFFFFFu, f != 0u)) {
      const uint32_t b0 = __ballot_sync(0xFFFFFFFFu, f & 1u), b1 = __ballot_sync(0xFFFFFFFFu, f & 2u);
      const uint32_t b2 = __ballot_sync(0xFFFFFFFFu, f & 4u), b3 = __ballot_sync(0xFFFFFFFFu, f & 8u);
      before[j] = __popc(b0 & ltm) + __popc(b1 & ltm) + __popc(b2 & ltm) + __popc(b3 & ltm);
      wtotal += __popc(b0) + __popc(b1) + __popc(b2) + __popc(b3);
    }
  }
  if (lane == 0) s_wtot[warp] = wtotal;
  __syncthreads();
  uint32_t woff = 0, total = 0;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) {
    const uint32_t c = s_wtot[w];
    woff += (w < (int)warp) ? c : 0u;
    total += c;
  }
  if (warp == 0) {
    uint64_t ex_a, ex_b;
    const bool ok = tile_lookback(reinterpret_cast<uint4*>(T.desc_emit), t, first, total, 0, ex_a, ex_b, T.ctl);
    if (lane == 0) { s_excl = ex_a; s_ok = ok ? 1 : 0; }
  }
  __syncthreads();
  if (!s_ok) return;
  const uint64_t excl = s_excl;
  if (cmask) {
    const uint64_t cap = d.cand_cap;
    uint32_t* cidx = T.cand_idx + d.cand_base;
    float* cval = T.cand_val + d.cand_base;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint32_t f = (cmask >> (4 * j)) & 15u;
      if (f) {
        uint64_t pos = excl + woff + rnd_off[j] + before[j];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          if (f & (1u << c)) {
            if (pos < cap) {
              cidx[pos] = (uint32_t)(wbase + j * 128 + c);
              cval[pos] = v[4 * j + c];
            }
            ++pos;
          }
        }
      }
    }
  }
  if (tid == 0 && lt == ntiles - 1) T.state[s].cand_count = excl + total;
}


// ---------------------------------------------------------------- exact radix select
// One pass histograms one digit of the 31-bit magnitude key among the elements that match the
// digits fixed so far; the last CTA of a scope to finish turns the histogram into the next digit.
// After three passes (11 + 10 + 10 bits) the state holds the rank-th largest key, the number of
// keys above it and how many keys equal to it belong to the top `rank`.
template <int VIEW>
__global__ void __launch_bounds__(kThreads) select_pass_kernel(const __grid_constant__ DevTables T, int pass) {
  constexpr int LK = VIEW == V_SAMPLE ? L_SAMP : (VIEW == V_CAND ? L_CAND : L_DSEL);
  constexpr uint32_t TILE = VIEW == V_DENSE ? kDenseSelTile : kTile;
  __shared__ uint32_t sh[kRadixBins0];
  __shared__ unsigned long long s_warp[kWarps];
  __shared__ int s_last;
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  if (T.ctl->status != GD_OK) return;   // set only by an earlier kernel of this call
  const uint32_t t = blockIdx.x;
  const uint32_t* tile0 = T.tile0[LK];
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
    if (!predicted_ok(T, d, *st)) return;
    len = st->cand_count; vals = T.cand_val + d.cand_base; rank = d.k;
  } else {
    if (predicted_ok(T, d, *st)) return;
    len = d.hi - d.lo; vals = T.residual + d.lo; rank = d.k;
  }
  const int shift = pass == 0 ? kShift0 : (pass == 1 ? kShift1 : kShift2);
  const int bits = pass == 0 ? kRadixBits0 : 10;
  const uint32_t nbins = 1u << bits;
  const int pshift = pass == 1 ? kShift0 : kShift1;   // shift that exposes the digits fixed so far
  uint32_t prefix = 0;
  uint64_t gt = 0;
  if (pass > 0) { prefix = st->sel[VIEW].prefix; rank = st->sel[VIEW].rank; gt = st->sel[VIEW].gt; }

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
  if (!s_last) return;
  __threadfence();

  // Last CTA of the scope: thread x owns the chunk of bins [top - x*C - C + 1, top - x*C], top first.
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

// ---------------------------------------------------------------- compaction of the survivors
// Single-pass look-back scan with two counters per tile: keys above tau, and keys equal to tau.  An
// element above tau goes to slot  (#above before it) + min(#ties before it, q); a tie is kept iff fewer
// than q ties precede it.  VIEW == V_CAND walks the candidate list, V_DENSE the dense range itself.
template <int VIEW>
__global__ void __launch_bounds__(kThreads) compact_kernel(const __grid_constant__ DevTables T) {
  constexpr int LK = VIEW == V_CAND ? L_CAND : L_DCOMP;
  constexpr int ROUNDS = kTile / kThreads;   // 16 elements per thread
  __shared__ uint32_t s_tile;
  __shared__ uint32_t s_wg[kWarps], s_we[kWarps];
  __shared__ uint64_t s_exg, s_exe;
  __shared__ int s_ok, s_single;
  __shared__ uint32_t s_layer;
  __shared__ double s_red[kWarps][2];
  __shared__ uint32_t s_redc[kWarps][2];
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  if (tid == 0) s_tile = atomicAdd(&T.ctl->ticket[LK], 1u);
  __syncthreads();
  const uint32_t t = s_tile;
  const uint32_t* tile0 = T.tile0[LK];
  const uint32_t s = scope_of_tile(tile0, T.n_scopes, t);
  const ScopeDesc& d = T.scopes[s];
  const ScopeState* st = T.state + s;
  const bool pred = predicted_ok(T, d, *st);
  if (VIEW == V_CAND ? !pred : pred) return;      // the other view owns this scope
  const uint32_t first = __ldg(tile0 + s);
  const uint32_t lt = t - first;
  const uint64_t len = VIEW == V_CAND ? st->cand_count : d.hi - d.lo;
  const uint64_t beg = (uint64_t)lt * kTile;
  if (beg >= len) return;                         // trailing tiles of a short candidate list
  const uint64_t end = (beg + kTile < len) ? beg + kTile : len;
  const float* vals = VIEW == V_CAND ? T.cand_val + d.cand_base : T.residual + d.lo;
  const uint32_t tau = st->tau;
  const uint64_t q = st->q;
  const bool two_means = T.value_mode == GD_VALUES_TWO_MEANS;

  if (two_means && tid == 0) {
    uint64_t i_first, i_last;
    if (VIEW == V_CAND) {
      i_first = T.cand_idx[d.cand_base + beg];
      i_last = T.cand_idx[d.cand_base + end - 1];
    } else {
      i_first = d.lo + beg;
      i_last = d.lo + end - 1;
    }
    const uint32_t l0 = range_of(T.layer_off, T.n_layers, i_first);
    const uint32_t l1 = range_of(T.layer_off, T.n_layers, i_last);
    s_layer = l0;
    s_single = (l0 == l1) ? 1 : 0;
  }

  // phase 1: load, classify, count
  const uint64_t wbeg = beg + (uint64_t)warp * (32u * ROUNDS) + lane;
  uint32_t vb[ROUNDS];
  uint32_t gtm = 0, eqm = 0, wg = 0, we = 0;
#pragma unroll
  for (int j = 0; j < ROUNDS; ++j) {
    const uint64_t i = wbeg + (uint64_t)j * 32u;
    uint32_t b = 0;
    bool isgt = false, iseq = false;
    if (i < end) {
      b = __float_as_uint(vals[i]);
      const uint32_t key = b & kAbsMask;
      isgt = key > tau;
      iseq = key == tau;
    }
    vb[j] = b;
    gtm |= (isgt ? 1u : 0u) << j;
    eqm |= (iseq ? 1u : 0u) << j;
    wg += __popc(__ballot_sync(0xFFFFFFFFu, isgt));
    we += __popc(__ballot_sync(0xFFFFFFFFu, iseq));
  }
  if (lane == 0) { s_wg[warp] = wg; s_we[warp] = we; }
  __syncthreads();
  uint32_t woff_g = 0, woff_e = 0, tot_g = 0, tot_e = 0;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) {
    const uint32_t cg = s_wg[w], ce = s_we[w];
    woff_g += (w < (int)warp) ? cg : 0u;
    woff_e += (w < (int)warp) ? ce : 0u;
    tot_g += cg;
    tot_e += ce;
  }
  if (warp == 0) {
    uint64_t ex_a, ex_b;
    uint4* desc = reinterpret_cast<uint4*>(VIEW == V_CAND ? T.desc_cand : T.desc_dcomp);
    const bool ok = tile_lookback(desc, t, first, tot_g, tot_e, ex_a, ex_b, T.ctl);
    if (lane == 0) { s_exg = ex_a; s_exe = ex_b; s_ok = ok ? 1 : 0; }
  }
  __syncthreads();
  if (!s_ok) return;

  // phase 2: place the survivors
  uint64_t rg = s_exg + woff_g, re = s_exe + woff_e;   // running counts before this warp's round
  const uint32_t ltm = lanemask_lt();
  const bool single = two_means && s_single;
  const uint32_t tile_layer = two_means ? s_layer : 0u;
  double sum_p = 0.0, sum_n = 0.0;
  uint32_t cnt_p = 0, cnt_n = 0;
  bool bad = false;
#pragma unroll
  for (int j = 0; j < ROUNDS; ++j) {
    const bool isgt = (gtm >> j) & 1u, iseq = (eqm >> j) & 1u;
    const uint32_t mg = __ballot_sync(0xFFFFFFFFu, isgt), me = __ballot_sync(0xFFFFFFFFu, iseq);
    if (isgt || iseq) {
      const uint64_t gb = rg + __popc(mg & ltm), eb = re + __popc(me & ltm);
      if (isgt || eb < q) {
        const uint64_t pos = gb + (eb < q ? eb : q);
        const uint64_t i = wbeg + (uint64_t)j * 32u;
        const uint64_t idx = VIEW == V_CAND ? (uint64_t)T.cand_idx[d.cand_base + i] : d.lo + i;
        if (pos < d.k && idx < T.n) {
          const uint32_t b = vb[j];
          T.residual[idx] = 0.0f;
          if (two_means) {
            const uint32_t sgn = b >> 31;
            T.out_idx[d.out_base + pos] = (uint32_t)idx | (sgn << 31);
            const double x = (double)__uint_as_float(b);
            if (single) {
              if (sgn) { sum_n += x; ++cnt_n; } else { sum_p += x; ++cnt_p; }
            } else {
              const uint32_t l = range_of(T.layer_off, T.n_layers, idx);
              atomicAdd(T.sums + 2 * (size_t)l + sgn, x);
              atomicAdd(T.cnts + 2 * (size_t)l + sgn, 1ull);
            }
          } else {
            T.out_idx[d.out_base + pos] = (uint32_t)idx;
            T.out_val[d.out_base + pos] = __uint_as_float(b);
          }
        } else {
          bad = true;
        }
      }
    }
    rg += __popc(mg);
    re += __popc(me);
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
}

// ---------------------------------------------------------------- thresholds, shard offsets, means
__global__ void __launch_bounds__(kThreads) finalize_kernel(const __grid_constant__ DevTables T) {
  const uint32_t tid = threadIdx.x;
  const bool two_means = T.value_mode == GD_VALUES_TWO_MEANS;
  uint32_t n_pred = 0, n_dense = 0;
  unsigned long long n_cand = 0;
  for (uint32_t s = tid; s < T.n_scopes; s += kThreads) {
    const ScopeDesc& d = T.scopes[s];
    const ScopeState& st = T.state[s];
    if (T.out_tau) T.out_tau[s] = d.k == 0 ? 0xFFFFFFFFu : st.tau;
    if (st.used_dense) ++n_dense; else ++n_pred;
    n_cand += st.cand_count;
  }
  if (n_pred) atomicAdd(&T.ctl->n_scopes_predicted, n_pred);
  if (n_dense) atomicAdd(&T.ctl->n_scopes_dense, n_dense);
  if (n_cand) atomicAdd(reinterpret_cast<unsigned long long*>(&T.ctl->n_candidates), n_cand);
  if (tid == 0) { T.ctl->n_scopes = T.n_scopes; T.ctl->n_kept = T.k_total; }
  // survivors are in ascending index order: shard j starts at the first index >= shard_off[j]
  for (uint32_t j = tid; j <= T.n_shards; j += kThreads) {
    const uint64_t bound = T.shard_off[j];
    uint64_t lo = 0, hi = T.k_total;
    while (lo < hi) {
      const uint64_t mid = (lo + hi) >> 1;
      uint32_t w = T.out_idx[mid];
      if (two_means) w &= kAbsMask;
      if ((uint64_t)w < bound) lo = mid + 1; else hi = mid;
    }
    T.out_shard_cnt_off[j] = (uint32_t)lo;
  }
  if (two_means) {
    for (uint32_t e = tid; e < 2 * T.n_layers; e += kThreads) {
      const unsigned long long c = T.cnts[e];
      T.out_means[e] = c ? (float)(T.sums[e] / (double)c) : 0.0f;
    }
  }
}

// ---------------------------------------------------------------- launch sequence
#define GD_LAUNCH_CHECK()                         \
  do {                                            \
    cudaError_t e_ = cudaPeekAtLastError();       \
    if (e_ != cudaSuccess) return e_;             \
    note_launches(1);                             \
  } while (0)

cudaError_t launch_compress(const DevTables& T, const uint32_t* tiles, uint64_t samp_total, cudaStream_t stream) {
  const bool predict = !(T.flags & GD_FLAG_NO_PREDICTION);
  if (predict && samp_total) {
    const uint32_t blocks = (uint32_t)((samp_total + kThreads - 1) / kThreads);
    sample_gather_kernel<<<blocks, kThreads, 0, stream>>>(T, samp_total);
    GD_LAUNCH_CHECK();
    for (int pass = 0; pass < 3; ++pass) {
      select_pass_kernel<V_SAMPLE><<<tiles[L_SAMP], kThreads, 0, stream>>>(T, pass);
      GD_LAUNCH_CHECK();
    }
  }
  if (tiles[L_EMIT]) {
    profile_mark(stream, true);
    add_emit_kernel<<<tiles[L_EMIT], kThreads, 0, stream>>>(T);
    GD_LAUNCH_CHECK();
    profile_mark(stream, false);
  }
  if (predict && tiles[L_CAND]) {
    for (int pass = 0; pass < 3; ++pass) {
      select_pass_kernel<V_CAND><<<tiles[L_CAND], kThreads, 0, stream>>>(T, pass);
      GD_LAUNCH_CHECK();
    }
    compact_kernel<V_CAND><<<tiles[L_CAND], kThreads, 0, stream>>>(T);
    GD_LAUNCH_CHECK();
  }
  if (tiles[L_DSEL]) {
    for (int pass = 0; pass < 3; ++pass) {
      select_pass_kernel<V_DENSE><<<tiles[L_DSEL], kThreads, 0, stream>>>(T, pass);
      GD_LAUNCH_CHECK();
    }
    compact_kernel<V_DENSE><<<tiles[L_DCOMP], kThreads, 0, stream>>>(T);
    GD_LAUNCH_CHECK();
  }
  finalize_kernel<<<1, kThreads, 0, stream>>>(T);
  GD_LAUNCH_CHECK();
  return cudaSuccess;
}

}  // namespace gd
