// Device code of the survivor compaction (Algorithm 1, steps 3-5: mask, residual rewrite, sparse
// output), the two-means sums of Section 5.4, and the code that finishes a call (thresholds, shard
// offsets of Section 3, the means).  Included by the translation units that define kernels on top of
// it; internal to libgd.so.
#pragma once

#include "gd_scan.cuh"

namespace gd {

namespace {

// Finishes a call: thresholds, statistics, shard offsets (Section 3: the survivors, ascending in
// index, are cut into one piece per server) and the two means (Section 5.4).  Run by one whole CTA
// after every survivor has been written.
__device__ void finalize_call(const DevTables& T, uint64_t k_total) {
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const bool two_means = T.value_mode == GD_VALUES_TWO_MEANS || T.value_mode == GD_VALUES_COLUMN_MEANS;
  const bool packed = T.value_mode != GD_VALUES_FP32;
  uint32_t n_pred = 0, n_dense = 0;
  unsigned long long n_cand = 0;
  for (uint32_t s = tid; s < T.n_scopes; s += kThreads) {
    const ScopeDesc& d = T.scopes[s];
    const ScopeState* st = T.state + s;
    if (T.out_tau) T.out_tau[s] = d.k == 0 ? 0xFFFFFFFFu : __ldcg(&st->tau);
    if (__ldcg(&st->used_dense) || (T.flags & kFlagDenseBound)) ++n_dense; else ++n_pred;
    n_cand += __ldcg(reinterpret_cast<const unsigned long long*>(&st->cand_count));
  }
  if (n_pred) atomicAdd(&T.ctl->n_scopes_predicted, n_pred);
  if (n_dense) atomicAdd(&T.ctl->n_scopes_dense, n_dense);
  if (n_cand) atomicAdd(reinterpret_cast<unsigned long long*>(&T.ctl->n_candidates), n_cand);
  if (tid == 0) { T.ctl->n_scopes = T.n_scopes; T.ctl->n_kept = k_total; }
  // shard j starts at the first survivor with index >= shard_off[j]: a 33-way search per warp
  for (uint32_t j = warp; j <= T.n_shards; j += kWarps) {
    const uint64_t bound = T.shard_off[j];
    uint64_t lo = 0, hi = k_total;                   // answer in [lo, hi]
    if (bound == 0) hi = 0;                           // nothing lies below the first boundary ...
    if (bound >= T.n) lo = k_total;                   // ... and everything below the last: no search
    while (hi - lo > 32) {
      const uint64_t span = hi - lo;
      const uint64_t p = lo + span * (lane + 1) / 33;   // lo < p < hi, ascending in lane
      uint32_t w = __ldcg(T.out_idx + p);
      if (packed) w &= kAbsMask;
      const uint32_t c = __popc(__ballot_sync(0xFFFFFFFFu, (uint64_t)w < bound));   // probes 0..c-1 are below
      const uint64_t nlo = c ? lo + span * c / 33 + 1 : lo;
      const uint64_t nhi = c < 32 ? lo + span * (c + 1) / 33 : hi;
      lo = nlo;
      hi = nhi;
    }
    const uint64_t p = lo + lane;
    bool below = false;
    if (p < hi) {
      uint32_t w = __ldcg(T.out_idx + p);
      if (packed) w &= kAbsMask;
      below = (uint64_t)w < bound;
    }
    lo += __popc(__ballot_sync(0xFFFFFFFFu, below));
    if (lane == 0) T.out_shard_cnt_off[j] = (uint32_t)lo;
  }
  if (two_means) {
    if (T.n_pairs <= kInlineMeansPairs) {              // otherwise a kernel of its own divides the sums
      for (uint32_t e = tid; e < 2 * T.n_pairs; e += kThreads) {
        const unsigned long long c = __ldcg(T.cnts + e);
        T.out_means[e] = c ? (float)(__ldcg(T.sums + e) / (double)c) : 0.0f;
      }
    }
  } else if (T.value_mode == GD_VALUES_THRESHOLD) {
    // every survivor of layer l stands for +-t, t = the threshold of the scope that holds the layer
    for (uint32_t l = tid; l < T.n_layers; l += kThreads) {
      const uint32_t s = T.n_scopes == 1 ? 0u : l;
      const uint32_t tau = T.scopes[s].k == 0 ? 0u : __ldcg(&T.state[s].tau);
      T.out_means[2 * l] = __uint_as_float(tau);
      T.out_means[2 * l + 1] = __uint_as_float(tau | 0x80000000u);
    }
  }
}

__global__ void __launch_bounds__(kThreads) finalize_kernel(const __grid_constant__ DevTables T) { finalize_call(T, T.k_total); }

// Compaction over the candidate list: a single-pass look-back scan with two counters per tile, keys
// above tau and keys equal to tau.  An element above tau goes to slot  (#above before it) +
// min(#ties before it, q); a tie is kept iff fewer than q ties precede it.  CTAs take tiles from an
// atomic ticket until none is left; the last CTA to leave finishes the call.
__device__ __forceinline__ void compact_cand_body(const DevTables& T, uint32_t total_tiles, int do_finalize) {
  constexpr int LK = L_CAND;
  constexpr int ROUNDS = kTile / kThreads;   // 16 elements per thread
  __shared__ uint32_t s_tile;
  __shared__ uint32_t s_wg[kWarps], s_we[kWarps];
  __shared__ uint64_t s_exg, s_exe;
  __shared__ int s_ok, s_single;
  __shared__ uint32_t s_layer;
  __shared__ double s_red[kWarps][2];
  __shared__ uint32_t s_redc[kWarps][2];
  __shared__ int s_last;
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  __shared__ SmemTables s_tab;
  const ScopeDesc* scopes;
  const uint32_t* tile0;
  load_tables(T, LK, &s_tab, &scopes, &tile0);
  const bool two_means = T.value_mode == GD_VALUES_TWO_MEANS || T.value_mode == GD_VALUES_COLUMN_MEANS;   // sums are kept
  const bool packed = T.value_mode != GD_VALUES_FP32;
  const bool feedback = (T.flags & GD_FLAG_QUANT_ERROR_FEEDBACK) != 0;   // kept slots keep v for feedback_kernel
  const bool early = early_zero_enabled(T);
  const uint32_t ltm = lanemask_lt();
  uint4* desc = reinterpret_cast<uint4*>(T.desc_cand);
  // The lists' capacities are a multiple of what they hold.  With few scopes only the tiles that hold
  // candidates are numbered (in list order), so that no ticket is spent on an empty tile.
  __shared__ uint32_t s_vt0[kVtScopes + 1];
  const bool compacted = T.n_scopes <= kVtScopes;
  if (compacted) {
    __syncthreads();                       // the table copy is complete
    for (uint32_t x = tid; x < T.n_scopes; x += kThreads) {
      const ScopeState* sx = T.state + x;
      s_vt0[x + 1] = predicted_ok(T, scopes[x], *sx) ? (uint32_t)((sx->cand_count + kTile - 1) / kTile) : 0u;
    }
    if (tid == 0) s_vt0[0] = 0;
    __syncthreads();
    block_inclusive_scan(s_vt0 + 1, T.n_scopes);
    total_tiles = s_vt0[T.n_scopes];
  }

  for (;;) {
    __syncthreads();                       // previous tile is done with the shared variables
    if (tid == 0) s_tile = atomicAdd(&T.ctl->ticket[LK], 1u);
    __syncthreads();
    const uint32_t t = s_tile;
    if (t >= total_tiles) break;
    uint32_t s, first;
    if (compacted) {
      s = scope_of_tile(s_vt0, T.n_scopes, t);   // a binary search in shared memory
      first = s_vt0[s];
    } else {
      s = scope_of_tile(tile0, T.n_scopes, t);
      first = tile0[s];
    }
    const ScopeDesc& d = scopes[s];
    const ScopeState* st = T.state + s;
    if (!predicted_ok(T, d, *st)) continue;         // the dense kernels own this scope
    const uint32_t lt = t - first;
    const uint64_t len = st->cand_count;
    const uint64_t beg = (uint64_t)lt * kTile;
    if (beg >= len) continue;                       // trailing tiles of a short candidate list
    const uint64_t end = (beg + kTile < len) ? beg + kTile : len;
    const float* vals = T.cand_val + d.cand_base;
    const uint32_t tau = __ldcg(&st->tau);     // from L2: the selection may have run in this same launch
    const uint64_t q = __ldcg(&st->q);
    // Entries with key > zthr had +0 written over their residual slot by the fused pass.  Kept ones
    // need no store then (unless some entry of the scope could not be treated so: early_bad); the few
    // that are not kept after all get v back.
    const uint32_t zthr = early ? st->tau_hi : 0xFFFFFFFFu;
    const bool skip_cleared = early && st->early_bad == 0u;

    if (two_means && tid == 0) {
      const uint64_t i_first = T.cand_idx[d.cand_base + beg];
      const uint64_t i_last = T.cand_idx[d.cand_base + end - 1];
      const uint32_t l0 = range_of(T.layer_off, T.n_layers, i_first);
      const uint32_t l1 = range_of(T.layer_off, T.n_layers, i_last);
      s_layer = (uint32_t)T.pair_off[l0];              // the one pair of the tile, if it has only one
      s_single = (l0 == l1 && T.layer_cols[l0] == 1u) ? 1 : 0;
    }

    // phase 1: load, classify, count.  Offsets inside the tile are 32-bit; a whole tile skips the bounds checks.
    const uint32_t wofs = warp * (32u * ROUNDS) + lane;          // this thread's first element inside the tile
    const uint32_t valid = (uint32_t)(end - beg);                // elements of this tile
    const bool whole = valid == kTile;
    const uint32_t* tile_idx = T.cand_idx + d.cand_base + beg;
    const float* tile_val = vals + beg;
    uint32_t vb[ROUNDS], ib[ROUNDS];
    uint32_t gtm = 0, eqm = 0, wg = 0, we = 0;
#pragma unroll
    for (int j = 0; j < ROUNDS; ++j) {   // the candidates' indices travel with their values: loaded up front
      const uint32_t o = wofs + (uint32_t)j * 32u;
      ib[j] = (whole || o < valid) ? tile_idx[o] : 0u;
    }
#pragma unroll
    for (int j = 0; j < ROUNDS; ++j) vb[j] = 0u;
#pragma unroll
    for (int j = 0; j < ROUNDS; ++j) {
      const uint32_t o = wofs + (uint32_t)j * 32u;
      if (whole || o < valid) vb[j] = __float_as_uint(tile_val[o]);
    }
#pragma unroll
    for (int j = 0; j < ROUNDS; ++j) {
      const uint32_t o = wofs + (uint32_t)j * 32u;
      const uint32_t b = vb[j];
      bool isgt = false, iseq = false;
      if (whole || o < valid) {
        const uint32_t key = b & kAbsMask;
        isgt = key > tau;
        iseq = key == tau;
      }
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
      const bool ok = tile_lookback(desc, t, first, tot_g, tot_e, ex_a, ex_b, T.ctl);
      if (lane == 0) { s_exg = ex_a; s_exe = ex_b; s_ok = ok ? 1 : 0; }
    }
    __syncthreads();
    if (!s_ok) continue;

    // phase 2: place the survivors.  Slot of an entry = (#above before it) + min(#ties before it, q); with
    // EXG / EXE the counts before this tile that is
    //   out_base + EXG + min(EXE, q)  +  (above before it in the tile) + min(ties before it in the tile, q - EXE),
    // one 64-bit base per tile and 32-bit arithmetic per entry.
    const uint64_t exg = s_exg, exe = s_exe;
    const uint64_t tie_base = exe < q ? exe : q;
    const uint64_t q_left64 = q - tie_base;               // ties of this tile that are still kept
    const uint32_t q_left = q_left64 < 0xFFFFu ? (uint32_t)q_left64 : 0xFFFFu;   // a tile has at most 4096 entries
    const uint64_t slot0 = exg + tie_base;                // slot, inside the scope, of the tile's first survivor
    const uint64_t room = d.k > slot0 ? d.k - slot0 : 0;  // slots left in the scope from there
    uint32_t* const oi = T.out_idx + d.out_base + slot0;
    float* const ov = T.out_val ? T.out_val + d.out_base + slot0 : nullptr;
    uint32_t rg = woff_g, re = woff_e;                    // counts inside the tile before this warp's round
    const bool single = two_means && s_single;
    const uint32_t tile_layer = two_means ? s_layer : 0u;
    double sum_p = 0.0, sum_n = 0.0;
    uint32_t cnt_p = 0, cnt_n = 0;
    bool bad = false;
#pragma unroll
    for (int j = 0; j < ROUNDS; ++j) {
      const bool isgt = (gtm >> j) & 1u, iseq = (eqm >> j) & 1u;
      const uint32_t mg = __ballot_sync(0xFFFFFFFFu, isgt), me = __ballot_sync(0xFFFFFFFFu, iseq);
      bool kept = false;
      if (isgt || iseq) {
        const uint32_t gb = rg + __popc(mg & ltm), eb = re + __popc(me & ltm);
        if (isgt || eb < q_left) {
          kept = true;
          const uint32_t pos = gb + (eb < q_left ? eb : q_left);
          const uint64_t idx = ib[j];
          if (pos < room && idx < T.n) {
            const uint32_t b = vb[j];
            if (!feedback && !(skip_cleared && (b & kAbsMask) > zthr)) T.residual[idx] = 0.0f;
            if (packed) {
              const uint32_t sgn = b >> 31;
              oi[pos] = (uint32_t)idx | (sgn << 31);
              const double x = (double)__uint_as_float(b);
              if (!two_means) {
                // threshold mode: the value is implied by the scope's tau
              } else if (single) {
                if (sgn) { sum_n += x; ++cnt_n; } else { sum_p += x; ++cnt_p; }
              } else {
                const uint64_t pr = pair_of(T.layer_off, T.pair_off, T.layer_cols, T.n_layers, idx);
                atomicAdd(T.sums + 2 * pr + sgn, x);
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
        }
      }
      // cleared early but not kept after all (the estimate was below tau, or a tie beyond the quota)
      if (!kept && (vb[j] & kAbsMask) > zthr && (whole || wofs + (uint32_t)j * 32u < valid) && ib[j] < T.n)
        T.residual[ib[j]] = __uint_as_float(vb[j]);
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
  if (!do_finalize) return;
  // the last CTA to leave finishes the call
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(&T.ctl->compact_done[0], 1u) == gridDim.x - 1u) ? 1 : 0;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  finalize_call(T, T.k_total);
}

// The larger shared arrays of the dense compaction: the kernel that runs it declares them, the kernel that only
// takes it over on rare occasions lends it memory it has another use for otherwise.
struct CompactDenseSmem {
  uint32_t cg[kDenseChunkTilesMax * kWarps], ce[kDenseChunkTilesMax * kWarps];   // per (tile, warp): keys above / equal
  uint32_t og[kDenseChunkTilesMax * kWarps], oe[kDenseChunkTilesMax * kWarps];   // their exclusive offsets in the chunk
  double red[kWarps][2];
  uint32_t redc[kWarps][2];
  SmemTables tab;
  uint32_t mask[kDenseChunkTilesMax][kThreads];   // per tile and thread; low 16 bits: key > tau, high 16: key == tau
};

// Compaction over the dense range itself, for scopes whose prediction failed.  Same placement rule
// as above, but one ticket covers a chunk of up to 16 tiles (256 KiB of values on long vectors) and the chunk does
// one look-back: at 4 bytes per element the chain of look-backs would otherwise have to advance about a
// hundred tiles per microsecond, which the L2 round trips between CTAs cannot sustain.
// The classification masks stay in registers; the values of the (few) survivors are read again.
__device__ __forceinline__ void compact_dense_body(const DevTables& T, uint32_t total_chunks, int do_finalize,
                                                   CompactDenseSmem& S) {
  constexpr int CD = (int)kDenseChunkTilesMax;   // shared arrays are sized for the largest chunk
  const int cd = (int)T.dense_chunk_tiles;        // tiles per chunk in this call
  constexpr int ROUNDS = kTile / kThreads;   // 16 elements per thread and tile
  constexpr int E = CD * kWarps;             // (tile, warp) counters of one chunk: 32
  __shared__ uint32_t s_chunk;
  __shared__ uint64_t s_exg, s_exe;
  __shared__ int s_ok, s_single, s_last;
  __shared__ uint32_t s_layer;
  uint32_t* const s_cg = S.cg;
  uint32_t* const s_ce = S.ce;
  uint32_t* const s_og = S.og;
  uint32_t* const s_oe = S.oe;
  double (*const s_red)[2] = S.red;
  uint32_t (*const s_redc)[2] = S.redc;
  SmemTables& s_tab = S.tab;
  uint32_t (*const s_mask)[kThreads] = S.mask;
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  if (!(T.flags & GD_FLAG_NO_PREDICTION) && T.ctl->dense_needed == 0u) return;
  const ScopeDesc* scopes;
  const uint32_t* tile0;
  load_tables(T, L_DCOMP, &s_tab, &scopes, &tile0);
  const bool two_means = T.value_mode == GD_VALUES_TWO_MEANS || T.value_mode == GD_VALUES_COLUMN_MEANS;   // sums are kept
  const bool packed = T.value_mode != GD_VALUES_FP32;
  const bool feedback = (T.flags & GD_FLAG_QUANT_ERROR_FEEDBACK) != 0;   // kept slots keep v for feedback_kernel
  const uint32_t ltm = lanemask_lt();
  uint4* desc = reinterpret_cast<uint4*>(T.desc_dcomp);

  for (;;) {
    __syncthreads();                       // previous chunk is done with the shared variables
    if (tid == 0) s_chunk = atomicAdd(&T.ctl->ticket[L_DCOMP], 1u);
    __syncthreads();
    const uint32_t t = s_chunk;
    if (t >= total_chunks) break;
    const uint32_t s = scope_of_tile(tile0, T.n_scopes, t);
    const ScopeDesc& d = scopes[s];
    const ScopeState* st = T.state + s;
    if (predicted_ok(T, d, *st)) continue;          // the candidate list owns this scope
    const uint32_t first = tile0[s];
    const uint32_t lt = t - first;
    const uint64_t len = d.hi - d.lo;
    const uint64_t span = (uint64_t)cd * kTile;
    const uint64_t beg = (uint64_t)lt * span;
    const uint64_t end = (beg + span < len) ? beg + span : len;
    const float* vals = T.residual + d.lo;
    const uint32_t tau = __ldcg(&st->tau);     // from L2: the selection may have run in this same launch
    const uint64_t q = __ldcg(&st->q);
    if (two_means && tid == 0) {
      const uint32_t l0 = range_of(T.layer_off, T.n_layers, d.lo + beg);
      const uint32_t l1 = range_of(T.layer_off, T.n_layers, d.lo + end - 1);
      s_layer = (uint32_t)T.pair_off[l0];              // the one pair of the chunk, if it has only one
      s_single = (l0 == l1 && T.layer_cols[l0] == 1u) ? 1 : 0;
    }

    // phase 1: classify every element of the chunk, count per (tile, warp)
#pragma unroll 2
    for (int c = 0; c < CD; ++c) {
      if (c >= cd || beg + (uint64_t)c * kTile >= end) {   // past the chunk, or the scope ends inside it (uniform)
        s_mask[c][tid] = 0;
        if (lane == 0) { s_cg[c * kWarps + warp] = 0; s_ce[c * kWarps + warp] = 0; }
        continue;
      }
      const uint64_t wbeg = beg + (uint64_t)c * kTile + (uint64_t)warp * (32u * ROUNDS) + lane;
      uint32_t vb[ROUNDS];
#pragma unroll
      for (int j = 0; j < ROUNDS; ++j) {
        const uint64_t i = wbeg + (uint64_t)j * 32u;
        vb[j] = i < end ? __float_as_uint(vals[i]) : 0xFFFFFFFFu;
      }
      uint32_t m = 0, wg = 0, we = 0;
#pragma unroll
      for (int j = 0; j < ROUNDS; ++j) {
        const uint64_t i = wbeg + (uint64_t)j * 32u;
        const uint32_t key = vb[j] & kAbsMask;
        const bool isgt = i < end && key > tau, iseq = i < end && key == tau;
        m |= (isgt ? 1u : 0u) << j;
        m |= (iseq ? 1u : 0u) << (16 + j);
        wg += __popc(__ballot_sync(0xFFFFFFFFu, isgt));
        we += __popc(__ballot_sync(0xFFFFFFFFu, iseq));
      }
      s_mask[c][tid] = m;
      if (lane == 0) { s_cg[c * kWarps + warp] = wg; s_ce[c * kWarps + warp] = we; }
    }
    __syncthreads();
    if (warp == 0) {                                // E counter pairs, PER consecutive ones per lane
      constexpr int PER = E / 32;
      uint32_t ag[PER], ae[PER], sg = 0, se = 0;
#pragma unroll
      for (int p = 0; p < PER; ++p) {
        ag[p] = s_cg[lane * PER + p];
        ae[p] = s_ce[lane * PER + p];
        sg += ag[p];
        se += ae[p];
      }
      uint32_t ig = sg, ie = se;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t yg = __shfl_up_sync(0xFFFFFFFFu, ig, o), ye = __shfl_up_sync(0xFFFFFFFFu, ie, o);
        if ((int)lane >= o) { ig += yg; ie += ye; }
      }
      uint32_t rg0 = ig - sg, re0 = ie - se;
#pragma unroll
      for (int p = 0; p < PER; ++p) {
        s_og[lane * PER + p] = rg0;
        s_oe[lane * PER + p] = re0;
        rg0 += ag[p];
        re0 += ae[p];
      }
      const uint32_t tot_g = __shfl_sync(0xFFFFFFFFu, ig, 31), tot_e = __shfl_sync(0xFFFFFFFFu, ie, 31);
      uint64_t ex_a, ex_b;
      const bool ok = tile_lookback(desc, t, first, tot_g, tot_e, ex_a, ex_b, T.ctl);
      if (lane == 0) { s_exg = ex_a; s_exe = ex_b; s_ok = ok ? 1 : 0; }
    }
    __syncthreads();
    if (!s_ok) continue;

    // phase 2: place the survivors
    const bool single = two_means && s_single;
    const uint32_t tile_layer = two_means ? s_layer : 0u;
    double sum_p = 0.0, sum_n = 0.0;
    uint32_t cnt_p = 0, cnt_n = 0;
    bool bad = false;
#pragma unroll 1
    for (int c = 0; c < cd; ++c) {
      const uint32_t m = s_mask[c][tid];
      if (!__any_sync(0xFFFFFFFFu, m != 0u)) continue;
      const uint64_t wbeg = beg + (uint64_t)c * kTile + (uint64_t)warp * (32u * ROUNDS) + lane;
      uint64_t rg = s_exg + s_og[c * kWarps + warp], re = s_exe + s_oe[c * kWarps + warp];
#pragma unroll
      for (int j = 0; j < ROUNDS; ++j) {
        const bool isgt = (m >> j) & 1u, iseq = (m >> (16 + j)) & 1u;
        const uint32_t mg = __ballot_sync(0xFFFFFFFFu, isgt), me = __ballot_sync(0xFFFFFFFFu, iseq);
        if (isgt || iseq) {
          const uint64_t gb = rg + __popc(mg & ltm), eb = re + __popc(me & ltm);
          if (isgt || eb < q) {
            const uint64_t pos = gb + (eb < q ? eb : q);
            const uint64_t i = wbeg + (uint64_t)j * 32u;
            const uint64_t idx = d.lo + i;
            if (pos < d.k && idx < T.n) {
              const uint32_t b = __float_as_uint(vals[i]);   // read again: only survivors get here
              if (!feedback) T.residual[idx] = 0.0f;
              if (packed) {
                const uint32_t sgn = b >> 31;
                T.out_idx[d.out_base + pos] = (uint32_t)idx | (sgn << 31);
                const double x = (double)__uint_as_float(b);
                if (!two_means) {
                  // threshold mode: the value is implied by the scope's tau
                } else if (single) {
                  if (sgn) { sum_n += x; ++cnt_n; } else { sum_p += x; ++cnt_p; }
                } else {
                  const uint64_t pr = pair_of(T.layer_off, T.pair_off, T.layer_cols, T.n_layers, idx);
                  atomicAdd(T.sums + 2 * pr + sgn, x);
                  atomicAdd(T.cnts + 2 * pr + sgn, 1ull);
                }
              } else {
                T.out_idx[d.out_base + pos] = (uint32_t)idx;
                T.out_val[d.out_base + pos] = __uint_as_float(b);
                if (T.delta_base) T.delta_base[idx] = __fadd_rn(T.delta_base[idx], __uint_as_float(b));
              }
            } else {
              bad = true;
            }
          }
        }
        rg += __popc(mg);
        re += __popc(me);
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
  }
  if (!do_finalize) return;
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(&T.ctl->compact_done[1], 1u) == gridDim.x - 1u) ? 1 : 0;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  finalize_call(T, T.k_total);
}

// (kept out of line so that the rare path does not weigh on the registers of the usual one)
__device__ __noinline__ void compact_dense_outlined(const DevTables& T, uint32_t dense_chunks, CompactDenseSmem& S) {
  compact_dense_body(T, dense_chunks, 0, S);
}

}  // namespace

}  // namespace gd
