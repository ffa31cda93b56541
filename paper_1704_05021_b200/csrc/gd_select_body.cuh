// Device code of the threshold selection (Algorithm 1, the threshold-selection step): an exact radix
// select on the bit pattern of |v| over the sample, the candidate lists or the dense range, plus the
// grid barrier and histogram walks it is built from.  Included by the translation units that define
// kernels on top of it; internal to libgd.so.
#pragma once

#include "gd_internal.cuh"

namespace gd {

namespace {

__device__ __forceinline__ uint32_t mix32(uint32_t x) {
  x ^= x >> 16; x *= 0x7FEB352Du; x ^= x >> 15; x *= 0x846CA68Bu; x ^= x >> 16;
  return x;
}


// All CTAs of a cooperative launch meet here.  `phase` counts the barriers this CTA has passed.
// Returns false (after recording GD_ERR_DEVICE_TIMEOUT) if the others did not arrive in time.
__device__ bool grid_barrier(uint32_t* counter, uint32_t& phase, Ctl* ctl) {
  __shared__ int s_pass;
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint32_t target = (++phase) * gridDim.x;
    __threadfence();
    atomicAdd(counter, 1u);
    uint32_t spins = 0;
    int ok = 1;
    const uint64_t t0 = global_timer_ns();
    while (ld_acquire_u32(counter) < target) {
      if (wait_expired(++spins, kLookbackSpinLimit, t0, kWaitBudgetNs)) { ok = 0; break; }
      if (spins > 4) __nanosleep(40);
    }
    if (!ok) atomicCAS(&ctl->status, (int)GD_OK, (int)GD_ERR_DEVICE_TIMEOUT);
    s_pass = ok;
  } else {
    ++phase;
  }
  __syncthreads();
  return s_pass != 0;
}

// The value of sample li of scope s: the scope is cut into m strata and one position inside stratum li
// is read.  The sample only steers the prediction; any sample gives the same final result.
__device__ __forceinline__ float sample_value(const DevTables& T, const ScopeDesc& d, uint32_t s, uint64_t li) {
  // m strata: the first (n_s mod m) have floor(n_s / m) + 1 elements, the others floor(n_s / m).
  // Where the strata are narrow, a sample per stratum would touch nearly every 32-byte sector of the
  // scope; there the strata are made of groups of 8 elements and a whole group is sampled (samples
  // 8c .. 8c+7 are group c), which reads an eighth of the sectors for the same number of samples.
  // Wide strata are sampled in pairs of neighbours (samp_cluster = 2): half the scattered reads, and the
  // sample still spreads over as many rows of a matrix as a pair allows.
  const uint32_t cl = d.samp_cluster;                          // 1, 2 or 8 elements per group
  const uint32_t sh = cl == 8u ? 3u : (cl == 2u ? 1u : 0u);
  const uint64_t u = li >> sh;                                 // stratum
  const uint64_t a = u * d.samp_w + (u < d.samp_rem ? u : d.samp_rem);
  const uint32_t width = (uint32_t)d.samp_w + (u < d.samp_rem ? 1u : 0u);
  uint64_t unit = a;
  if (width > 1) unit += mix32((uint32_t)u * 0x9E3779B9u + s) % width;
  const uint64_t pos = ((d.lo + cl - 1u) & ~(uint64_t)(cl - 1u)) + (unit << sh) + (li & (cl - 1u));
  return T.delta_base ? __fsub_rn(__ldg(T.grad + pos), T.delta_base[pos]) : __fadd_rn(__ldg(T.grad + pos), T.residual[pos]);
}

template <int VIEW>
__device__ __forceinline__ bool view_active(const DevTables& T, const ScopeDesc& d, const ScopeState* st) {
  if (VIEW == V_SAMPLE) return d.samp_m != 0;
  const bool pred = predicted_ok(T, d, *st);
  return VIEW == V_CAND ? pred : !pred;
}

// Running state of a radix selection: the digits fixed so far, the rank still to find inside that
// bucket, and the number of keys above the bucket.
struct SelRun {
  uint32_t prefix;
  uint64_t rank, gt;
};

// Histograms of one scope: up to three passes over the sample, then the three passes of the candidate
// (or dense) selection.  Each is filled once per call and never cleared inside a call.
__device__ __forceinline__ unsigned long long* hist_of(const DevTables& T, uint32_t s, int view, int pass) {
  unsigned long long* base = T.hist + (size_t)s * kHistBinsPerScope;
  const uint32_t off = pass == 0 ? 0u : (pass == 1 ? 2048u : 3072u);   // 2048 + 1024 + 1024 bins
  return base + (view == V_SAMPLE ? 0u : 4096u) + off;
}

__device__ __forceinline__ unsigned long long load_bin(const unsigned long long* p) { return __ldcg(p); }
__device__ __forceinline__ unsigned long long load_bin(const uint32_t* p) { return *p; }

// Run by a whole CTA on a finished histogram `gh` (a global one after the grid barrier that completes
// it, or the CTA's own in shared memory): walks it from the top bin down and fixes the next digit.
// Every CTA that needs the digit computes it for itself, so no second barrier is needed to hand it around.
// The same for two ranks at once (one pass over the bins): io[0] and io[1] are replaced by their successors.
template <typename Bin>
__device__ void next_digit_pair(const Bin* gh, int bits, SelRun* io, int count, Ctl* ctl) {
  __shared__ unsigned long long s_warp[kWarps];
  __shared__ unsigned long long s_acc[2];
  __shared__ uint32_t s_digit[2];
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const uint32_t nbins = 1u << bits;
  const uint32_t C = nbins / kThreads;                 // 8 or 4 bins per thread: [top - C + 1, top]
  const uint32_t top = nbins - 1u - tid * C;
  unsigned long long bin[8];
  unsigned long long cs = 0;
#pragma unroll
  for (uint32_t j = 0; j < 8; ++j) {
    bin[j] = j < C ? load_bin(gh + top - j) : 0ull;
    cs += bin[j];
  }
  unsigned long long inc = cs;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
    if ((int)lane >= o) inc += y;
  }
  __syncthreads();                                     // the shared scratch is free again
  if (lane == 31) s_warp[warp] = inc;
  __syncthreads();
  unsigned long long above = inc - cs;
  for (uint32_t w = 0; w < warp; ++w) above += s_warp[w];
  for (int r = 0; r < count; ++r) {
    const SelRun in = io[r];
    if (tid == kThreads - 1 && above + cs < in.rank) atomicCAS(&ctl->status, (int)GD_OK, (int)GD_ERR_INTERNAL);
    const bool owner = in.rank == 0 ? (tid == 0) : (above < in.rank && in.rank <= above + cs);
    if (owner) {
      uint32_t digit = nbins - 1u;
      unsigned long long acc = 0;
      if (in.rank != 0) {
        acc = above;
#pragma unroll
        for (uint32_t j = 0; j < 8; ++j) {
          if (j < C) {
            if (acc + bin[j] >= in.rank) { digit = top - j; break; }
            acc += bin[j];
          }
        }
      }
      s_digit[r] = digit;
      s_acc[r] = acc;
    }
  }
  __syncthreads();
  for (int r = 0; r < count; ++r) {
    SelRun out;
    out.prefix = (io[r].prefix << bits) | s_digit[r];
    out.rank = io[r].rank - s_acc[r];
    out.gt = io[r].gt + s_acc[r];
    io[r] = out;
  }
}

template <typename Bin>
__device__ SelRun next_digit(const Bin* gh, int bits, SelRun in, Ctl* ctl) {
  next_digit_pair(gh, bits, &in, 1, ctl);
  return in;
}

// Rank, in a scope's sample, of the best estimate of the threshold itself: the expected number of
// samples above it (the prediction tau_lo uses a larger rank, i.e. a lower key, for its margin).
__device__ __forceinline__ uint64_t rank_hi_of(const ScopeDesc& d) {
  const uint64_t ns = d.hi - d.lo;
  uint64_t r = ns ? (d.k * d.samp_m + ns / 2) / ns : 0;     // k <= 2^32, samp_m <= 2^22: no overflow
  if (r < 1) r = 1;
  if (r > d.samp_m) r = d.samp_m;
  return r;
}

// One key into the CTA's shared histogram.  A warp whose 32 keys share one bin (all zeros in a
// row-sparse layer, or nothing to count) issues one add; otherwise plain shared-memory adds.  Measured
// on skewed keys, this beats grouping equal digits with match.any, whose cost is paid on every round.
__device__ __forceinline__ void count_digit(uint32_t* sh, uint32_t digit, uint32_t lane) {
  constexpr uint32_t NONE = 0xFFFFFFFFu;
  const uint32_t d0 = __shfl_sync(0xFFFFFFFFu, digit, 0);
  if (__all_sync(0xFFFFFFFFu, digit == d0)) {
    if (lane == 0 && d0 != NONE) atomicAdd(&sh[d0], 32u);
  } else if (digit != NONE) {
    atomicAdd(&sh[digit], 1u);
  }
}

// The whole selection of a list of at most kTile entries, by one CTA in its shared histogram `sh`
// (all zero on entry and on return): no global histogram, no grid barrier.  The entries are read again
// in every pass (they sit in L2) so that the caller's registers stay free.
template <int VIEW>
__device__ __noinline__ SelRun local_select(const DevTables& T, const ScopeDesc& d, uint32_t s, uint32_t len,
                                            const float* vals, int passes, uint32_t* sh, uint64_t rank, bool gather) {
  constexpr uint32_t NONE = 0xFFFFFFFFu;
  const uint32_t tid = threadIdx.x, lane = tid & 31u;
  SelRun run;
  run.prefix = 0;
  run.rank = rank;
  run.gt = 0;
  for (int p = 0; p < passes; ++p) {
    const int shift = p == 0 ? kShift0 : (p == 1 ? kShift1 : kShift2);
    const int bits = p == 0 ? kRadixBits0 : 10;
    const int pshift = p == 1 ? kShift0 : kShift1;
    uint32_t keys[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const uint32_t i = (uint32_t)j * kThreads + tid;
      float x = 0.f;
      if (i < len) x = (VIEW == V_SAMPLE && p == 0 && gather) ? sample_value(T, d, s, i) : vals[i];
      keys[j] = __float_as_uint(x);
    }
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const uint32_t i = (uint32_t)j * kThreads + tid;
      uint32_t digit = NONE;
      if (i < len) {
        if (VIEW == V_SAMPLE && p == 0 && gather) T.samp_val[d.samp_base + i] = __uint_as_float(keys[j]);   // read back by this thread
        const uint32_t key = keys[j] & kAbsMask;
        if (p == 0 || (key >> pshift) == run.prefix) digit = (key >> shift) & ((1u << bits) - 1u);
      }
      count_digit(sh, digit, lane);
    }
    __syncthreads();
    run = next_digit(sh, bits, run, T.ctl);
    for (uint32_t b = tid; b < (1u << bits); b += kThreads) sh[b] = 0;
    __syncthreads();
  }
  return run;
}

// MANY = false: at most kSmemScopes scopes, all tables in shared memory, every list goes through the
// global histograms (with few scopes a CTA rarely holds tiles of more than one, and the per-scope
// steps run side by side in different CTAs).  MANY = true (models with hundreds of tensors): a CTA's
// run of tiles crosses several scopes, so it keeps a window of the tables from its first scope on, and
// selects every list of a single tile by itself in shared memory.
// The shared memory of one selection: the kernels that run one declare it, the kernel that only takes the dense
// selection over on rare occasions lends it memory it has another use for otherwise.
template <int VIEW, bool MANY>
struct SelectSmem {
  uint32_t sh[kRadixBins0];
  SmemTables tab;                              // the scopes [w0, w0 + kSmemScopes) this CTA starts in
  SelRun runs[kSmemScopes][2];                 // where the walks of those scopes stand ...
  int level[kSmemScopes];                      // ... and after how many histograms (0: not started)
  uint32_t vt0[VIEW == V_CAND ? (MANY ? kVtScopes : kSmemScopes) + 1 : 1];
};

template <int VIEW, bool MANY>
__device__ __forceinline__ void select_body(const DevTables& T, uint32_t total_tiles, SelectSmem<VIEW, MANY>& S) {
  constexpr int LK = VIEW == V_SAMPLE ? L_SAMP : (VIEW == V_CAND ? L_CAND : L_DSEL);
  const uint32_t TILE = VIEW == V_DENSE ? T.dense_sel_tile : (VIEW == V_SAMPLE ? T.samp_tile : kTile);
  const int PASSES = VIEW == V_SAMPLE ? (int)T.sample_passes : 3;   // the prediction needs 21 bits only
  constexpr uint32_t NONE = 0xFFFFFFFFu;
  uint32_t* const sh = S.sh;
  SmemTables& s_tab = S.tab;
  SelRun (*const s_runs)[2] = S.runs;
  int* const s_level = S.level;
  uint32_t* const s_vt0 = S.vt0;
  const uint32_t tid = threadIdx.x, lane = tid & 31u;
  if (T.ctl->status != GD_OK) return;   // set only by an earlier kernel of this call: uniform over the grid
  if (VIEW == V_DENSE && !(T.flags & GD_FLAG_NO_PREDICTION) && T.ctl->dense_needed == 0u) return;
  // Several candidate lists: their capacities are a multiple of what they hold, so only the tiles that
  // hold candidates are numbered (in list order); every CTA works the numbering out for itself.
  const bool compacted = VIEW == V_CAND && T.n_scopes > 1u && T.n_scopes <= (MANY ? kVtScopes : kSmemScopes);
  const uint32_t* base = T.tile0[LK];                   // base[s] = tiles before scope s
  if (compacted) {
    for (uint32_t x = tid; x < T.n_scopes; x += kThreads) {
      const ScopeState* sx = T.state + x;
      s_vt0[x + 1] = predicted_ok(T, T.scopes[x], *sx) ? (uint32_t)((sx->cand_count + kTile - 1) / kTile) : 0u;
    }
    if (tid == 0) s_vt0[0] = 0;
    __syncthreads();
    block_inclusive_scan(s_vt0 + 1, T.n_scopes);
    total_tiles = s_vt0[T.n_scopes];
    base = s_vt0;
  }
  // Each CTA takes a contiguous run of tiles (one flush of its histogram, and one pass over the finished
  // histograms, per scope it touches), except for a single list: its tiles beyond its length (the capacity
  // is a multiple of what it holds) are empty, and dealing the tiles out round-robin spreads the real ones
  // over all CTAs.  (With several scopes, round-robin and block-cyclic splits were measured and lose more
  // to the extra scope changes than they gain in balance.)
  const bool round_robin = VIEW != V_DENSE && T.n_scopes == 1u;
  const uint32_t per = (total_tiles + gridDim.x - 1) / gridDim.x;
  const uint32_t t_beg = round_robin ? blockIdx.x : blockIdx.x * per;
  const uint32_t t_end = round_robin ? total_tiles : ((t_beg + per < total_tiles) ? t_beg + per : total_tiles);
  const uint32_t t_step = round_robin ? gridDim.x : 1u;
  // The scope the run starts in, and a copy of the tables of the scopes from there on: with few
  // scopes per CTA (the usual case) every later lookup is a shared-memory read.
  uint32_t w0 = 0;
  if (MANY && t_beg < t_end) w0 = block_count_le(base, T.n_scopes, t_beg) - 1u;   // else all scopes fit
  {
    const uint32_t cnt = T.n_scopes - w0 < kSmemScopes ? T.n_scopes - w0 : kSmemScopes;
    const uint32_t words = cnt * (uint32_t)(sizeof(ScopeDesc) / 8);
    const uint64_t* src = reinterpret_cast<const uint64_t*>(T.scopes + w0);
    uint64_t* dst = reinterpret_cast<uint64_t*>(s_tab.scopes);
    for (uint32_t i = tid; i < words; i += kThreads) dst[i] = src[i];
    for (uint32_t i = tid; i <= cnt; i += kThreads) s_tab.tile0[i] = base[w0 + i];
    for (uint32_t i = tid; i < kSmemScopes; i += kThreads) s_level[i] = 0;
    __syncthreads();
  }
  auto desc_of = [&](uint32_t s) -> const ScopeDesc& {
    return (!MANY || s - w0 < kSmemScopes) ? s_tab.scopes[s - w0] : T.scopes[s];
  };
  auto base_of = [&](uint32_t s) -> uint32_t { return (!MANY || s - w0 <= kSmemScopes) ? s_tab.tile0[s - w0] : base[s]; };
  uint32_t phase = 0;

  if (VIEW == V_DENSE && early_zero_enabled(T)) {
    // Scopes that fall back to the dense range: the fused pass wrote +0 over the entries it expected
    // to be kept; all of them are in the scope's candidate list, from which v is put back before
    // anything reads the range.  (Entries that did not fit the list were put back by the fused pass.)
    const uint64_t gtid = (uint64_t)blockIdx.x * kThreads + tid, gsize = (uint64_t)gridDim.x * kThreads;
    for (uint32_t x = 0; x < T.n_scopes; ++x) {
      const ScopeDesc& dx = T.scopes[x];
      const ScopeState* sx = T.state + x;
      if (dx.samp_m == 0 || predicted_ok(T, dx, *sx)) continue;
      const uint64_t mm = sx->cand_count < dx.cand_cap ? sx->cand_count : dx.cand_cap;
      const uint32_t zthr = sx->tau_hi;
      for (uint64_t i = gtid; i < mm; i += gsize) {
        const float v = T.cand_val[dx.cand_base + i];
        if ((__float_as_uint(v) & kAbsMask) > zthr) T.residual[T.cand_idx[dx.cand_base + i]] = v;
      }
    }
    if (!grid_barrier(&T.ctl->barrier[VIEW], phase, T.ctl)) return;
  }

  for (int pass = 0; pass <= PASSES; ++pass) {
    const int shift = pass == 0 ? kShift0 : (pass == 1 ? kShift1 : kShift2);
    const int bits = pass == 0 ? kRadixBits0 : 10;
    const uint32_t nbins = 1u << bits;
    const int pshift = pass == 1 ? kShift0 : kShift1;   // shift that exposes the digits fixed so far

    for (uint32_t b = tid; b < kRadixBins0; b += kThreads) sh[b] = 0;
    __syncthreads();
    uint32_t cur = NONE;                                // scope the shared histogram belongs to
    uint32_t seen = NONE;                               // scope whose values are cached below
    uint32_t s = w0;
    bool active = false, have_run = false, zero_case = false, local = false;
    uint64_t len = 0;
    uint32_t prefix = 0, prefix_b = NONE;               // prefix_b: first digit of the second rank (sample view)
    const float* vals = nullptr;
    // In the second pass over a sample the upper half of the shared histogram counts the keys under the
    // second rank's first digit; the two halves go to the second and third histogram slots, which are adjacent.
    const uint32_t flush_bins = (VIEW == V_SAMPLE && PASSES == 2 && pass == 1) ? 2048u : nbins;
    auto flush = [&]() {                                // adds the shared histogram to scope cur's global one
      __syncthreads();
      unsigned long long* gh = hist_of(T, cur, VIEW, pass);
      for (uint32_t b = tid; b < flush_bins; b += kThreads) {
        const uint32_t c = sh[b];
        if (c) atomicAdd(gh + b, (unsigned long long)c);
        sh[b] = 0;
      }
      __syncthreads();
      cur = NONE;
    };
    for (uint32_t t = t_beg; t < t_end; t += t_step) {
      while (t >= base_of(s + 1)) ++s;                  // base[n_scopes] = total_tiles > t
      const uint32_t lt = t - base_of(s);
      const ScopeDesc& d = desc_of(s);
      if (s != seen) {                                  // per-scope values, worked out once per scope
        seen = s;
        ScopeState* st = T.state + s;
        active = view_active<VIEW>(T, d, st);
        if (VIEW == V_SAMPLE) { len = d.samp_m; vals = T.samp_val + d.samp_base; }
        else if (VIEW == V_CAND) { len = st->cand_count; vals = T.cand_val + d.cand_base; }
        else { len = d.hi - d.lo; vals = T.residual + d.lo; }
        have_run = false;
        // A scope predicted to have threshold 0 whose non-zero entries number fewer than k: tau = 0,
        // every non-zero entry is kept and the tie quota is the rest.  No histogram is needed.
        zero_case = VIEW == V_DENSE && active && !(T.flags & GD_FLAG_NO_PREDICTION) && d.k != 0 &&
                    st->tau_lo == 0u && st->cand_count < d.k;
        // A list of one tile is selected by this CTA alone, in shared memory, during the first pass.
        local = MANY && len <= kTile;
      }
      if (!active) continue;
      if (zero_case) {
        if (pass == PASSES && lt == 0 && tid == 0) {
          ScopeState* st = T.state + s;
          st->tau = 0u; st->gt = st->cand_count; st->q = d.k - st->cand_count; st->used_dense = 1u;
        }
        continue;
      }
      if (local) {
        if (pass != 0 || lt != 0) continue;
        if (cur != NONE) flush();                       // the shared histogram must be free (and is zero)
        const SelRun run = local_select<VIEW>(T, d, s, (uint32_t)len, vals, PASSES, sh,
                                              VIEW == V_SAMPLE ? d.samp_rank : d.k, true);
        uint32_t tau_hi = 0;
        if (VIEW == V_SAMPLE && PASSES == 2)
          tau_hi = local_select<VIEW>(T, d, s, (uint32_t)len, vals, PASSES, sh, rank_hi_of(d), false).prefix << kShift1;
        if (tid == 0) {
          ScopeState* st = T.state + s;
          if (VIEW == V_SAMPLE) {
            st->tau_lo = PASSES == 3 ? run.prefix : run.prefix << kShift1;
            if (PASSES == 3) st->tau = run.prefix; else st->tau_hi = tau_hi;
          } else {
            st->tau = run.prefix; st->q = run.rank; st->gt = run.gt;
            if (VIEW == V_DENSE) st->used_dense = 1u;
          }
        }
        continue;
      }
      const uint64_t beg = (uint64_t)lt * TILE;
      if (pass == PASSES ? lt != 0 : beg >= len) continue;
      if (pass > 0 && !have_run) {                      // digits fixed by the earlier passes
        // The walk down the finished histograms resumes from where this CTA left it in the previous pass
        // (kept in shared memory for the scopes of its window), else starts from the top.  In the sample
        // view two ranks walk together: the prediction's, and the rank of the estimate of tau itself; their
        // first digits may differ, and the second rank's second-pass histogram is then the one in the third slot.
        const bool pair = VIEW == V_SAMPLE && PASSES == 2;
        const uint32_t c = s - w0;
        SelRun two[2];
        int level = 0;
        if (c < kSmemScopes && s_level[c] > 0) {
          two[0] = s_runs[c][0];
          two[1] = s_runs[c][1];
          level = s_level[c];
        } else {
          two[0].prefix = 0; two[0].rank = VIEW == V_SAMPLE ? d.samp_rank : d.k; two[0].gt = 0;
          two[1].prefix = 0; two[1].rank = pair ? rank_hi_of(d) : 0; two[1].gt = 0;
        }
        for (; level < pass; ++level) {
          const int lbits = level == 0 ? kRadixBits0 : 10;
          if (!pair) {
            two[0] = next_digit(hist_of(T, s, VIEW, level), lbits, two[0], T.ctl);
          } else if (level == 0 || two[1].prefix == two[0].prefix) {
            next_digit_pair(hist_of(T, s, VIEW, level), lbits, two, 2, T.ctl);
          } else {
            two[0] = next_digit(hist_of(T, s, VIEW, 1), 10, two[0], T.ctl);
            two[1] = next_digit(hist_of(T, s, VIEW, 2), 10, two[1], T.ctl);
          }
        }
        if (c < kSmemScopes && tid == 0) {              // read again after the next grid barrier
          s_runs[c][0] = two[0];
          s_runs[c][1] = two[1];
          s_level[c] = pass;
        }
        const SelRun run = two[0];
        uint32_t tau_hi = 0;
        if (pair) {
          if (pass == 1) prefix_b = two[1].prefix;
          else tau_hi = two[1].prefix << kShift1;
        }
        have_run = true;
        prefix = run.prefix;
        if (pass == PASSES && tid == 0) {               // the CTA with the scope's first tile records the result
          ScopeState* st = T.state + s;
          if (VIEW == V_SAMPLE) {
            // prediction: lower edge of the 21-bit bucket; sampled-threshold mode: the full key, which is the result
            st->tau_lo = PASSES == 3 ? run.prefix : run.prefix << kShift1;
            if (PASSES == 3) st->tau = run.prefix; else st->tau_hi = tau_hi;
          } else {
            st->tau = run.prefix; st->q = run.rank; st->gt = run.gt;
            if (VIEW == V_DENSE) st->used_dense = 1u;
          }
        }
      }
      if (pass == PASSES) continue;
      if (s != cur) {
        if (cur != NONE) flush();
        cur = s;
      }
      const uint64_t end = (beg + TILE < len) ? beg + TILE : len;
      // batches of 16 elements per thread: all loads of a batch are in flight before the first is used
      for (uint64_t b0 = beg; b0 < end; b0 += kTile) {
        uint32_t keys[16];
        const bool gather = VIEW == V_SAMPLE && pass == 0;
        // a whole batch inside the list (the usual case): no bounds checks, one address computation
        const bool whole = b0 + kTile <= end;
        const uint32_t valid = whole ? kTile : (uint32_t)(end - b0);   // elements of this batch
        if (gather) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const uint32_t o = (uint32_t)j * kThreads + tid;
            keys[j] = o < valid ? __float_as_uint(sample_value(T, d, s, b0 + o)) : 0u;
          }
        } else if (whole) {
          const float* src = vals + b0 + tid;
#pragma unroll
          for (int j = 0; j < 16; ++j) keys[j] = __float_as_uint(src[j * kThreads]);
        } else {
          const float* src = vals + b0;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const uint32_t o = (uint32_t)j * kThreads + tid;
            keys[j] = o < valid ? __float_as_uint(src[o]) : 0u;
          }
        }
        uint32_t digs[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const uint32_t o = (uint32_t)j * kThreads + tid;
          uint32_t digit = NONE;                                           // "does not count"
          if (whole || o < valid) {
            if (gather) T.samp_val[d.samp_base + b0 + o] = __uint_as_float(keys[j]);
            const uint32_t key = keys[j] & kAbsMask;
            if (pass == 0 || (key >> pshift) == prefix) digit = (key >> shift) & (nbins - 1u);
            else if (VIEW == V_SAMPLE && pass == 1 && (key >> pshift) == prefix_b) digit = 1024u + ((key >> shift) & 1023u);
          }
          digs[j] = digit;
        }
        // Four keys per lane at a time: a warp whose 128 keys share one bin (all zeros in a row-sparse layer,
        // or nothing to count in a later pass) issues one add; otherwise plain shared-memory adds.  Measured
        // on skewed keys, this beats grouping equal digits with match.any, whose cost is paid on every round.
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          const uint32_t d0 = __shfl_sync(0xFFFFFFFFu, digs[4 * g], 0);
          const bool same = digs[4 * g] == d0 && digs[4 * g + 1] == d0 && digs[4 * g + 2] == d0 && digs[4 * g + 3] == d0;
          if (__all_sync(0xFFFFFFFFu, same)) {
            if (lane == 0 && d0 != NONE) atomicAdd(&sh[d0], 128u);
          } else {
#pragma unroll
            for (int q = 0; q < 4; ++q)
              if (digs[4 * g + q] != NONE) atomicAdd(&sh[digs[4 * g + q]], 1u);
          }
        }
      }
    }
    if (pass == PASSES) break;
    if (cur != NONE) flush();
    if (!grid_barrier(&T.ctl->barrier[VIEW], phase, T.ctl)) return;
  }
}

// (kept out of line so that the rare path does not weigh on the registers of the usual one)
template <bool MANY>
__device__ __noinline__ void select_dense_outlined(const DevTables& T, uint32_t dense_tiles, SelectSmem<V_DENSE, MANY>& S) {
  select_body<V_DENSE, MANY>(T, dense_tiles, S);
}

}  // namespace

}  // namespace gd
