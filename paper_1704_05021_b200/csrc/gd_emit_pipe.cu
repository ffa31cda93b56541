// The fused full pass of gd_compress (Algorithm 1, step 1: grad += residuals, over the whole gradient, fused with
// the emission of the threshold candidates) as a persistent, warp-specialised pipeline: one CTA per SM, fed by bulk
// asynchronous copies.
//
//   producer warp   takes chunks (C tiles of 4096 consecutive elements of one scope) from a ticket counter and keeps
//                   up to kStages tiles of g and r in flight into shared memory (cp.async.bulk, completion on an
//                   mbarrier per stage), across chunk boundaries, whatever the other warps are doing;
//   16 consumer     wait for a tile, form v = g + r from shared memory, store v over r (128-bit stores), and put the
//   warps           rare entries with |v| >= tau_lo, in index order, into a per-warp stash; a chunk's candidates are
//                   copied to their final, index-ordered positions in the scope's list two chunks LATER, when the
//                   prefix of the chunk is long known;
//   count warp      per finished chunk: its total is published at once, its (tile, warp) counts become offsets;
//   scan warp       per finished chunk: one decoupled look-back over the earlier chunks of the scope - off the
//                   consumers' path, so its round trips cost no streaming time, and never in the way of the totals
//                   that the look-backs of other CTAs are waiting for.
//
// Against one CTA per chunk with loads through registers (gd_emit.cu, which stays for calls this kernel does not
// take): the copies in flight do not depend on how many warps are between two phases, a chunk's start-up (ticket,
// tables, thresholds) and its look-back overlap the streaming of the next one, and chunks can be small enough for the
// last of them to end together.  Tiles cut by a scope's boundary or by the end of the vector are read with plain
// loads from global memory (bulk copies need 16-byte alignment and whole tiles are what they are good at).
//
// Behind the launch that starts a call and predicts the thresholds, the pass is a programmatic dependent that does
// not wait for that grid's end: it carries the tables in its own argument and looks at marks - the control region is
// cleared, a scope's prediction is final - before it uses what they stand for (PipeStart).  The copies of a scope's
// first chunk are issued before the scope's mark is up; only the consumers' view of them waits for it.
//
// Every wait - on an mbarrier, on a mark, in the look-back - is bounded; one that runs out records GD_ERR_DEVICE_TIMEOUT, raises
// the CTA's abort flag (all other waits look at it) and the CTA leaves after its copies in flight have landed.
#include <cstring>
#include <mutex>

#include "gd_scan.cuh"

namespace gd {

namespace {

// The shape below was measured against its neighbours on 20 M, 138 M and 2^30 elements (fused pass alone): chunks of 4
// tiles placed two chunks later 49 / 260 / 1839 us; chunks of 8 placed one later 53 / 274 / 1857; chunks of 2 placed
// two or three later 55 / 307 / 2223 and 53 / 283 / 1937 (the look-backs, one at a time per CTA, fall behind); one
// CTA per chunk with loads through registers 57 / 277 / 1975.
constexpr int kStages = 5;                       // tiles of g and r in flight per SM: 5 * 32 KiB
constexpr int kDefer = 2;                        // a chunk's candidates are placed when this many later chunks are through
constexpr int kBufs = kDefer + 1;                // chunks whose stash and counts are kept
constexpr int kConsumerWarps = 16;
constexpr int kProducerWarp = kConsumerWarps, kCountWarp = kConsumerWarps + 1, kScanWarp = kConsumerWarps + 2;
constexpr int kPipeThreads = (kConsumerWarps + 3) * 32;
constexpr uint32_t kWarpSpan = kTile / kConsumerWarps;   // 256 consecutive elements of a tile per consumer warp
constexpr int kRoundsPerTile = (int)(kWarpSpan / 128u);  // 2 rounds of 128-bit accesses
constexpr uint32_t kPipeStash = 128;             // candidate slots per warp and chunk
constexpr int kMaxChunkTiles = 4;
constexpr int kMaxCounts = kMaxChunkTiles * kConsumerWarps;   // (tile, warp) counters of one chunk
constexpr uint32_t kTileBytes = kTile * 4u;

enum : uint32_t { TM_LAST = 1u, TM_CUT = 2u, TM_DONE = 4u };

struct StashEntry {
  uint32_t idx;
  float val;
};

struct TileMeta {        // what the producer tells the consumers about the tile in a stage
  uint64_t base;         // first element
  uint32_t s, t;         // scope, chunk
  uint32_t flags;        // TM_*
  uint32_t i;            // number of the tile among the chunk's tiles that overlap the scope
  uint32_t tau_lo, zmin; // candidates: key >= tau_lo; cleared early: key >= zmin
};

struct ChunkMeta {       // what the consumers tell the scan warp about a finished chunk
  uint32_t t, s, ntiles, done;
};

struct ChunkFacts {      // what a consumer warp remembers of a chunk until it places the chunk's candidates
  uint64_t base0;        // first element of the chunk's first tile
  uint32_t s, ntiles, tau_lo, zmin;
  uint32_t fill;         // candidates of this warp in the chunk (warp-uniform)
};

struct PipeStart {       // kernel argument: what lets the pass start before the launch before it has ended (enabled != 0)
  SetupBlob blob;        // the call's tables
  const uint32_t* ready; // per scope: the call's number once the scope's prediction is final
  const uint32_t* cleared;   // per clearing CTA of the launch before: the call's number once its part is cleared
  uint32_t call, clearing_ctas, scopes_off, tile0_off, enabled;
};

struct PipeSmem {
  alignas(128) float g[kStages][kTile];
  alignas(128) float r[kStages][kTile];
  StashEntry stash[kBufs][kConsumerWarps][kPipeStash];
  uint32_t cnt[kBufs][kMaxCounts];                   // candidates per (tile, warp) of the chunk in each buffer
  uint32_t off[kBufs][kMaxCounts];                   // their exclusive offsets inside the chunk
  alignas(8) uint64_t full[kStages], empty[kStages], chunk_done[kBufs], counted[kBufs], prefix_ready[kBufs];
  TileMeta meta[kStages];
  ChunkMeta cmeta[kBufs];
  uint64_t excl[kBufs];                              // candidates of the scope before the chunk
  uint32_t total[kBufs];                             // candidates of the chunk
  int abort;
  SmemTables tab;
};

#ifdef GD_PIPE_STAMPS
// debug: earliest and latest time over the CTAs at which point `i` was reached (slots behind the control block)
#define GD_PSTAMP(i)                                                                                              \
  do {                                                                                                            \
    if ((threadIdx.x & 31u) == 0u) {                                                                              \
      const unsigned long long now_ = global_timer_ns();                                                          \
      atomicMax(reinterpret_cast<unsigned long long*>(T.ctl) + 24 + 2 * (i), ~now_);                             \
      atomicMax(reinterpret_cast<unsigned long long*>(T.ctl) + 25 + 2 * (i), now_);                              \
    }                                                                                                             \
  } while (0)
#else
#define GD_PSTAMP(i) do { } while (0)
#endif

__device__ __forceinline__ void give_up(PipeSmem& sm, Ctl* ctl) {
  atomicCAS(&ctl->status, (int)GD_OK, (int)GD_ERR_DEVICE_TIMEOUT);
  *(volatile int*)&sm.abort = 1;
}

// A scope's thresholds for the pass.  Zeros are never candidates: when the prediction is 0 the list holds the non-zero
// entries, and if there are fewer than k of them the threshold is 0 and the zeros that are kept are found by the dense
// compaction.  Entries with key >= zmin (above tau_hi, the sample's estimate of the threshold itself) are almost surely
// kept: their residual slot gets +0 in the streaming store.  Each is a candidate, so its value is in the list, from
// which the compaction puts it back should it not be kept after all.  In sampled-threshold mode tau_lo is the
// threshold itself and every candidate is kept.  (Read from L2: the launch that wrote them may still be running.)
__device__ __forceinline__ void scope_thresholds(const DevTables& T, uint32_t s, uint64_t k, uint32_t* tau_lo_out, uint32_t* zmin_out) {
  const bool sampled = (T.flags & GD_FLAG_SAMPLED_THRESHOLD) != 0;
  uint32_t tau_lo = ((T.flags & GD_FLAG_NO_PREDICTION) || k == 0) ? 0xFFFFFFFFu : __ldcg(&T.state[s].tau_lo);
  if (tau_lo == 0u && !sampled) tau_lo = 1u;
  uint32_t zmin = 0xFFFFFFFFu;
  if (tau_lo != 0xFFFFFFFFu) {
    if (sampled) { if (!(T.flags & GD_FLAG_NO_EARLY_ZERO)) zmin = tau_lo; }
    else if (early_zero_enabled(T)) zmin = __ldcg(&T.state[s].tau_hi) + 1u;
  }
  *tau_lo_out = tau_lo;
  *zmin_out = zmin;
}

// A consumer warp's part of one tile: v = g + r (or g - base), the store of v, candidates into the stash.
// Returns the warp's number of candidates in the tile (warp-uniform); `fill` is its count so far in the chunk.
__device__ __forceinline__ uint32_t consume_tile(const DevTables& T, const PipeSmem& sm, int stage, const TileMeta& m,
                                                 const ScopeDesc& d, StashEntry* stash, uint32_t fill, uint32_t warp,
                                                 uint32_t lane, bool delta, const float* second) {
  const uint32_t ltm = lanemask_lt();
  const uint32_t tau_lo = m.tau_lo, zmin = m.zmin;
  const uint32_t woff = warp * kWarpSpan + lane * 4u;         // this thread's first element inside the tile
  uint32_t wc = 0;
  if (!(m.flags & TM_CUT)) {
    static_assert(kRoundsPerTile == 2, "the packed counts below hold two rounds");
    const uint64_t e0 = m.base + woff;
    float4 g4[2], r4[2];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      g4[j] = *reinterpret_cast<const float4*>(&sm.g[stage][woff + j * 128]);
      r4[j] = *reinterpret_cast<const float4*>(&sm.r[stage][woff + j * 128]);
    }
    float x[2][4];
    uint32_t kmax = 0;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      x[j][0] = delta ? __fsub_rn(g4[j].x, r4[j].x) : __fadd_rn(g4[j].x, r4[j].x);
      x[j][1] = delta ? __fsub_rn(g4[j].y, r4[j].y) : __fadd_rn(g4[j].y, r4[j].y);
      x[j][2] = delta ? __fsub_rn(g4[j].z, r4[j].z) : __fadd_rn(g4[j].z, r4[j].z);
      x[j][3] = delta ? __fsub_rn(g4[j].w, r4[j].w) : __fadd_rn(g4[j].w, r4[j].w);
#pragma unroll
      for (int c = 0; c < 4; ++c) kmax = max(kmax, __float_as_uint(x[j][c]) & kAbsMask);
    }
    if (__any_sync(0xFFFFFFFFu, kmax >= tau_lo)) {
      // Candidates are rare: one vote per tile, one warp scan for both rounds' counts (packed in one word), and a
      // loop per round that runs as often as the lane with the most candidates has them (once, mostly).
      uint32_t f[2];
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        f[j] = 0;
#pragma unroll
        for (int c = 0; c < 4; ++c) f[j] |= ((__float_as_uint(x[j][c]) & kAbsMask) >= tau_lo ? 1u : 0u) << c;
      }
      const uint32_t packed = __popc(f[0]) | (__popc(f[1]) << 16);
      uint32_t inc = packed;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if ((int)lane >= o) inc += y;
      }
      const uint32_t tot = __shfl_sync(0xFFFFFFFFu, inc, 31);
      const uint32_t exc = inc - packed;
      uint32_t p[2] = {fill + (exc & 0xFFFFu), fill + (tot & 0xFFFFu) + (exc >> 16)};   // order: (round, lane, component)
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        uint32_t ff = f[j], zm = 0, pj = p[j];
        while (ff) {
          const uint32_t c = (uint32_t)__ffs((int)ff) - 1u;
          ff &= ff - 1u;
          const float v = c < 2u ? (c == 0u ? x[j][0] : x[j][1]) : (c == 2u ? x[j][2] : x[j][3]);
          if (pj < kPipeStash) {
            stash[pj].idx = (uint32_t)(e0 + j * 128) + c;
            stash[pj].val = v;
            if ((__float_as_uint(v) & kAbsMask) >= zmin) zm |= 1u << c;
          }
          ++pj;
        }
        if (zm) {
#pragma unroll
          for (int c = 0; c < 4; ++c)
            if (zm & (1u << c)) x[j][c] = 0.0f;
        }
      }
      wc = (tot & 0xFFFFu) + (tot >> 16);
    }
#pragma unroll
    for (int j = 0; j < 2; ++j)
      *reinterpret_cast<float4*>(T.residual + e0 + j * 128) = make_float4(x[j][0], x[j][1], x[j][2], x[j][3]);
  } else {
    // a tile cut by the scope (or by the end of the vector): plain loads, element by element
    const uint64_t lo = d.lo, hi = d.hi;
#pragma unroll 1
    for (int j = 0; j < kRoundsPerTile; ++j) {
      float x[4] = {0.f, 0.f, 0.f, 0.f};
      uint32_t f = 0, in = 0;
      const uint64_t e0 = m.base + woff + j * 128;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const uint64_t e = e0 + c;
        if (e >= lo && e < hi) {
          x[c] = delta ? __fsub_rn(__ldg(T.grad + e), second[e]) : __fadd_rn(__ldg(T.grad + e), second[e]);
          in |= 1u << c;
          f |= ((__float_as_uint(x[c]) & kAbsMask) >= tau_lo ? 1u : 0u) << c;
        }
      }
      if (__any_sync(0xFFFFFFFFu, f != 0u)) {
        const uint32_t b0 = __ballot_sync(0xFFFFFFFFu, f & 1u), b1 = __ballot_sync(0xFFFFFFFFu, f & 2u);
        const uint32_t b2 = __ballot_sync(0xFFFFFFFFu, f & 4u), b3 = __ballot_sync(0xFFFFFFFFu, f & 8u);
        if (f) {
          uint32_t p = fill + wc + __popc(b0 & ltm) + __popc(b1 & ltm) + __popc(b2 & ltm) + __popc(b3 & ltm);
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            if (f & (1u << c)) {
              if (p < kPipeStash) {
                stash[p].idx = (uint32_t)(e0 + c);
                stash[p].val = x[c];
                if ((__float_as_uint(x[c]) & kAbsMask) >= zmin) x[c] = 0.0f;
              }
              ++p;
            }
          }
        }
        wc += __popc(b0) + __popc(b1) + __popc(b2) + __popc(b3);
      }
#pragma unroll
      for (int c = 0; c < 4; ++c)
        if (in & (1u << c)) T.residual[e0 + c] = x[c];
    }
  }
  return wc;
}

// A consumer warp's candidates of the chunk in buffer `buf` go to their final positions in the scope's list.
__device__ __forceinline__ void place_chunk(const DevTables& T, PipeSmem& sm, int buf, const ChunkFacts& cm, uint32_t warp,
                                            uint32_t lane, const ScopeDesc* scopes) {
  const uint32_t fill = cm.fill;
  if (fill == 0u) return;
  const ScopeDesc& d = scopes[cm.s];
  const uint64_t excl = sm.excl[buf];
  const uint32_t tau_lo = cm.tau_lo, zmin = cm.zmin;
  const uint64_t cap = d.cand_cap;
  uint32_t* cidx = T.cand_idx + d.cand_base;
  float* cval = T.cand_val + d.cand_base;
  StashEntry* stash = sm.stash[buf][warp];
  const uint32_t ltm = lanemask_lt();
  if (fill <= kPipeStash) {
    // One loop over the warp's stash (a few entries per tile: a loop per tile would run with most lanes idle and four
    // times the shared-memory round trips).  Entry e belongs to the last tile whose run starts at or before it.
    uint32_t first[kMaxChunkTiles], shift[kMaxChunkTiles];   // first stash entry of tile i; (offset in the chunk) - first
    {
      uint32_t a = 0;
#pragma unroll
      for (int i = 0; i < kMaxChunkTiles; ++i) {
        const bool live = (uint32_t)i < cm.ntiles;
        const uint32_t c = live ? sm.cnt[buf][i * kConsumerWarps + warp] : 0u;
        const uint32_t o = live ? sm.off[buf][i * kConsumerWarps + warp] : 0u;
        first[i] = a;
        shift[i] = o - a;
        a += c;
      }
    }
    for (uint32_t e = lane; e < fill; e += 32) {
      uint32_t sh = shift[0];
#pragma unroll
      for (int i = 1; i < kMaxChunkTiles; ++i)
        if (e >= first[i]) sh = shift[i];
      const uint64_t pos = excl + (uint32_t)(e + sh);
      const StashEntry se = stash[e];
      if (pos < cap) {
        cidx[pos] = se.idx;
        cval[pos] = se.val;
      } else if ((__float_as_uint(se.val) & kAbsMask) >= zmin) {
        // the list is full (the scope will be selected densely): the slot must hold v again
        T.residual[se.idx] = se.val;
        T.state[cm.s].early_bad = 1u;
      }
    }
    return;
  }
  // more candidates than the stash holds: read this warp's elements back.  They are v, once the slots that were
  // cleared early (all of them are in the stash) hold v again; every entry at or above zmin is cleared (again) as it
  // goes to the list.
  if (zmin != 0xFFFFFFFFu) {
    for (uint32_t e = lane; e < kPipeStash; e += 32)
      if ((__float_as_uint(stash[e].val) & kAbsMask) >= zmin) T.residual[stash[e].idx] = stash[e].val;
    __syncwarp();
  }
  const uint64_t lo = d.lo, hi = d.hi;
  // one (tile, round) of this warp's elements, now in x[0..3] with in-scope mask `in`: its candidates go to the list
  auto emit_round = [&](const float* x, uint32_t in, uint64_t e0, uint64_t& run) {
    uint32_t f = 0;
#pragma unroll
    for (int c = 0; c < 4; ++c) f |= (((in >> c) & 1u) && (__float_as_uint(x[c]) & kAbsMask) >= tau_lo ? 1u : 0u) << c;
    const uint32_t b0 = __ballot_sync(0xFFFFFFFFu, f & 1u), b1 = __ballot_sync(0xFFFFFFFFu, f & 2u);
    const uint32_t b2 = __ballot_sync(0xFFFFFFFFu, f & 4u), b3 = __ballot_sync(0xFFFFFFFFu, f & 8u);
    if (f) {
      uint64_t pos = run + __popc(b0 & ltm) + __popc(b1 & ltm) + __popc(b2 & ltm) + __popc(b3 & ltm);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        if (f & (1u << c)) {
          if (pos < cap) {
            cidx[pos] = (uint32_t)(e0 + c);
            cval[pos] = x[c];
            if ((__float_as_uint(x[c]) & kAbsMask) >= zmin) T.residual[e0 + c] = 0.0f;
          }
          ++pos;
        }
      }
    }
    run += __popc(b0) + __popc(b1) + __popc(b2) + __popc(b3);
  };
  const uint64_t wbase = cm.base0 + warp * kWarpSpan + lane * 4u;        // this thread's first element in the chunk's first tile
  if (cm.base0 >= lo && cm.base0 + (uint64_t)cm.ntiles * kTile <= hi) {
    // whole tiles: 128-bit loads from L2 (other lanes may just have put v back), four tiles' worth in flight
    constexpr uint32_t kBatch = 4;
    for (uint32_t i0 = 0; i0 < cm.ntiles; i0 += kBatch) {
      float4 v[kBatch][kRoundsPerTile];
#pragma unroll
      for (uint32_t u = 0; u < kBatch; ++u) {
        const uint32_t i = i0 + u;
        const bool live = i < cm.ntiles && sm.cnt[buf][i * kConsumerWarps + warp] != 0u;    // (warp-uniform)
#pragma unroll
        for (int j = 0; j < kRoundsPerTile; ++j)
          v[u][j] = live ? __ldcg(reinterpret_cast<const float4*>(T.residual + wbase + (uint64_t)i * kTile + j * 128))
                         : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (uint32_t u = 0; u < kBatch; ++u) {
        const uint32_t i = i0 + u;
        if (i >= cm.ntiles || sm.cnt[buf][i * kConsumerWarps + warp] == 0u) continue;
        uint64_t run = excl + sm.off[buf][i * kConsumerWarps + warp];
#pragma unroll
        for (int j = 0; j < kRoundsPerTile; ++j) {
          const float x[4] = {v[u][j].x, v[u][j].y, v[u][j].z, v[u][j].w};
          emit_round(x, 0xFu, wbase + (uint64_t)i * kTile + j * 128, run);
        }
      }
    }
    return;
  }
  for (uint32_t i = 0; i < cm.ntiles; ++i) {                               // a chunk with cut tiles: element by element
    if (sm.cnt[buf][i * kConsumerWarps + warp] == 0u) continue;
    uint64_t run = excl + sm.off[buf][i * kConsumerWarps + warp];
#pragma unroll 1
    for (int j = 0; j < kRoundsPerTile; ++j) {
      float x[4] = {0.f, 0.f, 0.f, 0.f};
      uint32_t in = 0;
      const uint64_t e0 = wbase + (uint64_t)i * kTile + j * 128;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        if (e0 + c >= lo && e0 + c < hi) {
          x[c] = __ldcg(T.residual + e0 + c);
          in |= 1u << c;
        }
      }
      emit_round(x, in, e0, run);
    }
  }
}

__global__ void __launch_bounds__(kPipeThreads, 1) add_emit_pipe_kernel(const __grid_constant__ DevTables T, uint32_t total_chunks,
                                                                        const __grid_constant__ PipeStart start) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  PipeSmem& sm = *reinterpret_cast<PipeSmem*>(smem_raw);
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  const ScopeDesc* scopes;
  const uint32_t* tile0;
  if (tid == 0) {
    for (int st = 0; st < kStages; ++st) {
      mbar_init(&sm.full[st], 1u);                            // the producer's arrive (+ the bytes of its two copies)
      mbar_init(&sm.empty[st], (uint32_t)kConsumerWarps);
    }
    for (int b = 0; b < kBufs; ++b) {
      mbar_init(&sm.chunk_done[b], (uint32_t)kConsumerWarps);
      mbar_init(&sm.counted[b], 1u);
      mbar_init(&sm.prefix_ready[b], 1u);
    }
    sm.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (start.enabled) {
    // The tables come with the launch, and nothing else of the launch before this one (the start of the call and the
    // prediction) is touched before that launch has marked it done: the cleared control region before the first
    // ticket is taken, a scope's prediction before a tile of it is handed to the consumers.  So this grid need not wait for
    // that one to end - only for the CTA that finishes the prediction of the scope it is about to stream.
    const uint32_t words = T.n_scopes * (uint32_t)(sizeof(ScopeDesc) / 8);
    const uint64_t* src = reinterpret_cast<const uint64_t*>(start.blob.bytes + start.scopes_off);
    uint64_t* dst = reinterpret_cast<uint64_t*>(sm.tab.scopes);
    for (uint32_t i = tid; i < words; i += kPipeThreads) dst[i] = src[i];
    const uint32_t* t0 = reinterpret_cast<const uint32_t*>(start.blob.bytes + start.tile0_off);
    for (uint32_t i = tid; i <= T.n_scopes; i += kPipeThreads) sm.tab.tile0[i] = t0[i];
    scopes = sm.tab.scopes;
    tile0 = sm.tab.tile0;
  } else {
    pdl_wait();   // nothing the kernels before this one wrote - tables, thresholds, the residual - is read above this line
    load_tables(T, L_EMIT, &sm.tab, &scopes, &tile0);         // (at most kSmemScopes scopes: the launcher checks)
  }
  if (tid == 0) GD_PSTAMP(0);
  __syncthreads();
  const volatile int* abort = &sm.abort;
  const bool delta = T.delta_base != nullptr;                 // v = g - base instead of g + r
  const float* second = delta ? T.delta_base : T.residual;
  const uint32_t C = T.emit_chunk_tiles;
  const uint64_t CH = (uint64_t)C * kTile;

  if (warp == (uint32_t)kProducerWarp) {
    // ------------------------------------------------------------ producer
    if (start.enabled) {
      // the control region (ticket counter, look-back descriptors, status) must have been cleared: all lanes look
      uint32_t spins = 0;
      uint64_t t0w = 0;
      for (;;) {
        bool all = true;
        for (uint32_t z = lane; z < start.clearing_ctas; z += 32) all = all && ld_acquire_u32(start.cleared + z) == start.call;
        if (__all_sync(0xFFFFFFFFu, all)) break;
        ++spins;
        if (spins == 8u) t0w = global_timer_ns();
        if (spins > 8u) {
          __nanosleep(100);
          if (__any_sync(0xFFFFFFFFu, global_timer_ns() - t0w > kWaitBudgetNs)) {
            if (lane == 0) give_up(sm, T.ctl);
            return;
          }
        }
      }
    }
    if (lane != 0) return;
    uint32_t cached_s = 0xFFFFFFFFu, tau_lo = 0xFFFFFFFFu, zmin = 0xFFFFFFFFu;
    int stage = 0;
    uint32_t parity = 1;                   // (a fresh mbarrier reads as "the phase of parity 1 has completed")
    uint32_t armed = 0, armed_parity = 0;  // stages used, and the parity of the latest phase of each one's full barrier
    bool ok = true;
    // Chunks are handed out by a ticket counter, the first ones too: a chunk that another CTA's look-back waits for
    // is then always held by a CTA that is running, however many of the grid's CTAs are resident at once.
    uint32_t t_next = atomicAdd(&T.ctl->ticket[L_EMIT], 1u);
    while (ok) {
      const uint32_t t = t_next;
      if (t >= total_chunks) break;
      t_next = atomicAdd(&T.ctl->ticket[L_EMIT], 1u);         // (in flight while this chunk's copies are issued)
      const uint32_t s = scope_of_tile(tile0, T.n_scopes, t);
      const ScopeDesc& d = scopes[s];
      const uint64_t lo = d.lo, hi = d.hi;
      const uint64_t cbase = (lo / CH + (t - tile0[s])) * CH;
      // the chunk's tiles that overlap the scope are consecutive
      uint32_t i_first = 0, i_last = C - 1u;
      while (i_first < C && cbase + (uint64_t)(i_first + 1u) * kTile <= lo) ++i_first;
      while (i_last > i_first && cbase + (uint64_t)i_last * kTile >= hi) --i_last;
      uint32_t issued = 0;                 // tiles of this chunk whose copies are under way already
      if (s != cached_s) {
        if (start.enabled && ld_acquire_u32(start.ready + s) != start.call) {
          // The scope's prediction must be final before a consumer sees a tile of it - the copies need not wait:
          // they are issued now (their bytes announced on the stage's barrier, the producer's arrive held back), so
          // that the chunk has landed by the time the thresholds exist.
#ifndef GD_NO_EARLY_LOADS
          if (i_last - i_first < (uint32_t)kStages)
#else
          if (false)
#endif
          {
            int st = stage;
            uint32_t par = parity;
            for (uint32_t i = i_first; i <= i_last; ++i) {
              if (!mbar_wait(&sm.empty[st], par, abort)) { ok = false; break; }
              const uint64_t base = cbase + (uint64_t)i * kTile;
              if (base >= lo && base + kTile <= hi) {
                mbar_expect_tx(&sm.full[st], 2u * kTileBytes);
                bulk_load(sm.g[st], T.grad + base, kTileBytes, &sm.full[st]);
                bulk_load(sm.r[st], second + base, kTileBytes, &sm.full[st]);
              }
              ++issued;
              if (++st == kStages) { st = 0; par ^= 1u; }
            }
          }
          uint32_t spins = 0;
          uint64_t t0w = 0;
          while (ok && ld_acquire_u32(start.ready + s) != start.call) {
            ++spins;
            if (spins == 8u) t0w = global_timer_ns();
            if (spins > 8u) {
              __nanosleep(100);
              if (*abort || global_timer_ns() - t0w > kWaitBudgetNs) ok = false;
            }
          }
        }
        if (ok) {
          scope_thresholds(T, s, d.k, &tau_lo, &zmin);
          cached_s = s;
        } else {
          tau_lo = 0xFFFFFFFFu; zmin = 0xFFFFFFFFu;             // (giving up: the tiles under way are handed on empty-handed)
        }
      }
      for (uint32_t i = i_first; i <= i_last; ++i) {
        const bool under_way = i - i_first < issued;
        if (!under_way) {
          if (!ok) break;
          if (!mbar_wait(&sm.empty[stage], parity, abort)) { ok = false; break; }
        }
        const uint64_t base = cbase + (uint64_t)i * kTile;
        const bool cut = !(base >= lo && base + kTile <= hi);
        TileMeta m;
        m.base = base; m.s = s; m.t = t;
        m.flags = (i == i_last ? TM_LAST : 0u) | (cut ? TM_CUT : 0u);
        m.i = i - i_first;
        m.tau_lo = tau_lo; m.zmin = zmin;
        sm.meta[stage] = m;
        if (cut || under_way) {
          mbar_arrive(&sm.full[stage]);
        } else {
          mbar_arrive_expect_tx(&sm.full[stage], 2u * kTileBytes);
          bulk_load(sm.g[stage], T.grad + base, kTileBytes, &sm.full[stage]);
          bulk_load(sm.r[stage], second + base, kTileBytes, &sm.full[stage]);
        }
        armed |= 1u << stage;                                  // (the stage's latest phase, with or without copies)
        armed_parity = (armed_parity & ~(1u << stage)) | ((parity ^ 1u) << stage);
        if (++stage == kStages) { stage = 0; parity ^= 1u; }
      }
    }
    if (ok && mbar_wait(&sm.empty[stage], parity, abort)) {   // the end: a tile that says so
      TileMeta m;
      m.base = 0; m.s = 0; m.t = 0; m.flags = TM_DONE; m.i = 0; m.tau_lo = 0xFFFFFFFFu; m.zmin = 0xFFFFFFFFu;
      sm.meta[stage] = m;
      mbar_arrive(&sm.full[stage]);
      armed |= 1u << stage;
      armed_parity = (armed_parity & ~(1u << stage)) | ((parity ^ 1u) << stage);
    } else if (!*abort) {
      give_up(sm, T.ctl);
    }
    // nothing of this CTA's may still be in flight when it leaves (all landed long ago unless the CTA gave up)
    for (int st = 0; st < kStages; ++st)
      if ((armed >> st) & 1u) {
        uint32_t spins = 0;
        const uint64_t t0 = global_timer_ns();
        while (!mbar_try_wait(&sm.full[st], (armed_parity >> st) & 1u))
          if ((++spins & 31u) == 0u && global_timer_ns() - t0 > kWaitBudgetNs) break;
      }
    return;
  }

  if (warp == (uint32_t)kCountWarp) {
    // ------------------------------------------------------------ count warp: a finished chunk's total is published
    // at once (the look-backs of other chunks wait for nothing else), its (tile, warp) counts become offsets
    int buf = 0;
    uint32_t phases = 0;                   // bit b: parity of chunk_done[b]'s next phase
    for (;;) {
      if (!mbar_wait(&sm.chunk_done[buf], (phases >> buf) & 1u, abort)) {
        if (!*abort && lane == 0) give_up(sm, T.ctl);
        break;
      }
      phases ^= 1u << buf;
      const ChunkMeta cm = sm.cmeta[buf];
      if (!cm.done) {
        constexpr int PER = (kMaxCounts + 31) / 32;
        const uint32_t E = cm.ntiles * (uint32_t)kConsumerWarps;
        uint32_t a[PER], sum = 0;
#pragma unroll
        for (int p = 0; p < PER; ++p) {
          const uint32_t e = lane * PER + p;
          a[p] = e < E ? sm.cnt[buf][e] : 0u;
          sum += a[p];
        }
        uint32_t inc = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
          if ((int)lane >= o) inc += y;
        }
        if (lane == 31) {
          tile_publish(reinterpret_cast<uint4*>(T.desc_emit), cm.t, tile0[cm.s], inc, 0);
          sm.total[buf] = inc;
        }
        uint32_t run = inc - sum;
#pragma unroll
        for (int p = 0; p < PER; ++p) {
          const uint32_t e = lane * PER + p;
          if (e < E) sm.off[buf][e] = run;
          run += a[p];
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.counted[buf]);           // (the end of the stream is passed on the same way)
      if (cm.done) break;
      if (++buf == kBufs) buf = 0;
    }
    return;
  }

  if (warp == (uint32_t)kScanWarp) {
    // ------------------------------------------------------------ scan warp: the look-backs, one chunk after another
    int buf = 0;
    uint32_t phases = 0;                   // bit b: parity of counted[b]'s next phase
    for (;;) {
      if (!mbar_wait(&sm.counted[buf], (phases >> buf) & 1u, abort)) {
        if (!*abort && lane == 0) give_up(sm, T.ctl);
        break;
      }
      phases ^= 1u << buf;
      const ChunkMeta cm = sm.cmeta[buf];
      if (cm.done) break;
      const uint32_t total = sm.total[buf];
      const uint32_t first = tile0[cm.s], nchunks = tile0[cm.s + 1] - first;
      uint64_t ex_a, ex_b;
      const bool ok = tile_lookback(reinterpret_cast<uint4*>(T.desc_emit), cm.t, first, total, 0, ex_a, ex_b, T.ctl,
                                    kLookbackSpinLimit, kWaitBudgetNs, true);
      if (lane == 0) {
        sm.excl[buf] = ex_a;
        if (!ok) *(volatile int*)&sm.abort = 1;               // (the look-back has recorded the error)
        if (ok && cm.t - first == nchunks - 1u) {
          const ScopeDesc& d = scopes[cm.s];
          const uint64_t m = ex_a + total;
          T.state[cm.s].cand_count = m;
          if (T.flags & GD_FLAG_SAMPLED_THRESHOLD) {
            if (m > d.cand_cap) atomicCAS(&T.ctl->status, (int)GD_OK, (int)GD_ERR_OVERFLOW);
          } else if (!(T.flags & GD_FLAG_NO_PREDICTION) && (m < d.k || m > d.cand_cap)) {
            atomicAdd(&T.ctl->dense_needed, 1u);
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.prefix_ready[buf]);
      if (!ok) break;
      if (++buf == kBufs) buf = 0;
    }
    return;
  }

  // -------------------------------------------------------------- consumers
  int stage = 0, buf = 0;
  uint32_t parity = 0;                     // of full[stage]'s next phase
  uint32_t ready_phases = 0;               // bit b: parity of prefix_ready[b]'s next phase
  uint32_t fill = 0;                       // candidates of this warp in the current chunk (warp-uniform)
  uint64_t base0 = 0;                      // first element of the current chunk's first tile
  ChunkFacts pend[kDefer];                 // the chunks before the current one that are not placed yet, oldest first
  int n_pend = 0;
#pragma unroll
  for (int u = 0; u < kDefer; ++u) { pend[u].base0 = 0; pend[u].s = 0; pend[u].ntiles = 0; pend[u].tau_lo = 0; pend[u].zmin = 0; pend[u].fill = 0; }
  bool failed = false;
  // Places the oldest pending chunk (it lives n_pend buffers behind `buf`, the current one).
  auto place_oldest = [&]() -> bool {
    int pb = buf - n_pend;
    if (pb < 0) pb += kBufs;
    if (!mbar_wait(&sm.prefix_ready[pb], (ready_phases >> pb) & 1u, abort) || *abort) return false;
    ready_phases ^= 1u << pb;
    place_chunk(T, sm, pb, pend[0], warp, lane, scopes);
    __syncwarp();
#pragma unroll
    for (int u = 0; u + 1 < kDefer; ++u) pend[u] = pend[u + 1];
    --n_pend;
    return true;
  };
#ifdef GD_PIPE_STAMPS
  bool first_tile = true;
#endif
  for (;;) {
    if (!mbar_wait(&sm.full[stage], parity, abort)) { failed = true; break; }
    const TileMeta m = sm.meta[stage];
#ifdef GD_PIPE_STAMPS
    if (first_tile && warp == 0) { GD_PSTAMP(1); first_tile = false; }
    if ((m.flags & TM_DONE) && warp == 0) GD_PSTAMP(2);
#endif
    if (m.flags & TM_DONE) break;
    const uint32_t wc = consume_tile(T, sm, stage, m, scopes[m.s], sm.stash[buf][warp], fill, warp, lane, delta, second);
    if (lane == 0) sm.cnt[buf][m.i * kConsumerWarps + warp] = wc;
    if (m.i == 0u) base0 = m.base;
    fill += wc;
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm.empty[stage]);            // the stage may be filled again
    if (++stage == kStages) { stage = 0; parity ^= 1u; }
    if (m.flags & TM_LAST) {
      if (warp == 0 && lane == 0) {
        ChunkMeta cm;
        cm.t = m.t; cm.s = m.s; cm.ntiles = m.i + 1u; cm.done = 0u;
        sm.cmeta[buf] = cm;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.chunk_done[buf]);       // the scan warp takes it from here
      // the chunk kDefer chunks back: its prefix is long known; its buffer is the next one to be used
      if (n_pend == kDefer && !place_oldest()) { failed = true; break; }
      ChunkFacts done;
      done.base0 = base0; done.s = m.s; done.ntiles = m.i + 1u; done.tau_lo = m.tau_lo; done.zmin = m.zmin; done.fill = fill;
#pragma unroll
      for (int u = 0; u < kDefer; ++u)
        if (u == n_pend) pend[u] = done;
      ++n_pend;
      fill = 0;
      if (++buf == kBufs) buf = 0;
    }
  }
  if (failed) {
    if (!*abort && lane == 0) give_up(sm, T.ctl);
    return;
  }
  // no more chunks: tell the scan warp (the current buffer is free), then finish the pending chunks
  if (warp == 0 && lane == 0) {
    ChunkMeta cm;
    cm.t = 0; cm.s = 0; cm.ntiles = 0; cm.done = 1u;
    sm.cmeta[buf] = cm;
  }
  __syncwarp();
  if (lane == 0) mbar_arrive(&sm.chunk_done[buf]);
  while (n_pend > 0) {
    if (!place_oldest()) {
      if (!*abort && lane == 0) give_up(sm, T.ctl);
      return;
    }
  }
  if (warp == 0) GD_PSTAMP(3);
}

// Self-test of the bounded mbarrier wait: one warp waits, for at most budget_ns, on an mbarrier at which nothing
// arrives, records the timeout the way the pipeline does and notes that the wait gave up in the statistics' n_kept.
__global__ void __launch_bounds__(32) mbar_wait_selftest_kernel(Ctl* ctl, uint64_t budget_ns) {
  __shared__ alignas(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1u);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  const bool ok = mbar_wait(&bar, 0u, &abort_flag, budget_ns);
  if (threadIdx.x == 0) {
    if (!ok) atomicCAS(&ctl->status, (int)GD_OK, (int)GD_ERR_DEVICE_TIMEOUT);
    ctl->n_kept = ok ? 0u : 1u;
  }
}

}  // namespace

cudaError_t launch_mbar_wait_selftest(void* workspace, uint64_t budget_ns, cudaStream_t stream) {
  mbar_wait_selftest_kernel<<<1, 32, 0, stream>>>((Ctl*)workspace, budget_ns);
  GD_LAUNCH_CHECK();
  return cudaSuccess;
}

namespace {

// 1 if the current device gives the kernel its shared memory (asked once per device, with the attribute set on the
// way), -1 if it does not or cannot be asked.
int pipe_configured() {
  static PerDeviceInt configured;                          // 0: not asked yet
  int dev = -1;
  int c = configured.get(&dev);
  if (c != 0) return c;
  if (dev < 0) return -1;
  const cudaError_t e = cudaFuncSetAttribute(add_emit_pipe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(PipeSmem));
  if (e != cudaSuccess) (void)cudaGetLastError();          // (a device with less shared memory: the first version of the pass runs)
  c = e == cudaSuccess ? 1 : -1;
  configured.set(dev, c);
  return c;
}

}  // namespace

// Whether the pipelined kernel takes this call: tables that fit shared memory, 16-byte aligned vectors, a device that
// has the shared memory.
bool add_emit_pipe_takes(const DevTables& T) {
  if (T.n_scopes > kSmemScopes || T.emit_chunk_tiles > (uint32_t)kMaxChunkTiles) return false;
  const uintptr_t a = (uintptr_t)T.grad | (uintptr_t)T.residual | (uintptr_t)T.delta_base;
  return (a & 15u) == 0u && pipe_configured() > 0;
}

cudaError_t launch_add_emit_pipe(const DevTables& T, const uint32_t* tiles, cudaStream_t stream, const EmitEarly* early) {
  if (pipe_configured() <= 0) return cudaErrorInvalidDevice;
  uint32_t grid = (uint32_t)sm_count();
  if (grid > tiles[L_EMIT]) grid = tiles[L_EMIT];
  static PipeStart start;                                    // (large: kept off the stack; filled under the lock below)
  static std::mutex start_mutex;
  std::lock_guard<std::mutex> lock(start_mutex);
  start.enabled = 0;
  if (early && early->tables_bytes <= kSetupBlobBytes && early->clearing_ctas <= kStartMarks && T.n_scopes <= kSmemScopes) {
    std::memcpy(start.blob.bytes, early->tables_src, early->tables_bytes);
    start.ready = early->ready;
    start.cleared = early->cleared;
    start.call = early->call;
    start.clearing_ctas = early->clearing_ctas;
    start.scopes_off = (uint32_t)early->scopes_off;
    start.tile0_off = (uint32_t)early->tile0_emit_off;
    start.enabled = 1;
  }
  const cudaError_t e = launch_dependent(add_emit_pipe_kernel, dim3(grid), dim3(kPipeThreads), sizeof(PipeSmem), stream, T, tiles[L_EMIT], start);
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace gd
