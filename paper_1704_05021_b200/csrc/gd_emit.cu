// The fused full pass of gd_compress: Algorithm 1, step 1 (grad += residuals) over the whole
// gradient, fused with the emission of the threshold candidates.
//
// One CTA streams one chunk of C tiles (C * 4096 consecutive elements) of one scope:
//   phase A  per tile: 128-bit loads of g and r, v = g + r, 128-bit store of v over r; the rare
//            entries with |v| >= tau_lo (the predicted lower bound) are appended, in order, to a
//            small per-warp stash in shared memory;
//   scan     one decoupled look-back per chunk gives the number of candidates in all earlier
//            chunks of the scope;
//   phase B  every warp copies its stash to the scope's candidate list at its final, index-ordered
//            position.  A warp whose stash overflowed (a dense run of candidates) re-reads its own
//            part of the chunk instead.
// The look-back is per chunk, not per tile, so that its latency (a few L2 round trips) is paid
// once per C * 48 KiB of traffic and the chain of prefixes never limits the streaming rate.
#include "gd_scan.cuh"

namespace gd {

namespace {

#ifndef GD_EMIT_STASH
#define GD_EMIT_STASH 256
#endif
constexpr uint32_t kStash = GD_EMIT_STASH;   // candidate slots per warp and chunk in shared memory
#ifndef GD_EMIT_WARPS
#define GD_EMIT_WARPS 8
#endif
constexpr int kEmitWarps = GD_EMIT_WARPS;            // warps per CTA of the fused pass
constexpr int kEmitThreads = 32 * kEmitWarps;
constexpr uint32_t kEmitTile = 512u * kEmitWarps;    // elements one CTA handles per round trip: 512 per warp

struct StashEntry {
  uint32_t idx;
  float val;
};

// Chunks are aligned to C * kTile elements of the flat vector; a chunk that straddles a scope
// boundary is processed once per scope, each pass touching only its own scope's elements.  Inside a
// tile, warp w owns 512 consecutive elements and reads them as four rounds of 128-bit accesses (lane
// l, round j -> elements w*512 + j*128 + l*4 .. +3): candidate order inside a warp is (round, lane,
// component), across warps (warp), across tiles (tile).
template <int C>
__global__ void __launch_bounds__(kEmitThreads, 1024 / kEmitThreads) add_emit_kernel(const __grid_constant__ DevTables T) {
  constexpr int CT = C * (int)(kTile / kEmitTile);   // tiles of kEmitTile elements per chunk
  constexpr int E = CT * kEmitWarps;         // (tile, warp) counters of one chunk
  constexpr int PER = (E + 31) / 32;
  __shared__ uint32_t s_chunk;
  __shared__ uint32_t s_cnt[E];              // candidates per (tile, warp)
  __shared__ uint32_t s_off[E];              // their exclusive offsets inside the chunk
  __shared__ uint64_t s_excl;
  __shared__ uint32_t s_total;
  __shared__ int s_ok;
  __shared__ StashEntry s_stash[kEmitWarps][kStash];
  __shared__ SmemTables s_tab;
  const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
  if (tid == 0) s_chunk = atomicAdd(&T.ctl->ticket[L_EMIT], 1u);
  const ScopeDesc* scopes;
  const uint32_t* tile0;
  load_tables(T, L_EMIT, &s_tab, &scopes, &tile0);
  __syncthreads();
  const uint32_t t = s_chunk;
  // With more scopes than the shared tables hold, the chunk's scope is found by one CTA-wide count
  // over the global table (a binary search there would be a chain of dependent loads).
  const uint32_t s = T.n_scopes <= kSmemScopes ? scope_of_tile(tile0, T.n_scopes, t)
                                                : block_count_le(tile0, T.n_scopes, t) - 1u;
  const ScopeDesc& d = scopes[s];
  const uint64_t lo = d.lo, hi = d.hi;
  const uint32_t first = tile0[s], nchunks = tile0[s + 1] - first;
  const uint32_t lt = t - first;
  constexpr uint64_t CH = (uint64_t)C * kTile;
  const uint64_t cbase = (lo / CH + lt) * CH;
  // Zeros are never candidates: when the prediction is 0 the list holds the non-zero entries, and if
  // there are fewer than k of them the threshold is 0 and the zeros that are kept are found by the
  // dense compaction alone (no dense selection is needed to know tau = 0).
  uint32_t tau_lo = ((T.flags & GD_FLAG_NO_PREDICTION) || d.k == 0) ? 0xFFFFFFFFu : T.state[s].tau_lo;
  const bool sampled = (T.flags & GD_FLAG_SAMPLED_THRESHOLD) != 0;   // tau_lo is the threshold itself: keep key >= tau_lo
  if (tau_lo == 0u && !sampled) tau_lo = 1u;
  // Entries with key >= zmin (above tau_hi, the sample's estimate of the threshold itself) are almost surely kept:
  // their residual slot gets +0 right here, in the streaming store, instead of a scattered store later.
  // Each of them is a candidate, so its value is in the list, from which the compaction puts it back
  // should it not be kept after all.  Only entries that reached the stash are treated so.
  // In sampled-threshold mode every candidate is kept, so every candidate is treated so.
  uint32_t zmin = 0xFFFFFFFFu;               // smallest key cleared early (keys are at most 0x7FFFFFFF: none)
  if (tau_lo != 0xFFFFFFFFu) {
    if (sampled) { if (!(T.flags & GD_FLAG_NO_EARLY_ZERO)) zmin = tau_lo; }
    else if (early_zero_enabled(T)) zmin = T.state[s].tau_hi + 1u;
  }
  const uint64_t toff = (uint64_t)warp * 512u + lane * 4u;   // this thread's first element inside a tile
  const uint32_t ltm = lanemask_lt();
  StashEntry* stash = s_stash[warp];
  const bool delta = T.delta_base != nullptr;            // v = g - base instead of g + r
  const float* second = delta ? T.delta_base : T.residual;

  // ---- phase A
  uint32_t fill = 0;                         // candidates of this warp so far in the chunk (warp-uniform)
#pragma unroll 1
  for (int i = 0; i < CT; ++i) {
    const uint64_t base = cbase + (uint64_t)i * kEmitTile;
    uint32_t wc = 0;                         // candidates of this warp in this tile (warp-uniform)
    if (base >= lo && base + kEmitTile <= hi) {
      const uint64_t e0 = base + toff;
      float4 g4[4], r4[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) g4[j] = __ldcs(reinterpret_cast<const float4*>(T.grad + e0 + j * 128));
#pragma unroll
      for (int j = 0; j < 4; ++j) r4[j] = *reinterpret_cast<const float4*>(second + e0 + j * 128);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float x[4];
        x[0] = delta ? __fsub_rn(g4[j].x, r4[j].x) : __fadd_rn(g4[j].x, r4[j].x);
        x[1] = delta ? __fsub_rn(g4[j].y, r4[j].y) : __fadd_rn(g4[j].y, r4[j].y);
        x[2] = delta ? __fsub_rn(g4[j].z, r4[j].z) : __fadd_rn(g4[j].z, r4[j].z);
        x[3] = delta ? __fsub_rn(g4[j].w, r4[j].w) : __fadd_rn(g4[j].w, r4[j].w);
        uint32_t f = 0;
#pragma unroll
        for (int c = 0; c < 4; ++c) f |= ((__float_as_uint(x[c]) & kAbsMask) >= tau_lo ? 1u : 0u) << c;
        if (__any_sync(0xFFFFFFFFu, f != 0u)) {
          const uint32_t b0 = __ballot_sync(0xFFFFFFFFu, f & 1u), b1 = __ballot_sync(0xFFFFFFFFu, f & 2u);
          const uint32_t b2 = __ballot_sync(0xFFFFFFFFu, f & 4u), b3 = __ballot_sync(0xFFFFFFFFu, f & 8u);
          if (f) {
            uint32_t p = fill + wc + __popc(b0 & ltm) + __popc(b1 & ltm) + __popc(b2 & ltm) + __popc(b3 & ltm);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              if (f & (1u << c)) {
                if (p < kStash) {
                  stash[p].idx = (uint32_t)(e0 + j * 128 + c);
                  stash[p].val = x[c];
                  if ((__float_as_uint(x[c]) & kAbsMask) >= zmin) x[c] = 0.0f;
                }
                ++p;
              }
            }
          }
          wc += __popc(b0) + __popc(b1) + __popc(b2) + __popc(b3);
        }
        *reinterpret_cast<float4*>(T.residual + e0 + j * 128) = make_float4(x[0], x[1], x[2], x[3]);
      }
    } else if (base < hi && base + kEmitTile > lo) {   // tile cut by the scope (or by the end of the vector)
#pragma unroll 1
      for (int j = 0; j < 4; ++j) {
        float x[4] = {0.f, 0.f, 0.f, 0.f};
        uint32_t f = 0, in = 0;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const uint64_t e = base + toff + j * 128 + c;
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
                if (p < kStash) {
                  stash[p].idx = (uint32_t)(base + toff + j * 128 + c);
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
          if (in & (1u << c)) T.residual[base + toff + j * 128 + c] = x[c];
      }
    }
    fill += wc;
    if (lane == 0) s_cnt[i * kEmitWarps + warp] = wc;
  }
  __syncthreads();

  // ---- scan: counts -> exclusive offsets inside the chunk, then one look-back for the chunk
  if (warp == 0) {
    uint32_t a[PER], sum = 0;
#pragma unroll
    for (int p = 0; p < PER; ++p) {
      const int e = (int)lane * PER + p;
      a[p] = e < E ? s_cnt[e] : 0u;
      sum += a[p];
    }
    uint32_t inc = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xFFFFFFFFu, inc, o);
      if ((int)lane >= o) inc += y;
    }
    uint32_t run = inc - sum;
#pragma unroll
    for (int p = 0; p < PER; ++p) {
      const int e = (int)lane * PER + p;
      if (e < E) s_off[e] = run;
      run += a[p];
    }
    const uint32_t total = __shfl_sync(0xFFFFFFFFu, inc, 31);
    uint64_t ex_a, ex_b;
    const bool ok = tile_lookback(reinterpret_cast<uint4*>(T.desc_emit), t, first, total, 0, ex_a, ex_b, T.ctl);
    if (lane == 0) { s_excl = ex_a; s_total = total; s_ok = ok ? 1 : 0; }
  }
  __syncthreads();
  if (!s_ok) return;
  const uint64_t excl = s_excl;

  // ---- phase B: this warp's candidates go to their final positions
  if (fill) {
    const uint64_t cap = d.cand_cap;
    uint32_t* cidx = T.cand_idx + d.cand_base;
    float* cval = T.cand_val + d.cand_base;
    if (fill <= kStash) {
      uint32_t a = 0;                        // first stash entry of tile i
#pragma unroll 1
      for (int i = 0; i < CT; ++i) {
        const uint32_t c = s_cnt[i * kEmitWarps + warp];
        const uint64_t dst = excl + s_off[i * kEmitWarps + warp];
        for (uint32_t e = lane; e < c; e += 32) {
          const uint64_t pos = dst + e;
          if (pos < cap) {
            cidx[pos] = stash[a + e].idx;
            cval[pos] = stash[a + e].val;
          } else if ((__float_as_uint(stash[a + e].val) & kAbsMask) >= zmin) {
            // the list is full (the scope will be selected densely): the slot must hold v again
            T.residual[stash[a + e].idx] = stash[a + e].val;
            T.state[s].early_bad = 1u;
          }
        }
        a += c;
      }
    } else {
      // more candidates than the stash holds: read this warp's elements back.  They are v, once the
      // slots that were cleared early (all of them are in the stash) hold v again; every entry at or above zmin
      // is cleared (again) as it goes to the list.
      if (zmin != 0xFFFFFFFFu) {
        for (uint32_t e = lane; e < kStash; e += 32)
          if ((__float_as_uint(stash[e].val) & kAbsMask) >= zmin) T.residual[stash[e].idx] = stash[e].val;
        __syncwarp();
      }
#pragma unroll 1
      for (int i = 0; i < CT; ++i) {
        if (s_cnt[i * kEmitWarps + warp] == 0u) continue;
        uint64_t run = excl + s_off[i * kEmitWarps + warp];
        const uint64_t base = cbase + (uint64_t)i * kEmitTile;
#pragma unroll 1
        for (int j = 0; j < 4; ++j) {
          float x[4] = {0.f, 0.f, 0.f, 0.f};
          uint32_t f = 0;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const uint64_t e = base + toff + j * 128 + c;
            if (e >= lo && e < hi) {
              x[c] = __ldcg(T.residual + e);   // from L2: other lanes may just have put v back
              f |= ((__float_as_uint(x[c]) & kAbsMask) >= tau_lo ? 1u : 0u) << c;
            }
          }
          const uint32_t b0 = __ballot_sync(0xFFFFFFFFu, f & 1u), b1 = __ballot_sync(0xFFFFFFFFu, f & 2u);
          const uint32_t b2 = __ballot_sync(0xFFFFFFFFu, f & 4u), b3 = __ballot_sync(0xFFFFFFFFu, f & 8u);
          if (f) {
            uint64_t pos = run + __popc(b0 & ltm) + __popc(b1 & ltm) + __popc(b2 & ltm) + __popc(b3 & ltm);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              if (f & (1u << c)) {
                if (pos < cap) {
                  cidx[pos] = (uint32_t)(base + toff + j * 128 + c);
                  cval[pos] = x[c];
                  if ((__float_as_uint(x[c]) & kAbsMask) >= zmin) T.residual[base + toff + j * 128 + c] = 0.0f;
                }
                ++pos;
              }
            }
          }
          run += __popc(b0) + __popc(b1) + __popc(b2) + __popc(b3);
        }
      }
    }
  }
  if (tid == 0 && lt == nchunks - 1) {
    const uint64_t m = excl + s_total;
    T.state[s].cand_count = m;
    if (sampled) {
      if (m > d.cand_cap) atomicCAS(&T.ctl->status, (int)GD_OK, (int)GD_ERR_OVERFLOW);
    } else if (!(T.flags & GD_FLAG_NO_PREDICTION) && (m < d.k || m > d.cand_cap)) {
      atomicAdd(&T.ctl->dense_needed, 1u);
    }
  }
}

}  // namespace

cudaError_t launch_add_emit(const DevTables& T, const uint32_t* tiles, cudaStream_t stream, const EmitEarly* early) {
  if (!tiles[L_EMIT]) return cudaSuccess;
  ProfileScope prof(stream, PT_ADD_EMIT);
#ifndef GD_NO_EMIT_PIPE
  if (add_emit_pipe_takes(T)) {
    cudaError_t e = launch_add_emit_pipe(T, tiles, stream, early);
    if (e != cudaSuccess) return e;
    note_launches(1);
    return cudaSuccess;
  }
#endif
  switch (T.emit_chunk_tiles) {
    case 1: add_emit_kernel<1><<<tiles[L_EMIT], kEmitThreads, 0, stream>>>(T); break;
    case 2: add_emit_kernel<2><<<tiles[L_EMIT], kEmitThreads, 0, stream>>>(T); break;
    case 4: add_emit_kernel<4><<<tiles[L_EMIT], kEmitThreads, 0, stream>>>(T); break;
    default: add_emit_kernel<8><<<tiles[L_EMIT], kEmitThreads, 0, stream>>>(T); break;
  }
  GD_LAUNCH_CHECK();
  return cudaSuccess;
}

}  // namespace gd
