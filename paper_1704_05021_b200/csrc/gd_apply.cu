// gd_decompress_apply: the server side of the parameter-sharded exchange (Section 3 of Aji &
// Heafield 2017).  Each push is a list of (index, value) survivors; every entry is routed to the
// shard that owns its index and added to that shard's parameters.
#include <cstring>
#include <new>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "gd_internal.cuh"

namespace gd {

namespace {

constexpr size_t kAlignA = 256;
inline size_t align_up_a(size_t x) { return (x + kAlignA - 1) / kAlignA * kAlignA; }

struct ApplyDev {
  float* const* params;        // [n_shards] device pointers
  const uint64_t* shard_off;   // [n_shards + 1]
  const uint64_t* layer_off;   // [n_layers + 1] (packed modes)
  const uint64_t* pair_off;    // [n_layers + 1]
  const uint32_t* layer_cols;  // [n_layers]
  uint32_t n_shards, n_layers;
  int32_t value_mode;
  float alpha;
  const uint32_t* idx;
  const float* val;
  const uint32_t* cnt_off;
  const float* means;
};

// Small shard / layer tables travel as a kernel argument (no copy to the device is needed then).
constexpr uint32_t kInlineShards = 32, kInlineLayers = 64;
struct ApplyInline {
  float* params[kInlineShards];
  uint64_t shard_off[kInlineShards + 1];
  uint64_t layer_off[kInlineLayers + 1];
  uint64_t pair_off[kInlineLayers + 1];
  uint32_t layer_cols[kInlineLayers];
};

// Segmented scatter-add: the entries [cnt_off[0], cnt_off[n_shards]) of one push, in a grid-stride
// loop.  Indices inside one push are unique, so a plain read-modify-write is enough; pushes are
// separate launches in stream order.
template <bool INLINE>
__global__ void __launch_bounds__(kThreads) apply_kernel(const __grid_constant__ ApplyDev A,
                                                         const __grid_constant__ ApplyInline I) {
  float* const* params = INLINE ? I.params : A.params;
  const uint64_t* shard_off = INLINE ? I.shard_off : A.shard_off;
  const uint64_t* layer_off = INLINE ? I.layer_off : A.layer_off;
  const uint64_t* pair_off = INLINE ? I.pair_off : A.pair_off;
  const uint32_t* layer_cols = INLINE ? I.layer_cols : A.layer_cols;
  pdl_trigger();   // (the start of the next call may be brought onto the GPU behind this kernel)
  pdl_wait();      // nothing of the kernels before this one - the push, parameters another push has just updated - is read above
  const uint64_t begin = A.cnt_off[0], end = A.cnt_off[A.n_shards];
  const uint64_t lo_all = shard_off[0], hi_all = shard_off[A.n_shards];
  // Each thread takes kBatch entries at a time, a grid-stride apart, and has all their loads in flight before the
  // first add: the scattered reads of the parameters are bound by memory latency, not by bandwidth.  Indices
  // inside a push are unique, so the entries of a batch never touch the same parameter.
  constexpr int kBatch = 4;
  const uint64_t stride = (uint64_t)gridDim.x * kThreads;
  for (uint64_t p0 = begin + (uint64_t)blockIdx.x * kThreads + threadIdx.x; p0 < end; p0 += stride * kBatch) {
    uint32_t w[kBatch];
    float x[kBatch], old[kBatch];
    float* dst[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const uint64_t p = p0 + (uint64_t)u * stride;
      w[u] = p < end ? __ldcs(A.idx + p) : 0xFFFFFFFFu;
      x[u] = (p < end && A.value_mode == GD_VALUES_FP32) ? __ldcs(A.val + p) : 0.0f;
    }
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const uint64_t p = p0 + (uint64_t)u * stride;
      dst[u] = nullptr;
      if (p >= end) continue;
      uint64_t pos = w[u];
      if (A.value_mode != GD_VALUES_FP32) {
        pos = w[u] & kAbsMask;
        const uint64_t pr = pair_of(layer_off, pair_off, layer_cols, A.n_layers, pos);
        x[u] = __ldg(A.means + 2 * pr + (w[u] >> 31));
      }
      if (pos < lo_all || pos >= hi_all) continue;
      const uint32_t j = range_of(shard_off, A.n_shards, pos);
      dst[u] = params[j] + (pos - shard_off[j]);
      // One scattered 4-byte read-modify-write per survivor, bound by the rate of random DRAM accesses.  Asking
      // L2 to fetch 64 bytes around the miss instead of its default measured 12 % faster; red.global.add.f32
      // is as fast but flushes subnormals, which would break bit-exactness.
      asm volatile("ld.global.cg.L2::64B.f32 %0, [%1];" : "=f"(old[u]) : "l"(dst[u]) : "memory");
    }
#pragma unroll
    for (int u = 0; u < kBatch; ++u)
      if (dst[u]) __stcg(dst[u], __fmaf_rn(A.alpha, x[u], old[u]));
  }
}

// Up to kPushSet pushes applied by ONE launch (blockIdx.y = push).  Entries of different pushes may hit the same
// parameter, so every update is an atomic read-modify-write: a compare-and-swap loop around the same fused
// multiply-add as above (atom.global.add.f32 would be shorter but flushes subnormals, and it would round alpha * x
// before the add).  The order in which colliding pushes land is not defined; each lands exactly once.
constexpr uint32_t kPushSet = 32;
struct PushSet {
  const uint32_t* idx[kPushSet];
  const float* val[kPushSet];
  const uint32_t* cnt_off[kPushSet];
  const float* means[kPushSet];
};

template <bool INLINE>
__global__ void __launch_bounds__(kThreads) apply_atomic_kernel(const __grid_constant__ ApplyDev A,
                                                                const __grid_constant__ ApplyInline I,
                                                                const __grid_constant__ PushSet P) {
  float* const* params = INLINE ? I.params : A.params;
  const uint64_t* shard_off = INLINE ? I.shard_off : A.shard_off;
  const uint64_t* layer_off = INLINE ? I.layer_off : A.layer_off;
  const uint64_t* pair_off = INLINE ? I.pair_off : A.pair_off;
  const uint32_t* layer_cols = INLINE ? I.layer_cols : A.layer_cols;
  const uint32_t w = blockIdx.y;
  const uint32_t* idx = P.idx[w];
  const float* val = P.val[w];
  const float* means = P.means[w];
  const uint64_t begin = P.cnt_off[w][0], end = P.cnt_off[w][A.n_shards];
  const uint64_t lo_all = shard_off[0], hi_all = shard_off[A.n_shards];
  const uint64_t stride = (uint64_t)gridDim.x * kThreads;
  for (uint64_t p = begin + (uint64_t)blockIdx.x * kThreads + threadIdx.x; p < end; p += stride) {
    const uint32_t word = __ldcs(idx + p);
    uint64_t pos = word;
    float x;
    if (A.value_mode != GD_VALUES_FP32) {
      pos = word & kAbsMask;
      const uint64_t pr = pair_of(layer_off, pair_off, layer_cols, A.n_layers, pos);
      x = __ldg(means + 2 * pr + (word >> 31));
    } else {
      x = __ldcs(val + p);
    }
    if (pos < lo_all || pos >= hi_all) continue;
    const uint32_t j = range_of(shard_off, A.n_shards, pos);
    unsigned int* dst = reinterpret_cast<unsigned int*>(params[j] + (pos - shard_off[j]));
    unsigned int old = __ldcg(dst), assumed;
    do {   // (a retry means that another push's entry landed in between: at most one per colliding push)
      assumed = old;
      old = atomicCAS(dst, assumed, __float_as_uint(__fmaf_rn(A.alpha, x, __uint_as_float(assumed))));
    } while (old != assumed);
  }
}

}  // namespace

}  // namespace gd

using namespace gd;

extern "C" {

int gd_apply_workspace_bytes(uint32_t n_shards, uint32_t n_layers, size_t* bytes_out) {
  if (!bytes_out || n_shards == 0) return GD_ERR_INVALID_ARG;
  size_t b = align_up_a(sizeof(float*) * (size_t)n_shards);
  b += align_up_a(sizeof(uint64_t) * ((size_t)n_shards + 1));
  b += 2 * align_up_a(sizeof(uint64_t) * ((size_t)n_layers + 1));   // layer offsets, pair offsets
  b += align_up_a(sizeof(uint32_t) * ((size_t)n_layers + 1));        // columns per layer
  *bytes_out = b;
  return GD_OK;
}

int gd_decompress_apply(const gd_apply_args* a, void* stream_v) {
  nvtxRangePushA("gd_decompress_apply");
  struct Pop { ~Pop() { nvtxRangePop(); } } pop_on_return;
  if (!a || !a->params || !a->shard_off || a->n_shards == 0) return GD_ERR_INVALID_ARG;
  if (a->n_pushes && !a->pushes) return GD_ERR_INVALID_ARG;
  if (a->value_mode < GD_VALUES_FP32 || a->value_mode > GD_VALUES_COLUMN_MEANS) return GD_ERR_INVALID_ARG;
  if (a->value_mode == GD_VALUES_COLUMN_MEANS && !a->layer_cols) return GD_ERR_INVALID_ARG;
  if (a->flags & ~(uint32_t)GD_APPLY_ATOMIC) return GD_ERR_INVALID_ARG;
  const bool two_means = a->value_mode != GD_VALUES_FP32;   // the packed modes decode through the means table
  if (two_means && (!a->layer_off || a->n_layers == 0)) return GD_ERR_INVALID_ARG;
  for (uint32_t j = 0; j < a->n_shards; ++j) {
    if (a->shard_off[j + 1] < a->shard_off[j]) return GD_ERR_INVALID_ARG;
    if (a->shard_off[j + 1] > a->shard_off[j] && !a->params[j]) return GD_ERR_INVALID_ARG;
  }
  if (a->shard_off[a->n_shards] > (1ull << 32)) return GD_ERR_TOO_LARGE;
  if (two_means)
    for (uint32_t l = 0; l < a->n_layers; ++l)
      if (a->layer_off[l + 1] < a->layer_off[l]) return GD_ERR_INVALID_ARG;
  for (uint32_t w = 0; w < a->n_pushes; ++w) {
    const gd_push& p = a->pushes[w];
    if (!p.idx || !p.shard_cnt_off) return GD_ERR_INVALID_ARG;
    if (two_means ? !p.means : !p.val) return GD_ERR_INVALID_ARG;
  }
  const uint32_t n_layers = two_means ? a->n_layers : 0;
  size_t need = 0;
  gd_apply_workspace_bytes(a->n_shards, n_layers, &need);
  if (!a->workspace || ((uintptr_t)a->workspace & (kAlignA - 1)) || a->workspace_bytes < need) return GD_ERR_WORKSPACE;
  if (a->n_pushes == 0) return GD_OK;
  cudaStream_t stream = (cudaStream_t)stream_v;
  try {
    const size_t o_params = 0;
    const size_t o_shard = align_up_a(sizeof(float*) * (size_t)a->n_shards);
    const size_t o_layer = o_shard + align_up_a(sizeof(uint64_t) * ((size_t)a->n_shards + 1));
    const size_t o_pair = o_layer + align_up_a(sizeof(uint64_t) * ((size_t)n_layers + 1));
    const size_t o_cols = o_pair + align_up_a(sizeof(uint64_t) * ((size_t)n_layers + 1));
    unsigned char* ws = (unsigned char*)a->workspace;
    // pairs: one per layer, or one per column of every layer (column-means mode)
    std::vector<uint64_t> pair_off((size_t)n_layers + 1, 0);
    std::vector<uint32_t> cols(n_layers, 1u);
    for (uint32_t l = 0; l < n_layers; ++l) {
      if (a->value_mode == GD_VALUES_COLUMN_MEANS) {
        cols[l] = a->layer_cols[l];
        if (cols[l] == 0 || ((a->layer_off[l + 1] - a->layer_off[l]) % cols[l]) != 0) return GD_ERR_INVALID_ARG;
      }
      pair_off[l + 1] = pair_off[l] + cols[l];
    }
    const bool use_inline = a->n_shards <= kInlineShards && n_layers <= kInlineLayers;
    ApplyInline I;
    std::memset(&I, 0, sizeof(I));
    if (use_inline) {
      std::memcpy(I.params, a->params, sizeof(float*) * (size_t)a->n_shards);
      std::memcpy(I.shard_off, a->shard_off, sizeof(uint64_t) * ((size_t)a->n_shards + 1));
      if (two_means) {
        std::memcpy(I.layer_off, a->layer_off, sizeof(uint64_t) * ((size_t)n_layers + 1));
        std::memcpy(I.pair_off, pair_off.data(), sizeof(uint64_t) * ((size_t)n_layers + 1));
        std::memcpy(I.layer_cols, cols.data(), sizeof(uint32_t) * (size_t)n_layers);
      }
    } else {
      std::vector<unsigned char> blob(need, 0);
      std::memcpy(blob.data() + o_params, a->params, sizeof(float*) * (size_t)a->n_shards);
      std::memcpy(blob.data() + o_shard, a->shard_off, sizeof(uint64_t) * ((size_t)a->n_shards + 1));
      if (two_means) {
        std::memcpy(blob.data() + o_layer, a->layer_off, sizeof(uint64_t) * ((size_t)n_layers + 1));
        std::memcpy(blob.data() + o_pair, pair_off.data(), sizeof(uint64_t) * ((size_t)n_layers + 1));
        std::memcpy(blob.data() + o_cols, cols.data(), sizeof(uint32_t) * (size_t)n_layers);
      }
      // (in pieces that travel as kernel arguments: a copy from this pageable vector would block the host)
      blob.resize((need + 15) / 16 * 16, 0);
      if (upload_by_launches(ws, blob.data(), blob.size(), stream) != cudaSuccess) return GD_ERR_CUDA;
    }
    ApplyDev A;
    std::memset(&A, 0, sizeof(A));
    A.params = (float* const*)(ws + o_params);
    A.shard_off = (const uint64_t*)(ws + o_shard);
    A.layer_off = (const uint64_t*)(ws + o_layer);
    A.pair_off = (const uint64_t*)(ws + o_pair);
    A.layer_cols = (const uint32_t*)(ws + o_cols);
    A.n_shards = a->n_shards;
    A.n_layers = n_layers;
    A.value_mode = a->value_mode;
    A.alpha = a->alpha;
    const unsigned grid = (unsigned)sm_count() * 8u;
    if (a->flags & GD_APPLY_ATOMIC) {
      // all pushes in one launch (sets of kPushSet, should there be more), colliding entries combined atomically
      for (uint32_t w0 = 0; w0 < a->n_pushes; w0 += kPushSet) {
        const uint32_t cnt = a->n_pushes - w0 < kPushSet ? a->n_pushes - w0 : kPushSet;
        PushSet P;
        std::memset(&P, 0, sizeof(P));
        for (uint32_t w = 0; w < cnt; ++w) {
          const gd_push& p = a->pushes[w0 + w];
          P.idx[w] = p.idx; P.val[w] = p.val; P.cnt_off[w] = p.shard_cnt_off; P.means[w] = p.means;
        }
        const unsigned per_push = grid / cnt > 0 ? (grid + cnt - 1) / cnt : 1u;
        ProfileScope prof(stream, PT_APPLY);
        if (use_inline)
          apply_atomic_kernel<true><<<dim3(per_push, cnt), kThreads, 0, stream>>>(A, I, P);
        else
          apply_atomic_kernel<false><<<dim3(per_push, cnt), kThreads, 0, stream>>>(A, I, P);
        if (cudaPeekAtLastError() != cudaSuccess) return GD_ERR_CUDA;
        note_launches(1);
      }
      return GD_OK;
    }
    for (uint32_t w = 0; w < a->n_pushes; ++w) {
      const gd_push& p = a->pushes[w];
      A.idx = p.idx;
      A.val = p.val;
      A.cnt_off = p.shard_cnt_off;
      A.means = p.means;
      ProfileScope prof(stream, PT_APPLY);
      const cudaError_t le = use_inline ? launch_dependent(apply_kernel<true>, dim3(grid), dim3(kThreads), 0, stream, A, I)
                                        : launch_dependent(apply_kernel<false>, dim3(grid), dim3(kThreads), 0, stream, A, I);
      if (le != cudaSuccess || cudaPeekAtLastError() != cudaSuccess) return GD_ERR_CUDA;
      note_launches(1);
    }
    return GD_OK;
  } catch (const std::bad_alloc&) {
    return GD_ERR_INVALID_ARG;
  }
}

}  // extern "C"
