// All-cores restatement of the CPU oracle (Aji & Heafield 2017, Section 4, Algorithm 1).
//
// TEST INFRASTRUCTURE ONLY: used by the tests (where it is checked against the numpy oracle and
// against the same pins) and by the benchmark's cpu-baseline leg, never by the product.  It shares
// no code with the CUDA library.  It is the same definition as oracle/graddrop_oracle.py, taken in
// Algorithm 1's order, with the element-wise passes spread over the host cores (OpenMP) and the
// full sort done by the C++ library's parallel sort:
//
//   1. v = g + r                                   one fp32 add per element
//   2. per scope: sort (|v| bit pattern descending, index ascending); the first
//      k = n_s - floor(n_s * drop_ppm / 1e6) entries are kept; tau = the smallest kept key
//   3-5. survivors in ascending index as (index, value); residual = +0 where kept, v elsewhere
//   two-value quantisation (Section 5.4): per layer, mean of kept values by sign bit (fp64 sums)
//   shard split (Section 3): survivors below each shard boundary
//
// Build: g++ -O2 -fopenmp -shared -fPIC graddrop_oracle_par.cpp -o libgraddrop_oracle_par.so
#include <parallel/algorithm>
#include <omp.h>

#include <cstdint>
#include <cstring>
#include <functional>
#include <vector>

namespace {

inline uint32_t bits_of(float x) {
  uint32_t u;
  std::memcpy(&u, &x, 4);
  return u;
}

}  // namespace

extern "C" {

int oracle_par_threads() { return omp_get_max_threads(); }
// t > 0: use t threads from now on; t <= 0: as many as the process may run on.
void oracle_par_set_threads(int t) { omp_set_num_threads(t > 0 ? t : omp_get_num_procs()); }

// grad, residual_in: n floats (read).  residual_out: n floats (written).  layer_off: n_layers + 1,
// shard_off: n_shards + 1 ascending offsets from 0 to n.  scope_mode 0 = one threshold for the whole
// vector, 1 = one per layer.  value_mode 0 = fp32 values, 1 = two means per layer (out_idx carries
// the sign in bit 31, out_means gets n_layers pairs, out_val is still written).
// out_idx/out_val hold sum of k over scopes entries; out_tau one entry per scope;
// out_cnt_off n_shards + 1 entries.  Returns 0, or -1 on bad arguments.
int oracle_par_compress(const float* grad, const float* residual_in, float* residual_out, uint64_t n,
                        const uint64_t* layer_off, uint32_t n_layers, const uint64_t* shard_off, uint32_t n_shards,
                        uint32_t drop_ppm, int scope_mode, int value_mode, uint32_t* out_idx, float* out_val,
                        uint32_t* out_cnt_off, uint32_t* out_tau, float* out_means) {
  if (drop_ppm > 1000000u || n_layers == 0 || layer_off[0] != 0 || layer_off[n_layers] != n) return -1;
  if (n >= (1ull << 32) || (value_mode != 0 && value_mode != 1)) return -1;
  if (value_mode == 1 && n > (1ull << 31)) return -1;

  // step 1
  float* v = residual_out;
#pragma omp parallel for schedule(static)
  for (uint64_t i = 0; i < n; ++i) v[i] = grad[i] + residual_in[i];

  std::vector<uint8_t> kept(n, 0);
  const uint32_t n_scopes = scope_mode == 0 ? 1u : n_layers;
  uint64_t out_base = 0;
  std::vector<uint64_t> order;
  for (uint32_t s = 0; s < n_scopes; ++s) {
    const uint64_t lo = scope_mode == 0 ? 0 : layer_off[s];
    const uint64_t hi = scope_mode == 0 ? n : layer_off[s + 1];
    const uint64_t ns = hi - lo;
    const uint64_t k = ns - (uint64_t)(((unsigned __int128)ns * drop_ppm) / 1000000u);
    // step 2: a full sort of (key, index) composites; larger key first, lower index first among equals
    order.resize(ns);
#pragma omp parallel for schedule(static)
    for (uint64_t i = 0; i < ns; ++i) {
      const uint64_t key = bits_of(v[lo + i]) & 0x7FFFFFFFu;
      order[i] = (key << 32) | (0xFFFFFFFFull - i);
    }
    __gnu_parallel::sort(order.begin(), order.end(), std::greater<uint64_t>());
    out_tau[s] = k ? (uint32_t)(order[k - 1] >> 32) : 0xFFFFFFFFu;
#pragma omp parallel for schedule(static)
    for (uint64_t j = 0; j < k; ++j) kept[lo + (0xFFFFFFFFull - (order[j] & 0xFFFFFFFFull))] = 1;

    // steps 3-5: survivors in ascending index (per-thread counts, then per-thread fill)
    const int T = omp_get_max_threads();
    std::vector<uint64_t> start(T + 1, 0);
#pragma omp parallel num_threads(T)
    {
      const int t = omp_get_thread_num();
      const uint64_t a = lo + ns * t / T, b = lo + ns * (t + 1) / T;
      uint64_t c = 0;
      for (uint64_t i = a; i < b; ++i) c += kept[i];
      start[t + 1] = c;
#pragma omp barrier
#pragma omp single
      for (int u = 0; u < T; ++u) start[u + 1] += start[u];
      uint64_t o = out_base + start[t];
      for (uint64_t i = a; i < b; ++i) {
        if (kept[i]) {
          out_idx[o] = (uint32_t)i;
          out_val[o] = v[i];
          ++o;
        }
      }
    }
    out_base += k;
  }
  const uint64_t k_total = out_base;

  // two-value quantisation, before the residual rewrite destroys nothing it needs (values are in out_val)
  if (value_mode == 1) {
    for (uint32_t l = 0; l < n_layers; ++l) {
      double sp = 0.0, sn = 0.0;
      uint64_t cp = 0, cn = 0;
#pragma omp parallel for schedule(static) reduction(+ : sp, sn, cp, cn)
      for (uint64_t j = 0; j < k_total; ++j) {
        const uint64_t i = out_idx[j] & 0x7FFFFFFFu;
        if (i < layer_off[l] || i >= layer_off[l + 1]) continue;
        if (bits_of(out_val[j]) >> 31) { sn += (double)out_val[j]; ++cn; }
        else { sp += (double)out_val[j]; ++cp; }
      }
      out_means[2 * l] = cp ? (float)(sp / (double)cp) : 0.0f;
      out_means[2 * l + 1] = cn ? (float)(sn / (double)cn) : 0.0f;
    }
#pragma omp parallel for schedule(static)
    for (uint64_t j = 0; j < k_total; ++j) out_idx[j] |= (bits_of(out_val[j]) >> 31) << 31;
  }

  // step 4: the dropped mass stays
#pragma omp parallel for schedule(static)
  for (uint64_t i = 0; i < n; ++i)
    if (kept[i]) v[i] = 0.0f;

  // Section 3: one piece per server
  for (uint32_t h = 0; h <= n_shards; ++h) {
    uint64_t c = 0;
#pragma omp parallel for schedule(static) reduction(+ : c)
    for (uint64_t j = 0; j < k_total; ++j) c += ((uint64_t)(out_idx[j] & (value_mode ? 0x7FFFFFFFu : 0xFFFFFFFFu)) < shard_off[h]);
    out_cnt_off[h] = (uint32_t)c;
  }
  return 0;
}

// Server side (Section 3): p[idx] += alpha * value for one push over the flat parameter vector;
// value_mode 1 decodes a survivor as its layer's mean for its sign.  One fp32 fused multiply-add
// per survivor (indices inside a push are unique).
int oracle_par_apply(float* params, const uint32_t* idx, const float* val, uint64_t count, float alpha, int value_mode,
                     const float* means, const uint64_t* layer_off, uint32_t n_layers) {
#pragma omp parallel for schedule(static)
  for (uint64_t j = 0; j < count; ++j) {
    uint64_t i = idx[j];
    float x;
    if (value_mode == 0) {
      x = val[j];
    } else {
      const uint32_t sign = idx[j] >> 31;
      i &= 0x7FFFFFFFu;
      uint32_t l = 0;
      while (l + 1 < n_layers && layer_off[l + 1] <= i) ++l;
      x = means[2 * l + sign];
    }
    params[i] = __builtin_fmaf(alpha, x, params[i]);
  }
  return 0;
}

}  // extern "C"
