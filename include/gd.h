/*
 * gd.h - C ABI of the gradient-dropping library (libgd.so, CUDA, sm_100a).
 *
 * The library implements the hot path of "Sparse Communication for Distributed Gradient
 * Descent" (Aji & Heafield, EMNLP 2017): Algorithm 1 (GradDrop) on the worker side and the
 * decompress + scatter-add of sparse pushes on the server side (Section 3).
 *
 * Conventions
 *   - "device" pointers are CUDA device memory of the current device; "HOST" pointers are
 *     ordinary host memory that is read before the call returns.
 *   - A stream argument is a cudaStream_t passed as void* (NULL = the default stream).
 *   - Unless stated otherwise a call only enqueues work on the stream and returns; it never
 *     synchronises and never allocates or frees device memory.  All device buffers, the
 *     residual and the workspace included, are owned by the caller.
 *   - gd_compress keeps the plan it derives from a layout (offsets, drop ratio, scope mode) in a small
 *     per-process cache, so that a training loop pays for it once.  For layouts whose tables do not fit
 *     a kernel argument (roughly more than thirty tensors) the cached plan holds a page-locked HOST
 *     image of the tables, allocated by the first call with that layout (make that call outside any
 *     stream capture); without it, and always in gd_compress_static, such tables travel in pieces
 *     as arguments of a few extra small launches.  Host memory is never copied from pageable buffers.
 *   - Every function returns a gd_status_t.  Argument errors are detected on the host before
 *     anything is enqueued.  Conditions detected on the device (a bounded wait that ran out,
 *     an inconsistent count) are written to a status word in the workspace and are returned
 *     by gd_status(); device code never traps, asserts or spins without a limit.  After such a
 *     status the outputs AND the residual of that call are undefined (the call updates the
 *     residual in place); a caller that wants to retry keeps its own copy of the residual.
 *   - gd_compress and gd_decompress_apply open an NVTX range of their own name, for profilers that
 *     show them; without such a tool attached the ranges cost nothing to speak of.
 *   - No CUDA headers are needed to include this file.
 */
#ifndef GD_H
#define GD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  GD_OK = 0,
  GD_ERR_INVALID_ARG = -1,    /* NULL / misaligned pointer, offsets not ascending, bad enum value */
  GD_ERR_TOO_LARGE = -2,      /* n beyond what uint32 indices (or 31-bit packed indices) can address */
  GD_ERR_WORKSPACE = -3,      /* workspace missing or smaller than gd_workspace_bytes() */
  GD_ERR_CUDA = -4,           /* a CUDA runtime call failed (launch, memset, copy) */
  GD_ERR_DEVICE_TIMEOUT = -5, /* a bounded device-side wait gave up; outputs of that call are invalid */
  GD_ERR_INTERNAL = -6,       /* device-side consistency check failed; outputs of that call are invalid */
  GD_ERR_OVERFLOW = -7        /* sampled-threshold mode: more survivors than gd_sampled_capacity(); outputs invalid */
} gd_status_t;

enum { GD_SCOPE_GLOBAL = 0, GD_SCOPE_PER_LAYER = 1 };
enum { GD_VALUES_FP32 = 0, GD_VALUES_TWO_MEANS = 1, GD_VALUES_THRESHOLD = 2, GD_VALUES_COLUMN_MEANS = 3 };

/* gd_compress_args.flags */
enum {
  GD_FLAG_NO_PREDICTION = 1u, /* do not predict the threshold from a sample: always select over the
                                 whole dense vector (same results, more memory traffic) */
  GD_FLAG_SAMPLED_THRESHOLD = 2u, /* the approximation of Section 4: the threshold is selected on a 0.1 %
                                 sample and every entry at or above it is kept (see gd_compress) */
  GD_FLAG_QUANT_ERROR_FEEDBACK = 4u, /* 1-bit value modes only (Section 5.4).  The paper does not say whether
                                 the error of the 1-bit quantisation is kept; Algorithm 1 keeps only the
                                 dropped mass, which is the default here.  With this flag the residual of a
                                 KEPT entry is v minus the fp32 value the receiver will decode for it (one
                                 fp32 subtraction), as in the error feedback of 1-bit SGD that Section 2
                                 describes, instead of +0; dropped entries are unchanged. */
  GD_FLAG_NO_EARLY_ZERO = 8u, /* an implementation switch with no effect on results (for tests and timing):
                                 by default the fused pass already writes +0 into the residual slots
                                 of the entries the sample predicts to be kept, and the compaction
                                 only settles the few for which the prediction was wrong; with this
                                 flag the compaction clears every kept slot itself. */
  GD_FLAG_PLAIN_RADIX = 16u,  /* another switch with no effect on results: the selection among the candidates
                                 normally starts from a histogram the fused pass has prepared and needs one
                                 more pass; with this flag it always runs its three plain radix passes, as it
                                 does by itself when a threshold lies far above its prediction. */
  GD_FLAG_PREDICT_ALWAYS = 32u /* a third: predict the threshold from a sample however short the vector is (by
                                 default short vectors are selected densely, which is faster there).  Not
                                 together with GD_FLAG_NO_PREDICTION. */
};

const char* gd_status_string(int status);

/*
 * Entries kept in one threshold scope of n_scope elements when drop_ppm parts per million are
 * dropped: k = n_scope - floor(n_scope * drop_ppm / 1e6), in 64-bit integers.
 * Algorithm 1, the threshold-selection step (a fraction R of the magnitudes lies below the threshold);
 * R is passed as an integer so that
 * every party computes the same count.  drop_ppm must be <= 1000000.
 */
int gd_kept_count(uint64_t n_scope, uint32_t drop_ppm, uint64_t* k_out);

/*
 * Total survivors of one gd_compress call, so that outputs can be sized before the launch.
 * layer_off: HOST, n_layers + 1 ascending offsets (first 0, last n).  Section 4, last paragraph:
 * the threshold is chosen for every parameter matrix on its own (GD_SCOPE_PER_LAYER: one scope per layer) or
 * globally (GD_SCOPE_GLOBAL: one scope [0, n)).
 */
int gd_total_kept(const uint64_t* layer_off, uint32_t n_layers, int scope_mode, uint32_t drop_ppm,
                  uint64_t* k_total_out);

/*
 * Size, in entries, that out_idx / out_val must have for GD_FLAG_SAMPLED_THRESHOLD, where the number of
 * survivors is not known in advance: per scope min(n_s, 4 k_s + 8192), summed.
 */
int gd_sampled_capacity(const uint64_t* layer_off, uint32_t n_layers, int scope_mode, uint32_t drop_ppm,
                        uint64_t* capacity_out);

/*
 * Bytes of device workspace gd_compress needs for these arguments (same meaning as in gd_compress_args).
 * layer_cols may be NULL unless GD_VALUES_COLUMN_MEANS will be used.
 */
int gd_workspace_bytes(const uint64_t* layer_off, uint32_t n_layers, const uint32_t* layer_cols, uint32_t n_shards,
                       int scope_mode, uint32_t drop_ppm, size_t* bytes_out);

/* Bytes of device workspace gd_decompress_apply needs. */
int gd_apply_workspace_bytes(uint32_t n_shards, uint32_t n_layers, size_t* bytes_out);

/*
 * Number of (mu+, mu-) pairs of a push: n_layers for GD_VALUES_TWO_MEANS and GD_VALUES_THRESHOLD, the
 * sum of layer_cols for GD_VALUES_COLUMN_MEANS, 0 for GD_VALUES_FP32.  out_means holds 2 floats per pair.
 */
int gd_means_pairs(uint32_t n_layers, const uint32_t* layer_cols, int value_mode, uint64_t* pairs_out);

/*
 * gd_compress - Algorithm 1 (GradDrop) for one worker's flat fp32 gradient.
 *
 *   v[i]      = grad[i] + residual[i]                  (one fp32 add, round to nearest, no flush to zero)
 *   per scope: keep exactly k entries, the largest by |v| (order: bit pattern of |v| descending,
 *              then index ascending); tau = smallest kept |v| bit pattern (0xFFFFFFFF if k = 0)
 *   out       = survivors of all scopes in ascending index: out_idx[t], out_val[t] = v[out_idx[t]]
 *   residual  = v where dropped, +0.0f where kept      (Algorithm 1: residuals <- grad - dropped)
 *   out_shard_cnt_off[j] = number of survivors with index < shard_off[j]   (Section 3: the
 *              gradient is split into N pieces, one per server)
 *   two-means mode (Section 5.4, the 1-bit quantisation whose two centres are the means of the values they replace): per
 *              layer, mu+ = mean of kept v with sign bit 0 and mu- = mean of kept v with sign bit 1
 *              (fp64 accumulation, rounded to fp32, +0.0f for an empty group); out_idx[t] carries
 *              index | signbit << 31 and out_val is not written.  The residual is unchanged by the
 *              value mode: it holds the dropped mass only.
 *   column-means mode (Section 5.4: the centres are chosen per column of a matrix instead of one pair
 *              per tensor): layer l is a row-major matrix with layer_cols[l] columns (its size must
 *              be a multiple of layer_cols[l]; 1 = one pair for the whole layer, as in two-means mode), and
 *              every column c gets its own pair: pair index = sum of layer_cols of the earlier layers + c,
 *              out_means[2 * pair] = mu+, out_means[2 * pair + 1] = mu-.  Packing as in two-means mode.
 *   threshold mode (Section 5.4, the quantisation in which every survivor stands for the dropping
 *              threshold, i.e. the smallest magnitude that survived): same packing as two-means
 *              mode; out_means[l] = (+t, -t) with t the float whose bit pattern is the tau of the scope
 *              that holds layer l (+0, -0 if that scope keeps nothing), so that a push decodes exactly
 *              like a two-means push.
 *
 *   delta mode (delta_base != NULL; Section 4, third paragraph: the same function is applied to
 *              parameter pulls, sent as differences from the version the client pulled last, of which
 *              the server keeps a copy): grad holds the server's current parameters,
 *              delta_base the copy the client is known to hold, and
 *                  v[i] = grad[i] - delta_base[i]          (one fp32 subtraction)
 *              takes the place of grad + residual; the residual's old contents are not read.  After the
 *              selection delta_base[i] <- delta_base[i] + v[i] (one fp32 add) for every survivor, which is
 *              exactly what gd_decompress_apply with alpha = 1 does to the client's copy, so the two
 *              copies stay equal bit for bit; what was dropped stays in the next delta by itself.  The
 *              residual buffer is used as scratch and returns v where dropped, +0 where kept.  Delta
 *              mode needs GD_VALUES_FP32.
 *
 *   sampled-threshold mode (GD_FLAG_SAMPLED_THRESHOLD; Section 4, fourth paragraph: the threshold is
 *              selected on a 0.1 % sample of the gradient instead of on all of it): a scope of up to 4096
 *              elements is sampled completely; a longer one in m = max(4096, ceil(n_s / 1000)) (rounded up
 *              to even) positions, taken as m / 2 pairs of neighbours (first + 2 j, first + 2 j + 1), first =
 *              the smallest even index >= the scope's start, j < P = floor((end - first) / 2).  The P pairs
 *              are cut into m / 2 strata (with w = floor(P / (m/2)) and rem = P mod (m/2), stratum i starts
 *              at pair a = i w + min(i, rem) and has w + 1 pairs if i < rem, else w); stratum i of scope s
 *              contributes pair a + (h mod width), h = mix(i * 0x9E3779B9 + s) in 32-bit arithmetic with
 *              mix(x): x ^= x >> 16; x *= 0x7FEB352D; x ^= x >> 15; x *= 0x846CA68B; x ^= x >> 16);
 *              the threshold key t is the (m - floor(m * drop_ppm / 1e6))-th largest sample key and EVERY
 *              entry of the scope with key >= t is kept, so the number of survivors varies: out_idx and
 *              out_val must hold gd_sampled_capacity() entries, the count is out_shard_cnt_off[n_shards],
 *              out_tau[s] = t, and a scope with more than min(n_s, 4 k_s + 8192) survivors makes the call
 *              end with GD_ERR_OVERFLOW in the status word.  Needs GD_VALUES_FP32.
 *
 * Results are bit-exact functions of (grad, residual, offsets, drop_ppm) except the two means,
 * whose fp64 partial sums are combined in an unspecified order.  Non-finite inputs are ordered by
 * their bit pattern (NaN above Inf above finite); NaN payloads follow the device's fp32 add.
 * grad, residual, the outputs and the workspace must not overlap.  Calls that share a workspace
 * must be ordered (same stream, or otherwise serialised).  Host threads may call concurrently with
 * workspaces of their own, but calls on ONE device should be ordered with respect to each other
 * (one stream, or events): the selection kernels are cooperative launches sized to fill the device,
 * so two calls that overlap on a GPU gain nothing and may end with GD_ERR_DEVICE_TIMEOUT when neither
 * grid becomes fully resident (every device-side wait is bounded; nothing hangs).
 */
typedef struct gd_compress_args {
  const float* grad;          /* device, n fp32, 16-byte aligned, read-only */
  float* residual;            /* device, n fp32, 16-byte aligned, in/out */
  uint64_t n;                 /* <= 2^32 (GD_VALUES_FP32) or <= 2^31 (the packed modes) */
  const uint64_t* layer_off;  /* HOST, n_layers + 1 ascending offsets, [0] = 0, last = n */
  uint32_t n_layers;          /* >= 1 */
  uint32_t n_shards;          /* >= 1 */
  const uint64_t* shard_off;  /* HOST, n_shards + 1 ascending offsets, [0] = 0, last = n */
  uint32_t drop_ppm;          /* 990000 = 99 %, 999000 = 99.9 % */
  int32_t scope_mode;         /* GD_SCOPE_* */
  int32_t value_mode;         /* GD_VALUES_* */
  uint32_t flags;             /* GD_FLAG_* */
  uint32_t* out_idx;          /* device, gd_total_kept() words (gd_sampled_capacity() in sampled-threshold mode) */
  float* out_val;             /* device, as many fp32; may be NULL in the packed modes */
  uint32_t* out_shard_cnt_off;/* device, n_shards + 1 words */
  uint32_t* out_tau;          /* device, one word per scope (1, or n_layers); may be NULL */
  float* out_means;           /* device, gd_means_pairs() x 2 fp32 (mu+, mu-); the packed modes */
  void* workspace;            /* device, 256-byte aligned, >= gd_workspace_bytes() */
  size_t workspace_bytes;
  float* delta_base;          /* device, n fp32, 16-byte aligned, in/out, or NULL (see "delta mode" above) */
  const uint32_t* layer_cols; /* HOST, n_layers column counts; GD_VALUES_COLUMN_MEANS only, else may be NULL */
} gd_compress_args;

int gd_compress(const gd_compress_args* args, void* stream);

/*
 * One sparse push as produced by gd_compress (all pointers device memory).  The entries that
 * are applied are [shard_cnt_off[0], shard_cnt_off[n_shards]) of idx / val, n_shards being the
 * shard count of the gd_apply_args the push is used with.  A server that owns one shard j passes
 * the worker's out_shard_cnt_off + j.
 */
typedef struct gd_push {
  const uint32_t* idx;
  const float* val;              /* NULL in the packed modes */
  const uint32_t* shard_cnt_off;
  const float* means;            /* gd_means_pairs() x 2, packed modes only */
} gd_push;

/*
 * gd_decompress_apply - the server side of Section 3: each server owns 1/N of the parameters
 * and adds the pushed pieces into it.  For every push in array order and every entry of it
 * whose index lies in a shard [shard_off[j], shard_off[j+1]):
 *     params[j][index - shard_off[j]] += alpha * value
 * with value = val[t] (fp32 mode) or means[pair of the entry][sign] (the packed modes; the pair is the
 * entry's layer, or its layer and column in column-means mode).
 * One fused multiply-add in fp32 per entry; with alpha = 1 the result is fl32(p + value).
 * Pushes are applied one after another in stream order (unless GD_APPLY_ATOMIC is set); indices inside one push are unique.
 * Entries whose index lies outside every shard are skipped.  The optimiser is not part of
 * this library.
 */
/* gd_apply_args.flags */
enum {
  GD_APPLY_ATOMIC = 1u /* Section 3 has every server receive a piece from every worker.  By default the pushes of a
                          call are applied one after another (one launch each, array order).  With this flag all of
                          them are applied by one launch and entries of different pushes that meet in one parameter
                          are combined with atomic read-modify-writes, in no defined order: every entry still lands
                          exactly once as one fused multiply-add (subnormals kept), so the result differs from the
                          ordered one by the rounding of a different summation order only. */
};

typedef struct gd_apply_args {
  float* const* params;        /* HOST array of n_shards device pointers */
  const uint64_t* shard_off;   /* HOST, n_shards + 1 ascending global offsets */
  uint32_t n_shards;
  uint32_t n_pushes;
  const gd_push* pushes;       /* HOST array of n_pushes */
  int32_t value_mode;          /* GD_VALUES_* */
  float alpha;
  const uint64_t* layer_off;   /* HOST, n_layers + 1; packed modes only */
  uint32_t n_layers;
  uint32_t flags;              /* GD_APPLY_* (0: pushes applied one after another) */
  void* workspace;             /* device, 256-byte aligned, >= gd_apply_workspace_bytes() */
  size_t workspace_bytes;
  const uint32_t* layer_cols;  /* HOST, n_layers column counts; GD_VALUES_COLUMN_MEANS only, else may be NULL */
} gd_apply_args;

int gd_decompress_apply(const gd_apply_args* args, void* stream);

/* residual <- +0.0f: the state before the first step, when nothing has been dropped yet (Section 4). */
int gd_residual_reset(float* residual, uint64_t n, void* stream);

/*
 * Synchronises the stream and returns the device status word the last gd_compress left in this
 * workspace (GD_OK, GD_ERR_DEVICE_TIMEOUT or GD_ERR_INTERNAL), or GD_ERR_CUDA.
 */
int gd_status(const void* workspace, void* stream);

/* Diagnostics of the last gd_compress on this workspace (synchronises the stream). */
typedef struct gd_stats {
  int32_t status;
  uint32_t n_scopes;
  uint32_t n_scopes_predicted;  /* scopes whose threshold was found from the predicted candidate list */
  uint32_t n_scopes_dense;      /* scopes that needed selection over the whole dense range */
  uint64_t n_candidates;        /* candidates emitted by the fused pass, over all scopes */
  uint64_t n_kept;              /* survivors written */
} gd_stats;

int gd_get_stats(const void* workspace, void* stream, gd_stats* out);

/*
 * gd_step_host - one whole step for a caller whose gradient lives in host memory: copies grad_host
 * to the device buffer args->grad, runs gd_compress and then gd_decompress_apply (apply may be
 * NULL), and copies the push (indices, values or means, shard offsets) back to the host buffers.
 * Synchronises the stream before returning.  Host buffers should be page-locked for full copy
 * bandwidth.  gd_total_kept() entries (gd_sampled_capacity() with GD_FLAG_SAMPLED_THRESHOLD) are copied to
 * idx_host / val_host.
 */
typedef struct gd_host_io {
  const float* grad_host;        /* HOST, n fp32 */
  uint32_t* idx_host;            /* HOST, k_total words, or NULL */
  float* val_host;               /* HOST, k_total fp32, or NULL */
  uint32_t* shard_cnt_off_host;  /* HOST, n_shards + 1 words, or NULL */
  float* means_host;             /* HOST, n_layers x 2 fp32, or NULL */
} gd_host_io;

int gd_step_host(const gd_compress_args* args, const gd_apply_args* apply, const gd_host_io* io, void* stream);

/*
 * gd_compress_static - gd_compress for callers that cannot hand the library a workspace.
 * (No counterpart in the paper: this is a packaging variant of gd_compress.)
 *
 * Some hosts of this library run inside a memory plan that is fixed before the first step - an
 * inference or training runtime that has already carved up the whole device, a plug-in called from
 * a context where cudaMalloc is forbidden or would synchronise the device, a pre-sized arena whose
 * owner will not grow it.  Such a caller can still provide the gradient, the residual and the
 * output buffers, because those are part of its own plan, but it has nowhere to put the scratch
 * memory gd_compress wants.  For them the library carries a fixed scratch area of
 * GD_STATIC_WORKSPACE_BYTES inside its own device image, and this entry point uses it in place of
 * args->workspace (args->workspace and args->workspace_bytes are ignored).  Everything else -
 * arguments, results, error codes - is exactly gd_compress.
 *
 * Limits and rules:
 *   - the scratch is part of the loaded library: every GPU that loads libgd.so gives up
 *     GD_STATIC_WORKSPACE_BYTES of device memory until the process exits, used or not;
 *   - a call whose gd_workspace_bytes() exceeds GD_STATIC_WORKSPACE_BYTES is refused with
 *     GD_ERR_TOO_LARGE before anything is enqueued (as a guide: one flat scope of 2^24 elements at a
 *     99 % drop ratio needs about 5.4 MiB, 2^25 elements about 10.6 MiB);
 *   - the first call on each device looks up the scratch area's device address (once per device, with
 *     that device current); make that first call outside any stream capture;
 *   - no device memory is allocated or freed, here or in anything this entry point calls;
 *   - all calls on one device share the one scratch area.  Each call clears the part that must
 *     start at zero, but two calls that overlap on the GPU (different streams, no ordering between
 *     them) would race on it: keep calls on one device ordered;
 *   - *workspace_out (if workspace_out is not NULL) receives the scratch area's device address, the
 *     value to pass to gd_status() and gd_get_stats() after the call.
 */
#define GD_STATIC_WORKSPACE_BYTES (16u << 20)
int gd_compress_static(const gd_compress_args* args, void* stream, const void** workspace_out);

/*
 * Measurement hooks (no counterpart in the paper).  gd_profile_enable(1) makes every gd_compress
 * record a pair of CUDA events on its stream around the fused full pass (the kernel that streams
 * the dense gradient and residual once: tag 2 below, or 16 where a short vector takes one launch for
 * everything); gd_profile_enable(2) brackets every kernel the library
 * launches; 0 switches the hooks off.  gd_profile_collect waits for the recorded pairs, writes their
 * durations in milliseconds (oldest first, at most `capacity`) and, if tags_out is not NULL, which
 * kernel each belongs to (0 setup, 1 sample selection, 2 fused pass, 3 dense selection, 4 dense
 * compaction, 5 candidate selection, 6 candidate compaction, 7 finalize, 8 apply, 9 sampled-mode pack,
 * 10 means division, 11 quantisation-error feedback, 12 candidate selection and compaction in one launch,
 * 13 setup and prediction in one launch, 14 dense histogram pass, 15 walk of the dense histogram,
 * 16 add, selection and compaction of a short vector in one launch), then forgets them.
 * At most 4096 pairs are held between two collects; later launches are not recorded.  Not thread-safe.
 */
int gd_profile_enable(int mode);
int gd_profile_collect(float* ms_out, uint32_t* tags_out, uint32_t capacity, uint32_t* count_out);

/*
 * Self-test of the bounded device-side waits (no counterpart in the paper).  Every wait in the
 * library's kernels - on a predecessor tile of a scan, on a grid barrier, on the mbarrier of a
 * pipeline stage - gives up after a fixed number of polls or a fixed time, marks its tile aborted so
 * that nothing waits on it, and records GD_ERR_DEVICE_TIMEOUT in the workspace.  This call enqueues a
 * one-warp kernel that waits, for at most spin_limit polls, on a tile nothing will ever publish, and
 * then lets a second tile meet the aborted one; and a second one-warp kernel that waits, for at most
 * 100 ns x spin_limit, on an mbarrier at which nothing arrives.  Afterwards gd_status(workspace) is
 * GD_ERR_DEVICE_TIMEOUT and gd_get_stats reports n_scopes = 1 if the first wait gave up (as it must),
 * n_scopes_predicted = 1 if the second tile aborted without waiting, and n_kept = 1 if the wait on
 * the mbarrier gave up.  The context stays usable.  workspace: device, 256-byte aligned, >= 512 bytes.
 */
int gd_selftest_bounded_wait(void* workspace, size_t workspace_bytes, uint32_t spin_limit, void* stream);

/* Number of kernels this library has launched in this process (memsets and copies not counted). */
int gd_launch_count(uint64_t* count_out);

#ifdef __cplusplus
}
#endif
#endif /* GD_H */
