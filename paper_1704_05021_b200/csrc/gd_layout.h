// Plain declarations shared by the host-side planner and the kernels of libgd.so: sizes, the per-call tables and
// the control structures of the workspace.  No CUDA types: the planner is also built and tested by itself with
// the host compiler's sanitizers.  Internal to libgd.so; the public interface is include/gd.h.
#pragma once

#include <stddef.h>
#include <stdint.h>

#include "gd.h"

namespace gd {

constexpr int kThreads = 256;           // threads per CTA in every tiled kernel
constexpr int kWarps = kThreads / 32;
constexpr uint32_t kTile = 4096;        // elements per tile of the streaming kernels
constexpr uint32_t kDenseSelTileMax = 32768;  // most elements per tile in the dense histogram passes
constexpr uint32_t kDenseChunkTilesMax = 16;  // most tiles per ticket (and per look-back) in the dense compaction
constexpr int kRadixBits0 = 11;         // 31-bit magnitude key = 11 + 10 + 10 bits
constexpr int kRadixBins0 = 1 << kRadixBits0;
constexpr int kShift0 = 20, kShift1 = 10, kShift2 = 0;
constexpr uint32_t kHistBinsPerScope = 2 * (2048 + 1024 + 1024);   // three passes over the sample, three over the list
// The selection among the candidates of the fused pass first counts them in a histogram of D = key - base (base: the
// smallest key a candidate can have): 2047 bins of 2^kFineShift keys each, and a last bin for everything further up.
// The threshold is usually a few per cent above the base, i.e. inside the fine bins, and one more 11-bit pass finds it.
constexpr int kFineShift = 11;
constexpr uint32_t kFineBins = 2048, kFineTop = kFineBins - 1u;
constexpr uint32_t kAbsMask = 0x7FFFFFFFu;
constexpr uint32_t kLookbackSpinLimit = 1u << 21;  // a device-side wait gives up after this many polls ...
constexpr uint64_t kWaitBudgetNs = 2000000000ull;  // ... AND this much time (whichever comes later): on a GPU that is
                                                   // shared by time slices a poll count alone can run out while the
                                                   // CTA waited on is merely descheduled
constexpr uint64_t kInlineMeansPairs = 2048;       // up to this many pairs the finishing CTA divides the sums itself

// Kinds of tiled launches; each has its own tile -> scope table.
enum Launch : int { L_EMIT = 0, L_SAMP = 1, L_CAND = 2, L_DSEL = 3, L_DCOMP = 4, L_COUNT = 5 };
// Views a selection can run over.
enum View : int { V_SAMPLE = 0, V_CAND = 1, V_DENSE = 2 };

// Look-back descriptor flags (low two bits of a 64-bit word; the count sits above them).
enum : uint64_t { F_INVALID = 0, F_AGG = 1, F_PREFIX = 2, F_ABORT = 3 };

struct ScopeDesc {       // built on the host for every call, read-only on the device
  uint64_t lo, hi;       // element range [lo, hi) of the scope in the flat gradient
  uint64_t k;            // entries kept
  uint64_t out_base;     // first slot of the scope in out_idx / out_val
  uint64_t cand_base;    // first slot of the scope in the candidate buffers
  uint64_t cand_cap;     // slots reserved for the scope's candidates
  uint64_t samp_base;    // first slot of the scope in the sample buffer
  uint64_t samp_m;       // samples drawn from the scope
  uint64_t samp_rank;    // the prediction is the samp_rank-th largest sample key
  uint64_t samp_w;       // floor(n_s / samp_m): width of a stratum (the first samp_rem strata are one wider)
  uint32_t samp_rem;     // n_s mod samp_m
  uint32_t samp_cluster; // 1: strata of elements, one sample each.  8 (narrow strata) or 2 (wide ones): the prediction
                         // samples whole groups of that many consecutive elements (one 32-byte sector of each input);
                         // the strata (samp_w, samp_rem) then count groups, from the first multiple of it at or after lo
};

struct ScopeState {      // zeroed at the start of every call
  uint64_t cand_count;   // candidates the fused pass counted (may exceed cand_cap)
  uint32_t tau_lo;       // predicted lower bound of the threshold key
  uint32_t tau;          // threshold key: smallest kept |v| bit pattern
  uint64_t q;            // ties at tau that are kept (the lowest indices)
  uint64_t gt;           // entries with key > tau
  uint32_t tau_hi;       // the sample's estimate of tau itself: the fused pass writes +0 instead of v into the
                         // residual where key > tau_hi (these entries are almost surely kept; the compaction
                         // settles the few for which that is wrong, from the candidate list)
  uint32_t early_bad;    // set when some such entry could not be recorded (a full stash, a full list): the
                         // compaction then clears every kept slot itself
  uint32_t used_dense;   // 1 if the dense path produced this scope's result
  uint32_t top_bin_max;  // dense histogram pass: largest first digit (key >> 20) seen in the scope so far
};
static_assert(sizeof(ScopeState) == 48, "ScopeState is cleared and addressed in 16-byte units");

struct Ctl {             // zeroed at the start of every call
  int32_t status;
  uint32_t ticket[L_COUNT];
  uint32_t n_scopes;
  uint32_t n_scopes_predicted;
  uint32_t n_scopes_dense;
  uint32_t dense_needed;   // scopes whose prediction failed (set by the fused pass)
  uint32_t barrier[3];     // grid barriers of the three selection kernels
  uint32_t compact_done[2];// CTAs of each compaction kernel that have finished
  uint32_t barrier_mid;    // grid barrier between a dense selection and a dense compaction run by one kernel
  uint64_t n_candidates;
  uint64_t n_kept;
  uint32_t generic_needed; // some scope's threshold lies beyond the fine bins of the candidates' first histogram
  uint32_t hist_redo;      // dense histogram pass: some scope's k-th largest key lay below the window that was counted
};

constexpr uint32_t kSmemScopes = 32;          // most scopes whose tables the kernels keep in shared memory
constexpr size_t kSetupBlobBytes = 6144;      // the small host-built tables of a call travel as a kernel argument of this size at most
                                              // (the tables of 32 scopes are 4.6 KB; kernel arguments beyond 4 KB need CUDA 12.1)
constexpr uint32_t kSelectCompactMaxGrid = 4096;   // most CTAs of the kernel that selects and compacts in one launch
constexpr uint32_t kStartMarks = 128;                 // most CTAs that clear the control region in the setup-and-predict launch
constexpr uint32_t kLocalSampleMax = 32768;        // most samples of one scope that the setup-and-predict launch handles

}  // namespace gd
