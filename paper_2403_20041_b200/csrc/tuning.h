// Process-wide overrides of the launch heuristics, set through tl_e0m4_tuning_set (diagnostics
// and tests).  Every value is -1 unless a caller has set it, and -1 means "the library's own
// choice"; the launch paths read these atomics and never the environment.
#pragma once

#include <stdint.h>

namespace tl {

enum TuneKey {
  kTuneKsplit = 0,        // "ksplit": CTAs that share a tile along K in the tensor-core kernel (1..8)
  kTuneTcPair,            // "tc_pair": 0 / 1 = never / whenever the shape allows pairs of CTAs
  kTuneTcBig,             // "tc_big": 0 = rounds of 64 k even for small token tiles
  kTuneTcMtiles,          // "tc_mtiles": multiple (1, 2, 4, 8) of the fewest token tiles
  kTuneListPair,          // "list_pair": 0 / 1 = one-CTA / paired list kernel
  kTuneBatchTcMin,        // "batch_tc_min": first token count the tensor-core list kernel takes
  kTuneDecodeSplit,       // "decode_split": 1 = whole panels per CTA, 2 = stream-K ranges
  kTuneDecodeSlices,      // "decode_slices": CTAs per panel of a lone decode problem
  kTuneDecodeCtasPerSm,   // "decode_ctas_per_sm": 1 or 2
  kTuneDecodeRotMin,      // "decode_rot_min": first token count that uses the rotated chunk order
  kTuneWaitLimitCycles,   // "wait_limit_cycles": SM cycles after which a device-side wait gives up
  kTuneSkipCopies,        // "skip_copies": 1 = the producers of the matmul kernels issue no copies
                          //   (with a short wait limit: makes every bounded wait run out, faulting nothing)
  kTuneRegisterMaxM,      // "register_max_m": most tokens (1..16) a single call gives to the register-fragment kernel
  kTuneDecodeCluster,     // "decode_cluster": 0 = CTAs that share a panel meet in the global scratch, never in a cluster
  kTuneCount
};

int64_t tune(TuneKey key);

// Cycle budget of a bounded device-side wait: about two seconds unless overridden.
constexpr long long kDefaultWaitLimitCycles = 4000000000LL;
inline long long wait_limit_cycles() {
  const int64_t v = tune(kTuneWaitLimitCycles);
  return v >= 0 ? (long long)v : kDefaultWaitLimitCycles;
}

}  // namespace tl
