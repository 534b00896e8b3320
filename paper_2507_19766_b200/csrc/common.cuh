// Shared host/device definitions of the UloRL token-loss library.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ulorl.h"

namespace ulorl {

constexpr int kPartialStride = 4;   // floats per (token, vocab split): running max, sum exp, sum exp*z, pad
constexpr int kMaxSplits = 32;

// Device status word (first int of the workspace).  Bits, so that several problems can be kept.
constexpr int kStatusTimeout = 1;
constexpr int kStatusBadTarget = 2;
constexpr int kStatusBadOffsets = 4;   // seq_offsets not 0 = o[0] <= o[1] <= ... <= o[S] = T

// Per-block partial results of the decision kernel, reduced in block order by a final kernel
// so that the loss and the statistics do not depend on scheduling.
struct DecidePartial {
  double loss_sum;
  double kl_sum;
  double stale_abs[ULORL_N_STALENESS];
  int n_active, n_mpt, n_masked, n_clip_high, n_clip_low, pad;
  int stale_tokens[ULORL_N_STALENESS];
  int stale_clipped[ULORL_N_STALENESS];
};

// Values the host derives once per call for the decision stage.  The thresholds are float32
// roundings of float64 evaluations, so that no transcendental sits inside a comparison.
struct DecideConsts {
  float ln_tau, ln_hi, ln_lo, sigma;
  double eps_lo, eps_hi, inv_N, kl_beta;
  int is_mode, mpt_mode, ent_scope, adv_per_token, current_version, loss_norm;
};

// Per-sequence entropy sums (H-bar of Eq. 10) are kept as 64-bit integers in units of 2^-kEntropyFixShift
// nats: integer addition is associative, so the sum of a sequence does not depend on the order of its
// tokens, on how a launch spreads them over threads, or on how a token-range sharding cuts the
// sequence over ranks -- an integer all-reduce of the pieces gives the unsplit sum bit for bit.  One
// token is rounded by at most 2^-35 nats (its float32 entropy carries 2^-24 relative), and a sum holds
// up to 2^29 nats, which the host checks against T ln V.
constexpr int kEntropyFixShift = 34;
constexpr double kEntropyFixScale = 17179869184.0;          // 2^34
constexpr double kEntropyFixInv = 1.0 / 17179869184.0;
constexpr double kEntropyFixCapacity = 536870912.0;         // 2^29 nats per sum (2^63 / 2^34)

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace ulorl
