// Per-token kernels after the LM-head pass: merge of the vocabulary splits, per-sequence mean
// entropy, and the decision stage (ratio, mask, clipped surrogate, loss, d loss / d logp).
#pragma once

#include "common.cuh"

namespace ulorl {

// ------------------------------------------------------------------------------------------
// Merge of the online-softmax partials of the vocabulary splits (log-softmax of Eq. 6, entropy
// of Eq. 10).  partials[split][t] = (m, s, u, -) with m the running max of the raw accumulator
// a = hidden . W[v], s = sum_v exp(kappa (a_v - m)), u = sum_v exp(kappa (a_v - m)) (a_v - m).
//   lse = kappa m* + ln s*,  logp = kappa a_y - lse,  Hent = ln s* - kappa u* / s*.
// ------------------------------------------------------------------------------------------
// Tokens [t_begin, t_end) of a batch of T; ranges of tokens may have been given different split counts.
__global__ void merge_splits_kernel(int T, int t_begin, int t_end, int n_split, float kappa,
                                    const float4* __restrict__ partials, const float* __restrict__ acc_y,
                                    float* __restrict__ logp, float* __restrict__ entropy, float* __restrict__ lse) {
  const int t = t_begin + blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= t_end) return;
  float m = -INFINITY;
  for (int k = 0; k < n_split; ++k) m = fmaxf(m, partials[(size_t)k * T + t].x);
  float s = 0.f, u = 0.f;
  for (int k = 0; k < n_split; ++k) {
    const float4 p = partials[(size_t)k * T + t];
    if (!(p.y > 0.f)) continue;
    const float d = p.x - m;
    const float w = expf(kappa * d);
    s = fmaf(p.y, w, s);
    u = fmaf(w, fmaf(d, p.y, p.z), u);
  }
  const float ln_s = logf(s);
  const float l = fmaf(kappa, m, ln_s);
  if (lse) lse[t] = l;
  if (logp) logp[t] = fmaf(kappa, acc_y[t], -l);
  if (entropy) entropy[t] = fmaxf(ln_s - kappa * u / s, 0.f);
}

// ------------------------------------------------------------------------------------------
// H-bar_i of Eq. 10: mean per-token entropy of each sequence.  One block per sequence; the sum is
// an exact 64-bit integer sum of the entropies in units of 2^-34 nats (common.cuh), so it is the
// same whatever the order, and a sequence cut over several calls or ranks adds up to the same bits.
// ------------------------------------------------------------------------------------------
constexpr int kSeqThreads = 256;

__device__ __forceinline__ long long entropy_to_fixed(float e) {
  // NaN counts as 0 and absurd magnitudes are clipped, so that the conversion is always defined
  const float c = (e == e) ? fminf(fmaxf(e, -1024.f), 1024.f) : 0.f;
  return __double2ll_rn((double)c * kEntropyFixScale);
}
__device__ __forceinline__ float fixed_mean(long long sum, long long count) {
  return count > 0 ? (float)(((double)sum * kEntropyFixInv) / (double)count) : 0.f;
}

// Sum over tokens [a, b) of one sequence by the whole block; the result is valid in thread 0.
__device__ __forceinline__ long long block_entropy_sum(const float* __restrict__ entropy, int a, int b) {
  __shared__ long long red[kSeqThreads];
  long long acc = 0;
  for (int t = a + threadIdx.x; t < b; t += kSeqThreads) acc += entropy_to_fixed(entropy[t]);
  red[threadIdx.x] = acc;
  __syncthreads();
  for (int w = kSeqThreads / 2; w > 0; w >>= 1) {
    if (threadIdx.x < w) red[threadIdx.x] += red[threadIdx.x + w];
    __syncthreads();
  }
  return red[0];
}

// Offsets are device data the host never saw: a bad pair is reported and clamped, never followed out of range.
__device__ __forceinline__ void checked_range(const int* __restrict__ seq_offsets, int i, int S, int T, int& a, int& b,
                                              int* __restrict__ status) {
  a = seq_offsets[i];
  b = seq_offsets[i + 1];
  const bool bad = a < 0 || b < a || b > T || (i == 0 && a != 0) || (i == S - 1 && b != T);
  if (bad) {
    if (threadIdx.x == 0 && status) atomicOr(status, kStatusBadOffsets);
    a = a < 0 ? 0 : (a > T ? T : a);
    b = b < a ? a : (b > T ? T : b);
  }
}

// Step 1: blocks of kSeqChunk consecutive tokens add their entropies into the (zeroed) integer sum of the
// sequence they belong to.  A block that lies inside one sequence -- nearly all of them, and every one of an
// ultra-long response -- reduces first and adds once; a block that crosses a boundary adds token by token.
// Integer addition makes the result independent of how the tokens are grouped.
constexpr int kSeqChunk = 4096;

__device__ __forceinline__ int sequence_of_token(const int* __restrict__ seq_offsets, int S, int t) {
  int lo = 0, hi = S;   // largest i with seq_offsets[i] <= t (an empty sequence never owns a token)
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (seq_offsets[mid] <= t) lo = mid; else hi = mid;
  }
  return lo;
}

__global__ void seq_entropy_sum_kernel(int S, int T, const int* __restrict__ seq_offsets,
                                       const float* __restrict__ entropy, long long* __restrict__ seq_sum) {
  const int t0 = blockIdx.x * kSeqChunk;
  const int t1 = min(T, t0 + kSeqChunk);
  if (t0 >= t1) return;
  const int first = sequence_of_token(seq_offsets, S, t0);
  const int last = sequence_of_token(seq_offsets, S, t1 - 1);
  if (first == last) {
    const long long sum = block_entropy_sum(entropy, t0, t1);
    if (threadIdx.x == 0) atomicAdd(reinterpret_cast<unsigned long long*>(seq_sum + first), (unsigned long long)sum);
  } else {
    for (int t = t0 + threadIdx.x; t < t1; t += kSeqThreads) {
      const int i = sequence_of_token(seq_offsets, S, t);
      atomicAdd(reinterpret_cast<unsigned long long*>(seq_sum + i), (unsigned long long)entropy_to_fixed(entropy[t]));
    }
  }
}

// Step 2 (one block): the mean of every sequence from its sum and its checked length, and the token mean of
// the whole call from the (exact) sum of the sequence sums.
__global__ void seq_entropy_mean_kernel(int S, int T, const int* __restrict__ seq_offsets,
                                        const long long* __restrict__ seq_sum, float* __restrict__ seq_entropy,
                                        float* __restrict__ batch_mean, int* __restrict__ status) {
  __shared__ long long red[kSeqThreads];
  long long acc = 0;
  for (int i = threadIdx.x; i < S; i += kSeqThreads) {
    int a = seq_offsets[i], b = seq_offsets[i + 1];
    // offsets are device data the host never saw: a bad pair is reported and clamped
    const bool bad = a < 0 || b < a || b > T || (i == 0 && a != 0) || (i == S - 1 && b != T);
    if (bad) {
      if (status) atomicOr(status, kStatusBadOffsets);
      a = a < 0 ? 0 : (a > T ? T : a);
      b = b < a ? a : (b > T ? T : b);
    }
    const long long sum = seq_sum[i];
    acc += sum;
    if (seq_entropy) seq_entropy[i] = fixed_mean(sum, (long long)(b - a));
  }
  red[threadIdx.x] = acc;
  __syncthreads();
  for (int w = kSeqThreads / 2; w > 0; w >>= 1) {
    if (threadIdx.x < w) red[threadIdx.x] += red[threadIdx.x + w];
    __syncthreads();
  }
  if (threadIdx.x == 0) *batch_mean = fixed_mean(red[0], (long long)T);
}

// The pieces of sequences that one call holds, as rows (sum, count) of a table over ALL sequences of the
// step: piece k of the call is sequence seq_ids[k] (k itself without seq_ids).  Rows of other sequences
// stay as the caller's memset left them; tables of several calls or ranks add up element by element.
__global__ void seq_entropy_partials_kernel(int S, int T, const int* __restrict__ seq_offsets,
                                            const float* __restrict__ entropy, const int* __restrict__ seq_ids,
                                            int total_seqs, long long* __restrict__ table, int* __restrict__ status) {
  const int k = blockIdx.x;
  int a, b;
  checked_range(seq_offsets, k, S, T, a, b, status);
  const long long sum = block_entropy_sum(entropy, a, b);
  if (threadIdx.x == 0) {
    const int id = seq_ids ? seq_ids[k] : k;
    if (id < 0 || id >= total_seqs) {
      if (status) atomicOr(status, kStatusBadOffsets);
    } else {                                   // pieces of one sequence inside one call are added, too
      atomicAdd(reinterpret_cast<unsigned long long*>(table + 2 * (size_t)id), (unsigned long long)sum);
      atomicAdd(reinterpret_cast<unsigned long long*>(table + 2 * (size_t)id + 1), (unsigned long long)(b - a));
    }
  }
}

// Means of the sequences seq_ids[0..n) from a summed table, with the arithmetic of seq_entropy_mean_kernel:
// a sequence whose pieces were summed here gets the float32 mean the unsplit call would have given it.
__global__ void seq_entropy_combine_kernel(int n, const int* __restrict__ seq_ids, int total_seqs,
                                           const long long* __restrict__ table, float* __restrict__ seq_entropy,
                                           float* __restrict__ batch_entropy) {
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k < n) {
    const int id = seq_ids ? seq_ids[k] : k;
    seq_entropy[k] = (id >= 0 && id < total_seqs) ? fixed_mean(table[2 * (size_t)id], table[2 * (size_t)id + 1]) : 0.f;
  }
  if (batch_entropy && k == 0) {
    long long tot = 0, cnt = 0;
    for (int i = 0; i < total_seqs; ++i) { tot += table[2 * (size_t)i]; cnt += table[2 * (size_t)i + 1]; }
    *batch_entropy = fixed_mean(tot, cnt);
  }
}

// ------------------------------------------------------------------------------------------
// Decision stage: four consecutive tokens per thread, 1024 per block, 128-bit loads and stores
// where the arrays allow it.
//   MPT (Eq. 9):        A > 0 and logp >= ln tau          gate (Eq. 10): H-bar < sigma
//   ratio (Eq. 8):      d = logp - old_logp, r = exp(d)   (POIS: r = 1, nothing clipped)
//   surrogate (Eq. 10): s = min(r A, clip(r, 1 - eps_lo, 1 + eps_hi) A)
//   gradient:           g = -(1/N) (1 - msk) A r [not clipped]
// Decisions are float32 comparisons against host-computed thresholds; values are float64.
// ------------------------------------------------------------------------------------------
constexpr int kDecideThreads = 256;
constexpr int kDecideVec = 4;
constexpr int kDecideTokens = kDecideThreads * kDecideVec;

__device__ __forceinline__ int find_sequence(const int* __restrict__ seq_offsets, int S, int t) {
  int lo = 0, hi = S;   // largest i with seq_offsets[i] <= t
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (seq_offsets[mid] <= t) lo = mid; else hi = mid;
  }
  return lo;
}

// kVec: logp, old_logp, segment_version, per-token advantages, grad_coef are 16-byte aligned and flags
// 4-byte aligned, so a thread's four tokens move as one vector when all four exist.
template <bool kVec>
__global__ void decide_kernel(int T, int S, DecideConsts c, const float* __restrict__ logp,
                              const float* __restrict__ old_logp, const float* __restrict__ ref_logp,
                              const int* __restrict__ segment_version,
                              const float* __restrict__ advantages, const int* __restrict__ seq_offsets,
                              const float* __restrict__ gate_entropy, const float* __restrict__ batch_mean,
                              float* __restrict__ grad_coef, uint8_t* __restrict__ flags,
                              DecidePartial* __restrict__ partials) {
  __shared__ double sh_loss[kDecideThreads];
  __shared__ double sh_kl[kDecideThreads];
  __shared__ double sh_abs_warp[ULORL_N_STALENESS][kDecideThreads / 32];
  __shared__ int sh_cnt[5];
  __shared__ int sh_stale[2][ULORL_N_STALENESS];
  const int tid = threadIdx.x;
  const int t0 = blockIdx.x * kDecideTokens + tid * kDecideVec;
  if (tid < 5) sh_cnt[tid] = 0;
  if (tid < ULORL_N_STALENESS) { sh_stale[0][tid] = 0; sh_stale[1][tid] = 0; }
  __syncthreads();

  const bool sais = c.is_mode == ULORL_IS_SAIS;
  const bool with_kl = c.kl_beta > 0.0;
  const bool whole = kVec && t0 + kDecideVec <= T;
  float lp4[kDecideVec], old4[kDecideVec], adv4[kDecideVec], ref4[kDecideVec];
  int ver4[kDecideVec];
#pragma unroll
  for (int k = 0; k < kDecideVec; ++k) { lp4[k] = 0.f; old4[k] = 0.f; adv4[k] = 0.f; ref4[k] = 0.f; ver4[k] = c.current_version; }
  if (whole) {
    const float4 v = *reinterpret_cast<const float4*>(logp + t0);
    lp4[0] = v.x; lp4[1] = v.y; lp4[2] = v.z; lp4[3] = v.w;
    if (sais) {
      const float4 o = *reinterpret_cast<const float4*>(old_logp + t0);
      old4[0] = o.x; old4[1] = o.y; old4[2] = o.z; old4[3] = o.w;
    }
    if (with_kl) {
      const float4 rf = *reinterpret_cast<const float4*>(ref_logp + t0);
      ref4[0] = rf.x; ref4[1] = rf.y; ref4[2] = rf.z; ref4[3] = rf.w;
    }
    if (segment_version) {
      const int4 sv = *reinterpret_cast<const int4*>(segment_version + t0);
      ver4[0] = sv.x; ver4[1] = sv.y; ver4[2] = sv.z; ver4[3] = sv.w;
    }
    if (c.adv_per_token) {
      const float4 a = *reinterpret_cast<const float4*>(advantages + t0);
      adv4[0] = a.x; adv4[1] = a.y; adv4[2] = a.z; adv4[3] = a.w;
    }
  } else {
#pragma unroll
    for (int k = 0; k < kDecideVec; ++k) {
      const int t = t0 + k;
      if (t < T) {
        lp4[k] = logp[t];
        if (sais) old4[k] = old_logp[t];
        if (with_kl) ref4[k] = ref_logp[t];
        if (segment_version) ver4[k] = segment_version[t];
        if (c.adv_per_token) adv4[k] = advantages[t];
      }
    }
  }

  double contrib = 0.0, kl_acc = 0.0;
  float g4[kDecideVec], dabs4[kDecideVec];
  int bucket4[kDecideVec];
  unsigned f4[kDecideVec];
  int seq = t0 < T ? find_sequence(seq_offsets, S, t0) : 0;
#pragma unroll
  for (int k = 0; k < kDecideVec; ++k) {
    const int t = t0 + k;
    float dabs = 0.f;
    int bucket = -1;
    g4[k] = 0.f;
    f4[k] = 0u;
    if (t < T) {
      while (seq + 1 < S && seq_offsets[seq + 1] <= t) ++seq;   // the largest i with seq_offsets[i] <= t
      const int i = seq;
      const float A = c.adv_per_token ? adv4[k] : advantages[i];
      bool gate = false;
      if (c.mpt_mode == ULORL_MPT_ALWAYS) {
        gate = true;
      } else if (c.mpt_mode == ULORL_MPT_DYNAMIC) {
        const float h = (c.ent_scope == ULORL_ENT_BATCH) ? *batch_mean : gate_entropy[i];
        gate = h < c.sigma;
      }
      const float lp = lp4[k];
      const bool mpt = (A > 0.f) && (lp >= c.ln_tau);
      const bool msk = mpt && gate;
      double r = 1.0;
      bool hi = false, lo = false;
      if (sais) {
        const float d = __fsub_rn(lp, old4[k]);
        r = exp((double)d);
        hi = (A > 0.f) && (d > c.ln_hi);
        lo = (A < 0.f) && (d < c.ln_lo);
        dabs = fabsf(d);
      }
      const double Ad = (double)A;
      const double cl = fmin(fmax(r, 1.0 - c.eps_lo), 1.0 + c.eps_hi);
      const double s = fmin(r * Ad, cl * Ad);
      // weight of the token's term: 1/N (Eq. 10), or 1/(G |o_i|) for the per-sample mean of Eq. 5
      // (inv_N then holds 1/G)
      double wlen = 1.0;
      if (c.loss_norm == ULORL_NORM_SEQUENCE) {
        const int len = seq_offsets[i + 1] - seq_offsets[i];
        wlen = 1.0 / (double)(len > 0 ? len : 1);
      }
      // Eq. 5's KL-to-reference term, when asked for: token term s - beta k with k = e^u - u - 1,
      // u = ref_logp - logp (exact in float64), d k / d logp = 1 - e^u; inside the mask like the surrogate
      double k_t = 0.0, dk = 0.0;
      if (with_kl) {
        const double u = (double)ref4[k] - (double)lp;
        const double eu = exp(u);
        k_t = eu - u - 1.0;
        dk = 1.0 - eu;
        kl_acc += k_t;
      }
      if (!msk) contrib += (s - c.kl_beta * k_t) * wlen;
      const double g = msk ? 0.0 : -c.inv_N * (((hi || lo) ? 0.0 : Ad * r) - c.kl_beta * dk) * wlen + 0.0;   // + 0.0: no -0
      g4[k] = (float)g;
      f4[k] = (msk ? ULORL_FLAG_MASKED : 0u) | (hi ? ULORL_FLAG_CLIP_HIGH : 0u) |
              (lo ? ULORL_FLAG_CLIP_LOW : 0u) | (mpt ? ULORL_FLAG_MPT : 0u);
      int st = segment_version ? c.current_version - ver4[k] : 0;
      st = st < 0 ? 0 : (st > ULORL_N_STALENESS - 1 ? ULORL_N_STALENESS - 1 : st);
      bucket = st;
      if (g != 0.0) atomicAdd(&sh_cnt[0], 1);
      if (mpt) atomicAdd(&sh_cnt[1], 1);
      if (msk) atomicAdd(&sh_cnt[2], 1);
      if (hi) atomicAdd(&sh_cnt[3], 1);
      if (lo) atomicAdd(&sh_cnt[4], 1);
      atomicAdd(&sh_stale[0][st], 1);
      if (hi || lo) atomicAdd(&sh_stale[1][st], 1);
    }
    dabs4[k] = dabs;
    bucket4[k] = bucket;
  }
  if (whole) {
    if (grad_coef) *reinterpret_cast<float4*>(grad_coef + t0) = make_float4(g4[0], g4[1], g4[2], g4[3]);
    if (flags) *reinterpret_cast<uchar4*>(flags + t0) = make_uchar4((unsigned char)f4[0], (unsigned char)f4[1],
                                                                    (unsigned char)f4[2], (unsigned char)f4[3]);
  } else {
#pragma unroll
    for (int k = 0; k < kDecideVec; ++k) {
      const int t = t0 + k;
      if (t < T) {
        if (grad_coef) grad_coef[t] = g4[k];
        if (flags) flags[t] = (uint8_t)f4[k];
      }
    }
  }
  sh_loss[tid] = contrib;
  sh_kl[tid] = kl_acc;
  __syncthreads();
  for (int w = kDecideThreads / 2; w > 0; w >>= 1) {
    if (tid < w) { sh_loss[tid] += sh_loss[tid + w]; sh_kl[tid] += sh_kl[tid + w]; }
    __syncthreads();
  }
  DecidePartial* out = partials + blockIdx.x;
  // sum of |log ratio| per staleness bucket, in a fixed order: a thread's tokens in token order, a fixed
  // butterfly inside each warp, the warps in order; buckets without a token in this block are skipped
  // (the counts were complete at the barrier above)
  for (int s = 0; s < ULORL_N_STALENESS; ++s) {
    if (sh_stale[0][s] == 0 || !sais) continue;
    double a = 0.0;
#pragma unroll
    for (int k = 0; k < kDecideVec; ++k)
      if (bucket4[k] == s) a += (double)dabs4[k];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
    if ((tid & 31) == 0) sh_abs_warp[s][tid >> 5] = a;
  }
  __syncthreads();
  if (tid < ULORL_N_STALENESS) {
    double a = 0.0;
    if (sh_stale[0][tid] != 0 && sais)
      for (int w = 0; w < kDecideThreads / 32; ++w) a += sh_abs_warp[tid][w];
    out->stale_abs[tid] = a;
    out->stale_tokens[tid] = sh_stale[0][tid];
    out->stale_clipped[tid] = sh_stale[1][tid];
  }
  if (tid == 0) {
    out->loss_sum = sh_loss[0];
    out->kl_sum = sh_kl[0];
    out->n_active = sh_cnt[0];
    out->n_mpt = sh_cnt[1];
    out->n_masked = sh_cnt[2];
    out->n_clip_high = sh_cnt[3];
    out->n_clip_low = sh_cnt[4];
    out->pad = 0;
  }
}

// Sum of the per-block partials in a fixed order; writes the loss and the statistics.  One pass over the
// partials with every field in registers, then one fixed butterfly per field inside each warp and a fixed
// sum over the eight warps: the order of the additions never depends on scheduling.
constexpr int kFinalThreads = 256;

template <typename V>
__device__ __forceinline__ V warp_sum_fixed(V v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  return v;
}

__global__ void finalize_kernel(int T, int n_blocks, double inv_N, const DecidePartial* __restrict__ partials,
                                const float* __restrict__ batch_mean, const int* __restrict__ status,
                                float* __restrict__ loss, ulorl_stats_t* __restrict__ stats) {
  constexpr int kWarps = kFinalThreads / 32;
  constexpr int kD = 2 + ULORL_N_STALENESS;           // doubles: loss, stale_abs[], KL sum (last)
  constexpr int kI = 5 + 2 * ULORL_N_STALENESS;       // ints: five counters, stale_tokens[], stale_clipped[]
  __shared__ double shd[kWarps][kD];
  __shared__ int shi[kWarps][kI];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  double d[kD];
  int n[kI];
#pragma unroll
  for (int k = 0; k < kD; ++k) d[k] = 0.0;
#pragma unroll
  for (int k = 0; k < kI; ++k) n[k] = 0;
  for (int b = tid; b < n_blocks; b += kFinalThreads) {
    const DecidePartial& p = partials[b];
    d[0] += p.loss_sum;
    d[kD - 1] += p.kl_sum;
    n[0] += p.n_active;
    n[1] += p.n_mpt;
    n[2] += p.n_masked;
    n[3] += p.n_clip_high;
    n[4] += p.n_clip_low;
#pragma unroll
    for (int s = 0; s < ULORL_N_STALENESS; ++s) {
      d[1 + s] += p.stale_abs[s];
      n[5 + s] += p.stale_tokens[s];
      n[5 + ULORL_N_STALENESS + s] += p.stale_clipped[s];
    }
  }
#pragma unroll
  for (int k = 0; k < kD; ++k) {
    const double v = warp_sum_fixed<double>(d[k]);
    if (lane == 0) shd[warp][k] = v;
  }
#pragma unroll
  for (int k = 0; k < kI; ++k) {
    const int v = warp_sum_fixed<int>(n[k]);
    if (lane == 0) shi[warp][k] = v;
  }
  __syncthreads();
  if (tid != 0) return;
  double dt[kD];
  int nt[kI];
  for (int k = 0; k < kD; ++k) {
    dt[k] = 0.0;
    for (int w = 0; w < kWarps; ++w) dt[k] += shd[w][k];
  }
  for (int k = 0; k < kI; ++k) {
    nt[k] = 0;
    for (int w = 0; w < kWarps; ++w) nt[k] += shi[w][k];
  }
  const float loss_value = (float)(-dt[0] * inv_N);
  if (loss) loss[0] = loss_value;
  if (!stats) return;
  for (int s = 0; s < ULORL_N_STALENESS; ++s) {
    const int ntt = nt[5 + s];
    stats->stale_tokens[s] = ntt;
    stats->stale_clipped[s] = nt[5 + ULORL_N_STALENESS + s];
    stats->stale_mean_abs_logratio[s] = ntt > 0 ? (float)(dt[1 + s] / (double)ntt) : 0.f;
  }
  stats->loss = loss_value;
  stats->mean_entropy = *batch_mean;
  stats->n_tokens = T;
  stats->n_active = nt[0];
  stats->n_mpt = nt[1];
  stats->n_masked = nt[2];
  stats->n_clip_high = nt[3];
  stats->n_clip_low = nt[4];
  stats->device_status = *status;
  stats->mean_kl = T > 0 ? (float)(dt[kD - 1] / (double)T) : 0.f;
  stats->reserved[0] = stats->reserved[1] = 0;
}

// ------------------------------------------------------------------------------------------
// Group-normalised advantages (Eq. 4) and the dynamic-sampling filter of Eq. 7, one thread per
// group of `group` consecutive responses: A_i = (R_i - mean) / std with the population standard
// deviation in float64, 0 when the group has no spread; keep_i = 0 < #(R == 1) < G.
// ------------------------------------------------------------------------------------------
__global__ void group_advantage_kernel(int S, int group, const float* __restrict__ rewards, float* __restrict__ adv,
                                       uint8_t* __restrict__ keep) {
  const int gidx = blockIdx.x * blockDim.x + threadIdx.x;
  const int a = gidx * group;
  if (a >= S) return;
  const int b = min(S, a + group);
  const int G = b - a;
  double mean = 0.0;
  int n_correct = 0;
  for (int i = a; i < b; ++i) {
    mean += (double)rewards[i];
    n_correct += rewards[i] == 1.f ? 1 : 0;
  }
  mean /= (double)G;
  double var = 0.0;
  for (int i = a; i < b; ++i) {
    const double d = (double)rewards[i] - mean;
    var += d * d;
  }
  const double sd = sqrt(var / (double)G);
  const uint8_t kept = (n_correct > 0 && n_correct < G) ? 1 : 0;
  for (int i = a; i < b; ++i) {
    adv[i] = sd > 0.0 ? (float)(((double)rewards[i] - mean) / sd) : 0.f;
    if (keep) keep[i] = kept;
  }
}

// ------------------------------------------------------------------------------------------
// bf16 d_W: rows of the float32 sum over tokens that are final are rounded once (round to nearest
// even) into the caller's array, eight elements a thread; with `accumulate` the caller's values are
// added first.
// ------------------------------------------------------------------------------------------
__global__ void dw_round_kernel(const float* __restrict__ acc, __nv_bfloat16* __restrict__ out, size_t n8, int accumulate) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += (size_t)gridDim.x * blockDim.x) {
    const float4 a0 = reinterpret_cast<const float4*>(acc)[2 * i];
    const float4 a1 = reinterpret_cast<const float4*>(acc)[2 * i + 1];
    float v[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
    uint4* dst = reinterpret_cast<uint4*>(out) + i;
    if (accumulate) {
      const uint4 old = *dst;
      const __nv_bfloat162* o = reinterpret_cast<const __nv_bfloat162*>(&old);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 f = __bfloat1622float2(o[j]);
        v[2 * j] += f.x;
        v[2 * j + 1] += f.y;
      }
    }
    uint4 r;
    __nv_bfloat162* rp = reinterpret_cast<__nv_bfloat162*>(&r);
#pragma unroll
    for (int j = 0; j < 4; ++j) rp[j] = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
    *dst = r;
  }
}

// ------------------------------------------------------------------------------------------
// Active-row compaction of the backward.  Tokens whose d loss / d logp is exactly zero (masked
// well-mastered positive tokens of Eq. 10, clipped tokens, zero advantage) add nothing to dHidden or
// dW, so the backward contractions run on the remaining rows only.
//   compact_count_kernel   active tokens per block of 256
//   compact_offsets_kernel exclusive scan of the block counts (one block), total -> n_active
//   compact_gather_kernel  position of every token among the active ones; hidden rows, targets, lse
//                          and coefficient of the active tokens gathered in token order; the rows up
//                          to the next multiple of 256 zero-filled (they are read as padding)
//   compact_scatter_kernel dHidden rows back to their tokens, zeros for the inactive ones
// ------------------------------------------------------------------------------------------
constexpr int kCompactThreads = 256;

__global__ void compact_count_kernel(int T, const float* __restrict__ grad_coef, int* __restrict__ block_count) {
  const int t = blockIdx.x * kCompactThreads + threadIdx.x;
  const int active = (t < T && grad_coef[t] != 0.f) ? 1 : 0;
  const int n = __syncthreads_count(active);
  if (threadIdx.x == 0) block_count[blockIdx.x] = n;
}

__global__ void compact_offsets_kernel(int n_blocks, const int* __restrict__ block_count, int* __restrict__ block_offset,
                                       int* __restrict__ n_active) {
  __shared__ int sh[1024];
  // n_blocks can exceed the block size: every thread owns a contiguous run of blocks
  const int per = (n_blocks + 1023) / 1024;
  const int b0 = threadIdx.x * per, b1 = min(n_blocks, b0 + per);
  int sum = 0;
  for (int b = b0; b < b1; ++b) sum += block_count[b];
  sh[threadIdx.x] = sum;
  __syncthreads();
  for (int off = 1; off < 1024; off <<= 1) {          // inclusive scan of the per-thread sums
    const int v = threadIdx.x >= off ? sh[threadIdx.x - off] : 0;
    __syncthreads();
    sh[threadIdx.x] += v;
    __syncthreads();
  }
  int run = sh[threadIdx.x] - sum;
  for (int b = b0; b < b1; ++b) {
    block_offset[b] = run;
    run += block_count[b];
  }
  if (threadIdx.x == 1023) *n_active = sh[1023];
}

template <typename TIn>
__global__ void compact_gather_kernel(int T, int H, const float* __restrict__ grad_coef, const int* __restrict__ block_offset,
                                      const int* __restrict__ n_active, const TIn* __restrict__ hidden,
                                      const int* __restrict__ targets, const float* __restrict__ lse,
                                      int* __restrict__ position, TIn* __restrict__ hidden_c, int* __restrict__ targets_c,
                                      float* __restrict__ lse_c, float* __restrict__ coef_c) {
  __shared__ int sh_pos[kCompactThreads];
  const int t = blockIdx.x * kCompactThreads + threadIdx.x;
  const bool active = t < T && grad_coef[t] != 0.f;
  // rank inside the block by warp ballots
  const unsigned ballot = __ballot_sync(0xffffffffu, active);
  __shared__ int warp_base[kCompactThreads / 32];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) warp_base[warp] = __popc(ballot);
  __syncthreads();
  int base = block_offset[blockIdx.x];
  for (int w = 0; w < warp; ++w) base += warp_base[w];
  const int pos = active ? base + __popc(ballot & ((1u << lane) - 1u)) : -1;
  sh_pos[threadIdx.x] = pos;
  if (t < T) position[t] = pos;
  if (active) {
    targets_c[pos] = targets[t];
    lse_c[pos] = lse[t];
    coef_c[pos] = grad_coef[t];
  }
  __syncthreads();
  // rows: 16-byte vectors, the whole block cooperates on each active token of the block
  const int vec_per_row = H * (int)sizeof(TIn) / 16;
  for (int r = 0; r < kCompactThreads; ++r) {
    const int p = sh_pos[r];
    if (p < 0) continue;
    const uint4* src = reinterpret_cast<const uint4*>(hidden + (size_t)(blockIdx.x * kCompactThreads + r) * H);
    uint4* dst = reinterpret_cast<uint4*>(hidden_c + (size_t)p * H);
    for (int v = threadIdx.x; v < vec_per_row; v += kCompactThreads) dst[v] = src[v];
  }
  // the last block zero-fills the padding rows [n_active, next multiple of 256)
  if (blockIdx.x == gridDim.x - 1) {
    const int n = *n_active;
    const int n_pad = (n + 255) / 256 * 256;
    for (int p = n; p < n_pad; ++p) {
      uint4* dst = reinterpret_cast<uint4*>(hidden_c + (size_t)p * H);
      for (int v = threadIdx.x; v < vec_per_row; v += kCompactThreads) dst[v] = make_uint4(0u, 0u, 0u, 0u);
      if (threadIdx.x == 0) { targets_c[p] = 0; lse_c[p] = 0.f; coef_c[p] = 0.f; }
    }
  }
}

template <typename TIn>
__global__ void compact_scatter_kernel(int T, int H, const int* __restrict__ position, const TIn* __restrict__ d_hidden_c,
                                       TIn* __restrict__ d_hidden) {
  // one block per 8 tokens, 16-byte vectors
  const int vec_per_row = H * (int)sizeof(TIn) / 16;
  for (int r = 0; r < 8; ++r) {
    const int t = blockIdx.x * 8 + r;
    if (t >= T) return;
    const int p = position[t];
    uint4* dst = reinterpret_cast<uint4*>(d_hidden + (size_t)t * H);
    if (p >= 0) {
      const uint4* src = reinterpret_cast<const uint4*>(d_hidden_c + (size_t)p * H);
      for (int v = threadIdx.x; v < vec_per_row; v += blockDim.x) dst[v] = src[v];
    } else {
      for (int v = threadIdx.x; v < vec_per_row; v += blockDim.x) dst[v] = make_uint4(0u, 0u, 0u, 0u);
    }
  }
}

}  // namespace ulorl
