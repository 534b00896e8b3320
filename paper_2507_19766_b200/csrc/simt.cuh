// CUDA-core (SIMT, float32 accumulate) kernels: the path for float32 inputs and the on-device
// cross-check of the tensor-core path.  Same decomposition as the tensor path: a logits tile is
// formed in registers, reduced to online-softmax statistics (forward) or turned into
// dz = coef * (onehot - softmax) (backward), and never stored as logits.
#pragma once

#include "common.cuh"

namespace ulorl {

constexpr int kSimtTile = 64;     // tokens x vocabulary entries per block tile
constexpr int kSimtBK = 16;
constexpr int kSimtThreads = 256; // 16 x 16 threads, 4 x 4 outputs each

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void from_f32(float& d, float x) { d = x; }
__device__ __forceinline__ void from_f32(__nv_bfloat16& d, float x) { d = __float2bfloat16_rn(x); }

// acc[i][j] = sum_h hidden[row0 + ty*4 + i, h] * W[col0 + tx*4 + j, h]
template <typename TIn>
__device__ __forceinline__ void simt_logits_tile(const TIn* __restrict__ hidden, const TIn* __restrict__ W, int T,
                                                 int V, int H, int row0, int col0, float (&acc)[4][4],
                                                 float (*As)[kSimtTile + 1], float (*Bs)[kSimtTile + 1]) {
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  for (int k0 = 0; k0 < H; k0 += kSimtBK) {
#pragma unroll
    for (int e = tid; e < kSimtTile * kSimtBK; e += kSimtThreads) {
      const int r = e / kSimtBK, k = e % kSimtBK;
      const int gr = row0 + r, gc = col0 + r, gk = k0 + k;
      As[k][r] = (gr < T && gk < H) ? to_f32(hidden[(size_t)gr * H + gk]) : 0.f;
      Bs[k][r] = (gc < V && gk < H) ? to_f32(W[(size_t)gc * H + gk]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kSimtBK; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
}

// Forward statistics.  grid = (token tiles, vocabulary splits).  Each thread keeps running
// (max m, sum exp(kappa (a - m)), sum exp(kappa (a - m)) (a - m)) for its four rows over the columns it owns; the sixteen threads that
// share a row are merged with warp shuffles once at the end.
template <typename TIn>
__global__ void __launch_bounds__(kSimtThreads)
simt_stats_kernel(const TIn* __restrict__ hidden, const TIn* __restrict__ W, const int* __restrict__ targets, int T,
                  int V, int H, float kappa, int tiles_per_split, float4* __restrict__ partials,
                  float* __restrict__ acc_y, int* __restrict__ status) {
  __shared__ float As[kSimtBK][kSimtTile + 1];
  __shared__ float Bs[kSimtBK][kSimtTile + 1];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int row0 = blockIdx.x * kSimtTile;
  const int split = blockIdx.y;
  const int n_vtiles = (V + kSimtTile - 1) / kSimtTile;
  const int vt_begin = split * tiles_per_split;
  const int vt_end = min(n_vtiles, vt_begin + tiles_per_split);
  float m[4], s[4], u[4];
  int y[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    m[i] = -INFINITY;
    s[i] = 0.f;
    u[i] = 0.f;
    const int r = row0 + ty * 4 + i;
    int yy = r < T ? targets[r] : 0;
    if (yy < 0 || yy >= V) {
      if (tx == 0 && split == 0) atomicOr(status, kStatusBadTarget);
      yy = yy < 0 ? 0 : V - 1;
    }
    y[i] = yy;
  }
  for (int vt = vt_begin; vt < vt_end; ++vt) {
    float acc[4][4];
    const int col0 = vt * kSimtTile;
    simt_logits_tile<TIn>(hidden, W, T, V, H, row0, col0, acc, As, Bs);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float cmax = -INFINITY;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int col = col0 + tx * 4 + j;
        if (col < V) cmax = fmaxf(cmax, acc[i][j]);
      }
      if (cmax == -INFINITY) continue;
      const float mn = fmaxf(m[i], cmax);
      if (s[i] > 0.f) {                               // move the running sums to the new max
        const float d = m[i] - mn;
        const float sc = expf(kappa * d);
        u[i] = sc * fmaf(d, s[i], u[i]);
        s[i] *= sc;
      }
      m[i] = mn;
      float ls = 0.f, lu = 0.f;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int col = col0 + tx * 4 + j;
        if (col < V) {
          const float t = acc[i][j] - mn;
          const float e = expf(kappa * t);
          ls += e;
          lu = fmaf(e, t, lu);
          if (col == y[i] && row0 + ty * 4 + i < T) acc_y[row0 + ty * 4 + i] = acc[i][j];
        }
      }
      s[i] += ls;
      u[i] += lu;
    }
  }
  // merge the sixteen column owners of each row (lanes differing in the low four bits)
#pragma unroll
  for (int i = 0; i < 4; ++i) {
#pragma unroll
    for (int off = 1; off < 16; off <<= 1) {
      const float mo = __shfl_xor_sync(0xffffffffu, m[i], off);
      const float so = __shfl_xor_sync(0xffffffffu, s[i], off);
      const float uo = __shfl_xor_sync(0xffffffffu, u[i], off);
      const float mn = fmaxf(m[i], mo);
      if (mn != -INFINITY) {
        float sa = 0.f, ua = 0.f, sb = 0.f, ub = 0.f;
        if (s[i] > 0.f) {
          const float d = m[i] - mn, w = expf(kappa * d);
          sa = s[i] * w;
          ua = w * fmaf(d, s[i], u[i]);
        }
        if (so > 0.f) {
          const float d = mo - mn, w = expf(kappa * d);
          sb = so * w;
          ub = w * fmaf(d, so, uo);
        }
        s[i] = sa + sb;
        u[i] = ua + ub;
        m[i] = mn;
      }
    }
    const int r = row0 + ty * 4 + i;
    if (tx == 0 && r < T) partials[(size_t)split * T + r] = make_float4(m[i], s[i], u[i], 0.f);
  }
}

// Backward recompute: dz[t - t0, v] = coef_t * (1[v = y_t] - exp(kappa a - lse_t)) for the tokens of
// one panel, float32, leading dimension ld.  coef_t = kappa * grad_loss * grad_coef[t].
template <typename TIn>
__global__ void __launch_bounds__(kSimtThreads)
simt_dz_kernel(const TIn* __restrict__ hidden, const TIn* __restrict__ W, const int* __restrict__ targets,
               const float* __restrict__ lse, const float* __restrict__ grad_coef, const float* __restrict__ grad_loss,
               int T, int V, int H, float kappa, int t0, int t1, float* __restrict__ dz, size_t ld) {
  __shared__ float As[kSimtBK][kSimtTile + 1];
  __shared__ float Bs[kSimtBK][kSimtTile + 1];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int row0 = t0 + blockIdx.x * kSimtTile;
  const int col0 = blockIdx.y * kSimtTile;
  float acc[4][4];
  simt_logits_tile<TIn>(hidden, W, t1, V, H, row0, col0, acc, As, Bs);
  const float gl = grad_loss ? *grad_loss : 1.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = row0 + ty * 4 + i;
    if (r >= t1) continue;
    const float coef = kappa * gl * grad_coef[r];
    const float l = lse[r];
    int y = targets[r];
    y = y < 0 ? 0 : (y >= V ? V - 1 : y);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int col = col0 + tx * 4 + j;
      if (col < V) {
        const float p = expf(fmaf(kappa, acc[i][j], -l));
        dz[(size_t)(r - t0) * ld + col] = coef * ((col == y ? 1.f : 0.f) - p);
      }
    }
  }
}

// C[m, n] (+)= sum_k A(m, k) * B(k, n) with arbitrary element strides; float32 accumulate.
template <typename TA, typename TB, typename TC>
__global__ void __launch_bounds__(kSimtThreads)
simt_gemm_kernel(const TA* __restrict__ A, size_t a_sm, size_t a_sk, const TB* __restrict__ B, size_t b_sk,
                 size_t b_sn, TC* __restrict__ C, size_t c_sm, int M, int N, int K, int accumulate) {
  __shared__ float As[kSimtBK][kSimtTile + 1];
  __shared__ float Bs[kSimtBK][kSimtTile + 1];
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const int row0 = blockIdx.y * kSimtTile, col0 = blockIdx.x * kSimtTile;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  const bool a_m_fast = a_sm == 1, b_n_fast = b_sn == 1;
  for (int k0 = 0; k0 < K; k0 += kSimtBK) {
    for (int e = tid; e < kSimtTile * kSimtBK; e += kSimtThreads) {
      int r, k;
      if (a_m_fast) { r = e % kSimtTile; k = e / kSimtTile; } else { r = e / kSimtBK; k = e % kSimtBK; }
      const int gm = row0 + r, gk = k0 + k;
      As[k][r] = (gm < M && gk < K) ? to_f32(A[(size_t)gm * a_sm + (size_t)gk * a_sk]) : 0.f;
      int c, kk;
      if (b_n_fast) { c = e % kSimtTile; kk = e / kSimtTile; } else { c = e / kSimtBK; kk = e % kSimtBK; }
      const int gn = col0 + c, gk2 = k0 + kk;
      Bs[kk][c] = (gn < N && gk2 < K) ? to_f32(B[(size_t)gk2 * b_sk + (size_t)gn * b_sn]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kSimtBK; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gm = row0 + ty * 4 + i;
    if (gm >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gn = col0 + tx * 4 + j;
      if (gn >= N) continue;
      TC& dst = C[(size_t)gm * c_sm + gn];
      const float v = accumulate ? acc[i][j] + to_f32(dst) : acc[i][j];
      from_f32(dst, v);
    }
  }
}

}  // namespace ulorl
