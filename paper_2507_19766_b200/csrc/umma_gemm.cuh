// Tensor-core kernels (tcgen05 / tensor memory / TMA) for the four dense contractions of the
// token-loss path, bf16 inputs and float32 accumulation:
//
//   kModeStats   a = hidden . W^T per (token tile, vocabulary tile); the epilogue reduces the tile to
//                online-softmax statistics per token (Eq. 6, Eq. 10) -- logits never leave the SM
//   kModeDz      same contraction, epilogue writes dz = coef * (onehot - softmax) as bf16 to a token panel
//   kModeDHidden d_hidden[t, :] = sum_v dz[t, v] W[v, :]
//   kModeDW      d_W[v, :] (+)= sum_t dz[t, v] hidden[t, :]
//
// One kernel template umma_kernel<mode, CTAs per MMA, accumulators per unit>, persistent, one CTA per
// SM, 192 threads: one thread of warp 0 feeds a shared-memory ring with TMA tile loads (128-byte
// swizzle), one thread of warp 1 issues tcgen05.mma into tensor memory, warps 2-5 drain accumulators
// with tcgen05.ld (one output row per thread) and run the mode's epilogue.
//   <m, 2, 1>  CTA pair, one 256 x 256 MMA tile over both CTAs, two 256-column accumulator buffers: the
//              epilogue of tile i overlaps the contraction of tile i + 1 (statistics, dz)
//   <m, 2, 2>  CTA pair, 256 x 512 unit = two accumulators fed from the same A stage, tensor memory as
//              one buffer (d_hidden, d_W: long reductions, light epilogues)
//   <m, 1, 1>  single CTA, 128 x 256 tile, two accumulator buffers (cross-check variant)
// Operands whose contraction index is not the contiguous one in memory (W and hidden in the two
// gradient contractions, dz in the d_W one) are loaded as MN-major tiles; nothing is transposed in
// global memory.  No TMA multicast is used.  Every mbarrier wait is bounded.
#pragma once

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace ulorl {

constexpr int kBM = 128;           // accumulator rows (tensor-memory lanes)
constexpr int kBN = 256;           // accumulator columns
constexpr int kBK = 64;            // contraction elements per pipeline stage (128 bytes of bf16)
constexpr int kUmmaK = 16;         // contraction elements per tcgen05.mma
constexpr int kUmmaThreads = 192;
constexpr int kTmemCols = 512;     // two accumulators of kBN columns
constexpr uint32_t kABytes = kBM * kBK * 2;
constexpr uint32_t kBBytes = kBN * kBK * 2;
constexpr uint32_t kChunkBytes = 64 * kBK * 2;   // one MN-major box: 64 k-rows of 64 contiguous elements

// Shared-memory ring per CTA.  One CTA alone loads the whole 256-row B tile (48 KB a stage, 4 stages);
// in a CTA pair each CTA loads its 128 rows of A and half of B (32 KB a stage, 6 stages), and one
// tcgen05.mma over the pair covers 256 x 256 outputs: a third less L2 traffic per flop.  With two
// accumulators per unit (kAcc = 2) a pair covers 256 x 512 outputs per k-block: A is loaded once
// for both column blocks (48 KB a stage, 4 stages), eight MMAs are queued per barrier round trip,
// and tensor memory is used as one 512-column buffer, so the epilogue does not overlap the next
// unit -- right for the gradient contractions, whose reduction runs over 10^4..10^5 elements.

// Two staging tiles (128 rows x 128 bytes each, 128-byte swizzle) through which the d_W epilogue
// hands 32-column chunks of the accumulator to TMA store / reduce-add.
constexpr uint32_t kOutStageBytes = kBM * 128;

// A stage holds kKA "atoms" of 64 contraction elements (one 128-byte swizzle span each); the two
// logits kernels use two atoms a stage, so that eight MMAs are queued per barrier round trip there too.
template <int kMode, int kCta>
struct KAtoms { static constexpr int value = (kCta == 2 && (kMode == 0 || kMode == 1)) ? 2 : 1; };

template <int kCta, int kAcc, int kKA>
struct PipeConfig {
  static constexpr uint32_t atom_bytes = kABytes + kAcc * kBBytes / kCta;
  static constexpr uint32_t stage_bytes = kKA * atom_bytes;
  static constexpr int stages = (int)(196608u / stage_bytes);
  static constexpr size_t smem_bytes = (size_t)stages * stage_bytes + 1024 + 2 * kOutStageBytes;
};
constexpr long long kWaitLimitCycles = 4000000000LL;   // about two seconds at the maximum SM clock

enum UmmaMode { kModeStats = 0, kModeDz = 1, kModeDHidden = 2, kModeDW = 3 };

struct UmmaArgs {
  int M, N, K;              // extents of the contraction handled by this launch (valid elements)
  int m_tiles, n_tiles;     // ceil(M / rows per unit), ceil(N / columns per unit)
  int n_split;              // kModeStats: vocabulary splits; a unit is (token tile, split)
  int tiles_per_split;
  // kModeStats: split s owns the vocabulary tiles [s * split_stride, (s + 1) * split_stride); a launch sweeps the
  // tiles_per_split tiles of each split that start at offset tile_base inside it.  A whole sweep has tile_base = 0
  // and tiles_per_split = split_stride; a sweep cut into several launches (W still arriving) sets `resume` on
  // all but the first, and a row's running (max, sum, sum) then continues from `partials` exactly where the
  // launch before left it, so the cut does not change a bit of the result.
  int split_stride, tile_base, resume;
  int group_m;              // other modes: token tiles per raster group (tiles of a group run m-fastest)
  int a_mn0, a_k0;          // coordinate offsets of operand A in its tensor map (MN index, K index)
  int b_mn0, b_k0;
  int row0;                 // global token (or vocabulary row) index of accumulator row 0 of tile 0
  float kappa;
  const int* targets;
  const float* lse;
  const float* grad_coef;
  const float* grad_loss;
  float4* partials;         // kModeStats: [n_split][T_total]
  float* acc_y;             // kModeStats: raw accumulator at the target column, [T_total]
  int T_total;
  int dz_cols;              // kModeDz: columns of the panel written per row (>= N, zero beyond N); the panel
                            // itself is reached through the kernel's third tensor map
  __nv_bfloat16* d_hidden;  // kModeDHidden: [T][out_ld]
  float* d_W;               // kModeDW: [V][out_ld]
  size_t out_ld;
  int accumulate;
  int* status;
  int l2_a, l2_b;           // ptx::L2Hint of the loads of A and of B (CTA-pair kernels)
  const int* dyn_rows;      // optional device count of rows of the whole (compacted) batch: the launch then
  int dyn_base;             // covers rows [dyn_base, min(dyn_base + capacity, *dyn_rows)) of it (M, or K for d_W)
};

template <int kMode>
struct ModeTraits {
  static constexpr bool a_mn = (kMode == kModeDW);
  static constexpr bool b_mn = (kMode == kModeDHidden || kMode == kModeDW);
};

// Raster of the (m, n) output tiles for the modes without vocabulary splits: groups of `group_m`
// row tiles, m fastest inside a group, so that the CTAs running at one time share a few B tiles and
// keep the group's A tiles resident in L2 instead of streaming all of B once per row tile.
__device__ __forceinline__ void unit_to_tile(int unit, const UmmaArgs& args, int& m_tile, int& n_tile) {
  const int per_group = args.group_m * args.n_tiles;
  const int group = unit / per_group;
  const int first_m = group * args.group_m;
  const int rows = min(args.group_m, args.m_tiles - first_m);
  const int local = unit - group * per_group;
  m_tile = first_m + local % rows;
  n_tile = local / rows;
}

// Vocabulary tiles [n_begin, n_end) that this launch sweeps for split `split` (kModeStats); may be empty.
__device__ __forceinline__ void stats_tile_range(const UmmaArgs& args, int split, int& n_begin, int& n_end) {
  const int first = split * args.split_stride;
  n_begin = first + args.tile_base;
  n_end = min(min(n_begin + args.tiles_per_split, first + args.split_stride), args.n_tiles);
  if (n_end < n_begin) n_end = n_begin;
}

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// raw[idx] for an index only known at run time, as a chain of predicated moves over registers.  Written
// as a plain select loop the compiler turns it into an indexed read, which puts the whole chunk in
// local memory: every accumulator then goes through a store and a load (128 bytes of stack per
// thread), and the statistics kernel loses a sixth of its rate.
__device__ __forceinline__ float pick_column(const uint32_t (&raw)[32], int idx) {
  uint32_t v = 0u;
#pragma unroll
  for (int j = 0; j < 32; ++j)
    asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.s32 p, %1, %2;\n\t@p mov.b32 %0, %3;\n\t}"
                 : "+r"(v) : "r"(idx), "r"(j), "r"(raw[j]));
  return __uint_as_float(v);
}

// One 32-column chunk of a row folded into the running (m, s, u) with m the max of the raw
// accumulators a, s = sum 2^(c2 (a - m)) and u = sum 2^(c2 (a - m)) (a - m).  Keeping u relative to the
// max makes the entropy ln s - kappa u / s free of cancellation for sharply peaked rows, and the
// chunk's terms are summed among themselves before they meet the running totals, so 10^5 tiny
// terms are not lost one by one against a total near one.
template <bool kFull>
__device__ __forceinline__ void stats_chunk(const uint32_t (&raw)[32], int nvalid, float c2, float& run_m,
                                            float& run_s, float& run_u) {
  float cmax = -INFINITY;
#pragma unroll
  for (int j = 0; j < 32; ++j)
    if (kFull || j < nvalid) cmax = fmaxf(cmax, __uint_as_float(raw[j]));
  const float m_new = fmaxf(run_m, cmax);
  if (run_s > 0.f) {                                  // move the running sums to the new max
    const float d = run_m - m_new;                    // <= 0
    const float sc = ex2f(d * c2);
    run_u = sc * fmaf(d, run_s, run_u);
    run_s *= sc;
  }
  run_m = m_new;
  float s0 = 0.f, s1 = 0.f, u0 = 0.f, u1 = 0.f;       // two chains for instruction-level parallelism
#pragma unroll
  for (int j = 0; j < 32; j += 2) {
    if (kFull || j < nvalid) {
      const float t = __uint_as_float(raw[j]) - m_new;
      const float e = ex2f(t * c2);
      s0 += e;
      u0 = fmaf(e, t, u0);
    }
    if (kFull || j + 1 < nvalid) {
      const float t = __uint_as_float(raw[j + 1]) - m_new;
      const float e = ex2f(t * c2);
      s1 += e;
      u1 = fmaf(e, t, u1);
    }
  }
  run_s += s0 + s1;
  run_u += u0 + u1;
}

// One 32-column chunk of dz without its one-hot term: -coef * softmax = -sgn(coef) 2^(c2 a + k_row) with
// k_row = log2|coef| - lse log2(e), so an element costs one fused multiply-add and one exponential; the sign
// is applied to the packed bf16 pairs (sign_mask = 0x80008000 for coef > 0, else 0).  Columns at or beyond
// nvalid give zero, and so does a row with coef = 0 (k_row = -inf).
template <bool kFull>
__device__ __forceinline__ void dz_chunk(const uint32_t (&raw)[32], int nvalid, float c2, float k_row,
                                         uint32_t sign_mask, uint32_t* packed) {
#pragma unroll
  for (int j = 0; j < 32; j += 2) {
    float e0 = 0.f, e1 = 0.f;
    if (kFull || j < nvalid) e0 = ex2f(fmaf(__uint_as_float(raw[j]), c2, k_row));
    if (kFull || j + 1 < nvalid) e1 = ex2f(fmaf(__uint_as_float(raw[j + 1]), c2, k_row));
    __nv_bfloat162 h = __floats2bfloat162_rn(e0, e1);
    packed[j >> 1] = *reinterpret_cast<uint32_t*>(&h) ^ sign_mask;
  }
}

// packed[idx >> 1] with its half (idx & 1) replaced by the bf16 `half_bits`, for an index only known at run
// time; predicated moves over registers for the same reason as pick_column.
__device__ __forceinline__ void put_bf16(uint32_t (&packed)[32], int idx, uint32_t half_bits) {
  const int word = idx >> 1;
  const uint32_t keep = (idx & 1) ? 0x0000FFFFu : 0xFFFF0000u;
  const uint32_t ins = (idx & 1) ? (half_bits << 16) : half_bits;
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    const uint32_t cand = (packed[j] & keep) | ins;
    asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.s32 p, %1, %2;\n\t@p mov.b32 %0, %3;\n\t}"
                 : "+r"(packed[j]) : "r"(word), "r"(j), "r"(cand));
  }
}

template <int kMode, int kCta, int kAcc>
__global__ void __launch_bounds__(kUmmaThreads, 1)
umma_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
            const __grid_constant__ CUtensorMap map_c, const UmmaArgs args_in) {
  using namespace ptx;
  UmmaArgs args = args_in;
  if (args.dyn_rows != nullptr) {
    // The number of rows is only known on the device (rows kept by the compaction of the backward):
    // this launch was sized for its capacity and shrinks itself to what is really there.
    int n = *args.dyn_rows - args.dyn_base;
    if (kMode == kModeDW) {
      n = n < 0 ? 0 : (n > args.K ? args.K : n);
      args.K = n;
    } else {
      n = n < 0 ? 0 : (n > args.M ? args.M : n);
      args.M = n;
      args.m_tiles = (n + kBM * kCta - 1) / (kBM * kCta);
    }
  }
  constexpr int kKA = KAtoms<kMode, kCta>::value;
  using Cfg = PipeConfig<kCta, kAcc, kKA>;
  static_assert(kAcc == 1 || (kCta == 2 && (kMode == kModeDHidden || kMode == kModeDW)), "two accumulators: gradient modes, CTA pairs");
  constexpr int kBufs = 2 / kAcc;                          // tensor-memory buffers of kAcc accumulators
  constexpr int kUnitN = kBN * kAcc;                       // output columns per unit
  constexpr bool kPair = (kCta == 2);
  constexpr bool kAmn = ModeTraits<kMode>::a_mn;
  constexpr bool kBmn = ModeTraits<kMode>::b_mn;
  constexpr int kStagesT = Cfg::stages;
  constexpr int kBNcta = kBN / kCta;                       // rows of B that this CTA loads
  constexpr uint32_t kBBytesCta = kBNcta * kBK * 2;
  constexpr uint32_t kAtomBytesCta = kABytes + kAcc * kBBytesCta;
  constexpr uint32_t kStageBytesCta = kKA * kAtomBytesCta;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[kStagesT];
  __shared__ __align__(8) uint64_t bar_empty[kStagesT];
  __shared__ __align__(8) uint64_t bar_tmem_full[2];
  __shared__ __align__(8) uint64_t bar_tmem_empty[2];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  volatile int* abort_p = &abort_flag;
  const int cta_rank = kPair ? (int)cluster_ctarank() : 0;   // 0 = the CTA that issues the pair's MMAs
  const int worker = kPair ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int n_workers = kPair ? (int)(gridDim.x >> 1) : (int)gridDim.x;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < kStagesT; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 1);
      mbar_init(smem_u32(&bar_empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {   // with kAcc = 2 only entry 0 is used
      mbar_init(smem_u32(&bar_tmem_full[b]), 1);
      mbar_init(smem_u32(&bar_tmem_empty[b]), 4 * kCta);   // one arrival per epilogue warp of every CTA
    }
    mbar_fence_init();
    fence_async_proxy();
  }
  if (warp == 0 && lane == 0) {
    prefetch_tensormap(&map_a);
    prefetch_tensormap(&map_b);
  }
  if (warp == 1) {
    if (kPair) {
      tmem_alloc_pair(smem_u32(&tmem_base_slot), kTmemCols);
      tmem_relinquish_pair();
    } else {
      tmem_alloc(smem_u32(&tmem_base_slot), kTmemCols);
      tmem_relinquish();
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (kPair) cluster_sync_all();                           // the peer's barriers exist before anyone signals them
  tc_fence_after_sync();
  const uint32_t tmem_base = tmem_base_slot;

  const int k_blocks = (args.K + kBK * kKA - 1) / (kBK * kKA);
  const int n_units = (k_blocks == 0) ? 0
                      : (kMode == kModeStats) ? args.m_tiles * args.n_split : args.m_tiles * args.n_tiles;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (every CTA)
    // One thread runs the whole loop: nothing in it needs the other lanes, and a warp-wide
    // rendezvous per k-block would sit on the critical path of the ring.
    if (lane == 0) {
      uint32_t stage = 0, phase = 0;
      uint32_t issued = 0;
      const uint32_t full0 = kPair ? map_to_cta(smem_u32(&bar_full[0]), 0) : smem_u32(&bar_full[0]);
      // which operand is worth keeping in L2: the hidden tile that a pair re-reads for every vocabulary
      // tile (statistics, dz), the slices of W / the hidden panel that every pair sweeps (d_hidden, d_W);
      // the dz stream of the gradient kernels is read by four pairs and then dead
      const uint64_t pol_a = make_l2_policy(args.l2_a);
      const uint64_t pol_b = make_l2_policy(args.l2_b);
      for (int unit = worker; unit < n_units; unit += n_workers) {
        int m_tile, n_begin, n_end;
        if (kMode == kModeStats) {
          m_tile = unit / args.n_split;
          stats_tile_range(args, unit % args.n_split, n_begin, n_end);
        } else {
          unit_to_tile(unit, args, m_tile, n_begin);
          n_end = n_begin + 1;
        }
        const int a_row = args.a_mn0 + (m_tile * kCta + cta_rank) * kBM;
        for (int n_tile = n_begin; n_tile < n_end; ++n_tile) {
          const int b_row = args.b_mn0 + n_tile * kUnitN + cta_rank * kBNcta;   // + kBN per further accumulator
          for (int kb = 0; kb < k_blocks; ++kb) {
            if (!mbar_wait_bounded(smem_u32(&bar_empty[stage]), phase ^ 1u, abort_p, kWaitLimitCycles)) goto producer_drain;
            const uint32_t full = full0 + stage * (uint32_t)sizeof(uint64_t);
            if (kPair) {
              // both CTAs' bytes are counted on the issuing CTA's barrier, which alone is armed
              if (cta_rank == 0) mbar_arrive_expect_tx(smem_u32(&bar_full[stage]), 2 * kStageBytesCta);
            } else {
              mbar_arrive_expect_tx(full, kStageBytesCta);
            }
#pragma unroll
            for (int t = 0; t < kKA; ++t) {
              const uint32_t sa = smem_base + stage * kStageBytesCta + t * kAtomBytesCta;
              const uint32_t sb = sa + kABytes;
              const int ka = args.a_k0 + (kb * kKA + t) * kBK, kbb = args.b_k0 + (kb * kKA + t) * kBK;
              if (kPair) {
                if (kAmn) {
#pragma unroll
                  for (int j = 0; j < kBM / 64; ++j) tma_load_2d_pair(sa + j * kChunkBytes, &map_a, full, a_row + j * 64, ka, pol_a);
                } else {
                  tma_load_2d_pair(sa, &map_a, full, ka, a_row, pol_a);
                }
#pragma unroll
                for (int q = 0; q < kAcc; ++q) {
                  if (kBmn) {
#pragma unroll
                    for (int j = 0; j < kBNcta / 64; ++j)
                      tma_load_2d_pair(sb + q * kBBytesCta + j * kChunkBytes, &map_b, full, b_row + q * kBN + j * 64, kbb, pol_b);
                  } else {
                    tma_load_2d_pair(sb + q * kBBytesCta, &map_b, full, kbb, b_row + q * kBN, pol_b);
                  }
                }
              } else {
                if (kAmn) {
#pragma unroll
                  for (int j = 0; j < kBM / 64; ++j) tma_load_2d(sa + j * kChunkBytes, &map_a, full, a_row + j * 64, ka);
                } else {
                  tma_load_2d(sa, &map_a, full, ka, a_row);
                }
                if (kBmn) {
#pragma unroll
                  for (int j = 0; j < kBNcta / 64; ++j) tma_load_2d(sb + j * kChunkBytes, &map_b, full, b_row + j * 64, kbb);
                } else {
                  tma_load_2d(sb, &map_b, full, kbb, b_row);
                }
              }
            }
            ++issued;
            if (++stage == kStagesT) { stage = 0; phase ^= 1u; }
          }
        }
      }
      // tail: every slot this CTA filled has been released again, i.e. the MMAs that read this CTA's
      // shared memory are done and no release signal is still on its way to this CTA
      {
        const uint32_t n_tail = issued < (uint32_t)kStagesT ? issued : (uint32_t)kStagesT;
        for (uint32_t b = 0; b < n_tail; ++b) {
          if (!mbar_wait_bounded(smem_u32(&bar_empty[stage]), phase ^ 1u, abort_p, kWaitLimitCycles)) goto producer_drain;
          if (++stage == kStagesT) { stage = 0; phase ^= 1u; }
        }
      }
    producer_drain:
      if (*abort_p && cta_rank == 0) {
        // give the copies still in flight a bounded time to land before the block goes away
        const uint32_t n_back = issued < (uint32_t)kStagesT ? issued : (uint32_t)kStagesT;
        for (uint32_t b = 0; b < n_back; ++b) {
          if (stage == 0) { stage = kStagesT; phase ^= 1u; }
          --stage;
          const long long t0 = clock64();
          while (!mbar_try_wait(smem_u32(&bar_full[stage]), phase) && clock64() - t0 < 200000000LL) {
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (rank 0 of a pair)
    // One thread, and as little as possible between two tcgen05.mma: descriptors advance by
    // constants, and the barrier of the next stage is polled right after this stage's MMAs are
    // queued, so that its latency runs under them.
    if (cta_rank == 0 && lane == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(kBM * kCta, kBN, kAmn ? 1 : 0, kBmn ? 1 : 0);
      // K-major: 16 elements = 32 bytes along the swizzled row; MN-major: 16 k-rows of 128 bytes
      constexpr uint64_t a_step = (kAmn ? kUmmaK * 128 : kUmmaK * 2) >> 4;
      constexpr uint64_t b_step = (kBmn ? kUmmaK * 128 : kUmmaK * 2) >> 4;
      constexpr uint64_t stage_step = kStageBytesCta >> 4;
      constexpr uint64_t atom_step = kAtomBytesCta >> 4;
      const uint64_t da_base = kAmn ? make_smem_desc(smem_base, kChunkBytes, 1024) : make_smem_desc(smem_base, 16, 1024);
      const uint64_t db_base = kBmn ? make_smem_desc(smem_base + kABytes, kChunkBytes, 1024)
                                    : make_smem_desc(smem_base + kABytes, 16, 1024);
      uint32_t stage = 0, phase = 0;
      uint32_t acc_iter = 0;
      bool ready = false;
      for (int unit = worker; unit < n_units; unit += n_workers) {
        int n_tiles_here = 1;
        if (kMode == kModeStats) {
          int n_begin, n_end;
          stats_tile_range(args, unit % args.n_split, n_begin, n_end);
          n_tiles_here = n_end - n_begin;
        }
        for (int t = 0; t < n_tiles_here; ++t, ++acc_iter) {
          const uint32_t buf = acc_iter % kBufs;
          const uint32_t buf_phase = (acc_iter / kBufs) & 1u;
          if (!mbar_wait_bounded(smem_u32(&bar_tmem_empty[buf]), buf_phase ^ 1u, abort_p, kWaitLimitCycles)) goto mma_done;
          const uint32_t tmem_d = tmem_base + buf * kUnitN;
          for (int kb = 0; kb < k_blocks; ++kb) {
            if (!ready && !mbar_wait_bounded(smem_u32(&bar_full[stage]), phase, abort_p, kWaitLimitCycles)) goto mma_done;
            tc_fence_after_sync();
            const uint64_t da = da_base + stage * stage_step;
            const uint64_t db = db_base + stage * stage_step;
#pragma unroll
            for (int t = 0; t < kKA; ++t) {
#pragma unroll
              for (int q = 0; q < kAcc; ++q) {
#pragma unroll
                for (int k = 0; k < kBK / kUmmaK; ++k) {
                  const uint64_t daq = da + t * atom_step + k * a_step;
                  const uint64_t dbq = db + t * atom_step + q * (uint64_t)(kBBytesCta >> 4) + k * b_step;
                  const uint32_t acc = (kb > 0 || t > 0 || k > 0) ? 1u : 0u;
                  if (kPair) umma_bf16_pair(tmem_d + q * kBN, daq, dbq, idesc, acc);
                  else umma_bf16(tmem_d + q * kBN, daq, dbq, idesc, acc);
                }
              }
            }
            if (kPair) {
              umma_commit_pair(smem_u32(&bar_empty[stage]), 3);                        // frees the slot in both CTAs
              if (kb == k_blocks - 1) umma_commit_pair(smem_u32(&bar_tmem_full[buf]), 3);  // accumulator ready
            } else {
              umma_commit(smem_u32(&bar_empty[stage]));
              if (kb == k_blocks - 1) umma_commit(smem_u32(&bar_tmem_full[buf]));
            }
            if (++stage == kStagesT) { stage = 0; phase ^= 1u; }
            ready = mbar_try_wait(smem_u32(&bar_full[stage]), phase);
          }
        }
      }
    mma_done:;
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5, every CTA)
    const int quarter = warp & 3;                       // tensor-memory lanes 32 * quarter ..
    const int row_in_tile = quarter * 32 + lane;
    const float c2 = args.kappa * 1.4426950408889634f;  // exp(kappa a) = 2^(c2 a)
    uint32_t acc_iter = 0;
    // The dz and d_W epilogues alternate between two staging tiles and only ever wait until at most ONE
    // tile copy is still reading shared memory, so the tile must be chosen by a count of the copies
    // issued that runs across accumulators and units: a last column tile that ends after an odd number
    // of copies would otherwise hand the next unit the tile whose copy is the one still in flight.
    uint32_t stage_iter = 0;
    for (int unit = worker; unit < n_units; unit += n_workers) {
      int m_tile, n_begin, n_end, split = 0;
      if (kMode == kModeStats) {
        m_tile = unit / args.n_split;
        split = unit % args.n_split;
        stats_tile_range(args, split, n_begin, n_end);
      } else {
        unit_to_tile(unit, args, m_tile, n_begin);
        n_end = n_begin + 1;
      }
      const int row = (m_tile * kCta + cta_rank) * kBM + row_in_tile;   // row within this launch's M extent
      const bool row_ok = row < args.M;
      const int grow = args.row0 + row;                 // global token / vocabulary row

      // per-row state
      float run_m = -INFINITY, run_s = 0.f, run_u = 0.f;
      int y = -1;
      float coef = 0.f, lse2 = 0.f;
      if (kMode == kModeStats || kMode == kModeDz) {
        if (row_ok) {
          y = args.targets[grow];
          if (y < 0 || y >= args.N) {
            if (kMode == kModeStats) atomicOr(args.status, kStatusBadTarget);
            y = y < 0 ? 0 : args.N - 1;
          }
        }
      }
      if (kMode == kModeStats && args.resume && row_ok) {  // continue the sweep the launch before left off
        const float4 p = args.partials[(size_t)split * args.T_total + grow];
        run_m = p.x; run_s = p.y; run_u = p.z;
      }
      float k_row = -INFINITY;                          // kModeDz: log2|coef| - lse log2(e); -inf gives a zero row
      uint32_t sign_mask = 0u;
      if (kMode == kModeDz) {
        if (row_ok) {
          const float gl = args.grad_loss ? *args.grad_loss : 1.f;
          coef = args.kappa * gl * args.grad_coef[grow];
          lse2 = args.lse[grow] * 1.4426950408889634f;
          if (coef != 0.f) k_row = log2f(fabsf(coef)) - lse2;
          sign_mask = coef > 0.f ? 0x80008000u : 0u;
        }
      }

      for (int n_tile = n_begin; n_tile < n_end; ++n_tile, ++acc_iter) {
        const uint32_t buf = acc_iter % kBufs;
        const uint32_t buf_phase = (acc_iter / kBufs) & 1u;
        const int col_base = n_tile * kUnitN;
        // The give-up decision is taken by the 128 epilogue threads together: a thread that saw the wait
        // complete while another saw the abort flag would otherwise go on alone to warp-wide tensor-memory
        // loads and to the epilogue barrier, which the others never reach.
        if (!epilogue_all(mbar_wait_bounded<true>(smem_u32(&bar_tmem_full[buf]), buf_phase, abort_p, kWaitLimitCycles)))
          goto role_done;
        tc_fence_after_sync();
        const uint32_t taddr = tmem_base + buf * kUnitN + ((uint32_t)(quarter * 32) << 16);
        if (kMode == kModeDz) {
          // 64 columns (one 128-byte row of bf16) at a time: two accumulator chunks -> packed registers ->
          // swizzled staging tile in shared memory -> one TMA store of 128 rows x 128 bytes, so that the
          // panel is written in whole lines by the copy engine instead of 16 bytes a thread
          const int tile_row = (m_tile * kCta + cta_rank) * kBM;
          const bool issuer = (threadIdx.x == 64);             // first thread of the epilogue warps
#pragma unroll 1
          for (int g = 0; g < kUnitN / 64; ++g) {
            const int col0 = col_base + g * 64;
            if (col0 >= args.dz_cols) break;
            uint32_t raw0[32], raw1[32];
            tmem_ld_32x32(taddr + g * 64, raw0);
            tmem_ld_32x32(taddr + g * 64 + 32, raw1);
            tmem_ld_wait();
            uint32_t packed[32];
            const int nv0 = args.N - col0, nv1 = args.N - col0 - 32;
            if (nv0 >= 32) dz_chunk<true>(raw0, 32, c2, k_row, sign_mask, packed);
            else dz_chunk<false>(raw0, nv0, c2, k_row, sign_mask, packed);
            if (nv1 >= 32) dz_chunk<true>(raw1, 32, c2, k_row, sign_mask, packed + 16);
            else dz_chunk<false>(raw1, nv1, c2, k_row, sign_mask, packed + 16);
            if (row_ok && y >= col0 && y < col0 + 64) {        // the one-hot term: coef (1 - p_y) at the target column
              const int idx = y - col0;
              const float ay = idx < 32 ? pick_column(raw0, idx) : pick_column(raw1, idx - 32);
              const float vy = coef * (1.f - ex2f(fmaf(ay, c2, -lse2)));
              const __nv_bfloat16 hv = __float2bfloat16_rn(vy);
              put_bf16(packed, idx, (uint32_t)(*reinterpret_cast<const uint16_t*>(&hv)));
            }
            const uint32_t out_buf = smem_base + kStagesT * kStageBytesCta + (stage_iter++ & 1u) * kOutStageBytes;
            if (issuer) bulk_wait_read_le1();                  // the copy that last read this staging tile is done with it
            epilogue_bar_sync();
            const uint32_t row_addr = out_buf + (uint32_t)row_in_tile * 128u;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              const uint32_t dst = row_addr + ((uint32_t)(q ^ (row_in_tile & 7)) << 4);
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(packed[4 * q]), "r"(packed[4 * q + 1]),
                           "r"(packed[4 * q + 2]), "r"(packed[4 * q + 3])
                           : "memory");
            }
            fence_async_proxy();
            epilogue_bar_sync();
            if (issuer) {
              tma_store_2d(&map_c, out_buf, col0, tile_row);   // rows past the panel's capacity are clipped
              bulk_commit_group();
            }
          }
        }
#pragma unroll 1
        for (int c = 0; kMode != kModeDz && c < kUnitN / 32; ++c) {
          const int col0 = col_base + c * 32;
          if (col0 >= args.N) break;                           // whole chunk beyond the valid columns
          const int nvalid = min(32, args.N - col0);
          uint32_t raw[32];
          tmem_ld_32x32(taddr + c * 32, raw);
          tmem_ld_wait();

          if (kMode == kModeStats) {
            if (nvalid >= 32) stats_chunk<true>(raw, 32, c2, run_m, run_s, run_u);
            else stats_chunk<false>(raw, nvalid, c2, run_m, run_s, run_u);
            if (row_ok && y >= col0 && y < col0 + 32) {
              args.acc_y[grow] = pick_column(raw, y - col0);
            }
          } else if (kMode == kModeDHidden) {
            if (row_ok) {
              uint32_t packed[16];
#pragma unroll
              for (int j = 0; j < 32; j += 2) {
                __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(raw[j]), __uint_as_float(raw[j + 1]));
                packed[j >> 1] = *reinterpret_cast<uint32_t*>(&h);
              }
              uint4* dst = reinterpret_cast<uint4*>(args.d_hidden + (size_t)grow * args.out_ld + col0);
#pragma unroll
              for (int q = 0; q < 4; ++q)
                if (q * 8 < nvalid) dst[q] = make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
            }
          } else {  // kModeDW: swizzled staging tile, then one TMA store (first panel) or reduce-add
            const uint32_t out_buf = smem_base + kStagesT * kStageBytesCta + (stage_iter++ & 1u) * kOutStageBytes;
            const bool issuer = (threadIdx.x == 64);             // first thread of the epilogue warps
            if (issuer) bulk_wait_read_le1();                    // the copy that last read this tile is done with it
            epilogue_bar_sync();
            const uint32_t row_addr = out_buf + (uint32_t)row_in_tile * 128u;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              const uint32_t dst = row_addr + ((uint32_t)(q ^ (row_in_tile & 7)) << 4);
              asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(raw[4 * q]), "r"(raw[4 * q + 1]),
                           "r"(raw[4 * q + 2]), "r"(raw[4 * q + 3])
                           : "memory");
            }
            fence_async_proxy();
            epilogue_bar_sync();
            if (issuer) {
              const int tile_row = (m_tile * kCta + cta_rank) * kBM;      // rows past M never reach memory
              if (tile_row < args.M) {
                if (args.accumulate) tma_reduce_add_2d(&map_c, out_buf, col0, args.row0 + tile_row);
                else tma_store_2d(&map_c, out_buf, col0, args.row0 + tile_row);
              }
              bulk_commit_group();
            }
          }
        }
        // accumulator drained: hand the buffer back to the MMA warp (of rank 0)
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) {
          if (kPair) mbar_arrive_cluster(map_to_cta(smem_u32(&bar_tmem_empty[buf]), 0));
          else mbar_arrive(smem_u32(&bar_tmem_empty[buf]));
        }
      }

      if (kMode == kModeStats && row_ok)
        args.partials[(size_t)split * args.T_total + grow] = make_float4(run_m, run_s, run_u, 0.f);
    }
  }

role_done:
  if ((kMode == kModeDW || kMode == kModeDz) && threadIdx.x == 64) bulk_wait_all();   // the tile copies have left shared memory and landed
  if (*abort_p && lane == 0) atomicOr(args.status, kStatusTimeout);
  tc_fence_before_sync();
  __syncthreads();
  if (kPair) cluster_sync_all();       // neither CTA leaves while the other may still signal its barriers
  if (warp == 1) {
    tc_fence_after_sync();
    if (kPair) tmem_dealloc_pair(tmem_base, kTmemCols);
    else tmem_dealloc(tmem_base, kTmemCols);
  }
}

// The bounded wait on its own: one block, one mbarrier on which nobody ever arrives, no copy and no tensor
// memory in flight.  The wait gives up after limit_cycles, the kernel records the timeout in the status word
// and returns normally -- the way umma_kernel reports a stall, exercised without stalling anything.
__global__ void bounded_wait_selftest_kernel(long long limit_cycles, int* status) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    ptx::mbar_fence_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    volatile int* abort_p = &abort_flag;
    const bool done = ptx::mbar_wait_bounded(ptx::smem_u32(&bar), 0u, abort_p, limit_cycles);
    if (!done) atomicOr(status, kStatusTimeout);
  }
}

}  // namespace ulorl
