// C ABI of the UloRL token-loss library: argument validation, workspace carve-up, tensor-map
// construction and kernel launches.  No device allocation and no synchronisation (except
// ulorl_check_status and ulorl_kernel_timing_end).  What the process keeps between calls is listed
// in ulorl.h ("State kept by the library") and is created under g_setup_mutex.
#include <atomic>
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <functional>
#include <mutex>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "common.cuh"
#include "elementwise.cuh"
#include "simt.cuh"
#include "umma_gemm.cuh"

namespace ulorl {

static std::atomic<long long> g_launches{0};
constexpr size_t kStatsHiddenBudget = 40u << 20;   // live hidden tiles of the statistics kernel that L2 keeps beside W
constexpr int kMaxDevices = 64;            // per-device set-up tables
constexpr int kFallbackSMs = 148;         // B200; used for the plan when no device can be asked
constexpr int kDefaultPanelTensor = 16384;       // single-CTA kernels
constexpr int kDefaultPanelSimt = 1024;
constexpr int kRasterGroup = 16;          // dz: row tiles per raster group (m fastest inside a group)
constexpr int kGradRasterGroup = 1;       // d_hidden, d_W: column blocks of one row tile run side by side, so its A stream is read once

// Everything the library creates lazily and keeps (per-device tables, events, streams, the driver
// entry point) is created and looked up under this one mutex, so that first calls from several host
// threads do not race.
static std::mutex g_setup_mutex;

// Multiprocessor count of the current device (asked once per device); kFallbackSMs when there is
// no device to ask, so that ulorl_workspace_bytes stays usable on a host without a GPU.
static int device_sm_count() {
  static int sms[kMaxDevices] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    (void)cudaGetLastError();
    return kFallbackSMs;
  }
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (sms[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
      (void)cudaGetLastError();
      return kFallbackSMs;
    }
    sms[dev] = n;
  }
  return sms[dev];
}

// A named range on the calling host thread for the time its launches are being queued: a timeline tool
// attached to the process shows which call, pass and panel a kernel belongs to.  Without a tool attached
// the calls do nothing.
struct TraceRange {
  explicit TraceRange(const char* name) { nvtxRangePushA(name); }
  ~TraceRange() { nvtxRangePop(); }
  TraceRange(const TraceRange&) = delete;
  TraceRange& operator=(const TraceRange&) = delete;
};

struct Plan {
  bool tensor;            // tensor-core path (bf16) or SIMT path
  int cta;                // CTAs per tcgen05.mma: 2 (a CTA pair per 256 x 256 tile) or 1 (ULORL_PATH_TENSOR_1CTA)
  int sms;                // multiprocessors the persistent kernels are spread over
  int n_split, tiles_per_split;
  int panel_tokens;
  size_t dz_ld;           // leading dimension of the dz panel (elements)
  size_t off_status, off_batch_mean, off_seq_sum, off_partials, off_acc_y, off_decide, off_dz, total;
  bool compact;           // backward on the rows with a non-zero coefficient only (tensor path)
  int compact_blocks;     // blocks of 256 tokens of the compaction kernels
  size_t t_pad;           // rows of the compacted buffers
  size_t off_n_active, off_blk_count, off_blk_offset, off_position, off_targets_c, off_lse_c, off_coef_c,
      off_hidden_c, off_dh_c;
  bool dw_bf16;           // d_W leaves as bf16: the float32 sum over tokens is kept at off_dw_acc
  size_t off_dw_acc;
  int decide_blocks;
};

static bool use_tensor_path(const ulorl_params_t* p) {
  if (p->kernel_path == ULORL_PATH_SIMT) return false;
  return p->dtype == ULORL_BF16;
}

static int validate_params(const ulorl_params_t* p) {
  if (!p) return ULORL_ERR_INVALID_ARG;
  if (p->T < 0 || p->H <= 0 || p->V <= 0 || p->num_seqs < 0) return ULORL_ERR_INVALID_ARG;
  if (p->T > 0 && p->num_seqs == 0) return ULORL_ERR_INVALID_ARG;
  if (p->dtype != ULORL_F32 && p->dtype != ULORL_BF16) return ULORL_ERR_UNSUPPORTED;
  if (p->is_mode != ULORL_IS_SAIS && p->is_mode != ULORL_IS_POIS) return ULORL_ERR_INVALID_ARG;
  if (p->mpt_mode < ULORL_MPT_OFF || p->mpt_mode > ULORL_MPT_DYNAMIC) return ULORL_ERR_INVALID_ARG;
  if (p->ent_scope < ULORL_ENT_PER_SEQ || p->ent_scope > ULORL_ENT_SUPPLIED) return ULORL_ERR_INVALID_ARG;
  if (p->loss_norm < ULORL_NORM_TOKENS || p->loss_norm > ULORL_NORM_SEQUENCE || p->norm_seqs < 0)
    return ULORL_ERR_INVALID_ARG;
  if (p->kernel_path < ULORL_PATH_AUTO || p->kernel_path > ULORL_PATH_TENSOR_1CTA) return ULORL_ERR_INVALID_ARG;
  if ((p->kernel_path == ULORL_PATH_TENSOR || p->kernel_path == ULORL_PATH_TENSOR_1CTA) && p->dtype != ULORL_BF16)
    return ULORL_ERR_UNSUPPORTED;
  if (!(p->inv_temperature > 0.f) || !std::isfinite(p->inv_temperature)) return ULORL_ERR_INVALID_ARG;
  if (!(p->clip_eps_low >= 0.f) || !(p->clip_eps_high >= 0.f) || p->clip_eps_low > 1.f) return ULORL_ERR_INVALID_ARG;
  if (!(p->mpt_tau > 0.f) || p->mpt_tau > 1.f) return ULORL_ERR_INVALID_ARG;
  if (p->norm_tokens < 0 || p->bwd_panel_tokens < 0) return ULORL_ERR_INVALID_ARG;
  if (p->compact_rows != 0 && p->compact_rows != 1) return ULORL_ERR_INVALID_ARG;
  if (p->dw_dtype != ULORL_F32 && p->dw_dtype != ULORL_BF16) return ULORL_ERR_INVALID_ARG;
  if (!(p->kl_beta >= 0.f) || !std::isfinite(p->kl_beta)) return ULORL_ERR_INVALID_ARG;
  if (p->H % 8 != 0) return ULORL_ERR_UNSUPPORTED;
  // the exact integer entropy sums hold 2^29 nats; no token's entropy exceeds ln V
  if ((double)p->T * std::log((double)p->V + 1.0) >= kEntropyFixCapacity) return ULORL_ERR_UNSUPPORTED;
  return ULORL_OK;
}

static Plan make_plan(const ulorl_params_t* p) {
  Plan pl{};
  pl.tensor = use_tensor_path(p);
  pl.cta = p->kernel_path == ULORL_PATH_TENSOR_1CTA ? 1 : 2;
  pl.sms = device_sm_count();
  const int T = p->T, V = p->V;
  const int tile_m = pl.tensor ? kBM * pl.cta : kSimtTile;
  const int tile_n = pl.tensor ? kBN : kSimtTile;
  const int workers = pl.tensor ? std::max(1, pl.sms / pl.cta) : pl.sms;
  const int m_tiles = (T + tile_m - 1) / tile_m;
  const int n_tiles = (V + tile_n - 1) / tile_n;
  int want = m_tiles > 0 ? (8 * workers + m_tiles - 1) / m_tiles : 1;
  want = want < 1 ? 1 : want;
  want = want > kMaxSplits ? kMaxSplits : want;
  want = want > n_tiles ? n_tiles : want;
  if (pl.tensor && m_tiles > 0) {
    // Units (row tile, split) are dealt round-robin, splits fastest, to the persistent workers: at any time
    // workers / splits row tiles are live, each sweeping its splits' slices of W side by side.  Their hidden
    // tiles are re-read from L2 for every vocabulary tile, so they must fit beside the W streams -- few
    // splits would not do (at H = 2048 one split means 74 MB of live hidden tiles) -- while every further
    // split is one more pass of all of W through HBM per wave and one more stream for L2 to hold.  So:
    // the smallest count that keeps the live hidden tiles within kStatsHiddenBudget, then the best of the
    // next few for wave quantisation (time = waves of units x vocabulary tiles per split).
    const size_t live_bytes = (size_t)workers * (size_t)tile_m * (size_t)p->H * 2;
    const int fit = (int)((live_bytes + kStatsHiddenBudget - 1) / kStatsHiddenBudget);
    if (fit > want) want = fit > n_tiles ? n_tiles : (fit > kMaxSplits ? kMaxSplits : fit);
    auto cost_of = [&](int s) {
      const int tps = (n_tiles + s - 1) / s;
      const int s_eff = (n_tiles + tps - 1) / tps;
      const long waves = ((long)m_tiles * s_eff + workers - 1) / workers;
      return waves * tps;
    };
    const int s_max = std::min(std::min(want + 3, kMaxSplits), n_tiles);
    long best_cost = cost_of(want);
    for (int s = want + 1; s <= s_max; ++s) best_cost = cost_of(s) < best_cost ? cost_of(s) : best_cost;
    // the fewest splits within one percent of the best: a split more costs HBM passes over W, not time
    for (int s = want; s <= s_max; ++s)
      if (cost_of(s) * 100 <= best_cost * 101) { want = s; break; }
  }
  pl.tiles_per_split = (n_tiles + want - 1) / want;
  pl.n_split = (n_tiles + pl.tiles_per_split - 1) / pl.tiles_per_split;
  int panel = p->bwd_panel_tokens > 0 ? p->bwd_panel_tokens
                                      : (pl.tensor ? (pl.cta == 2 ? workers * kBM * 2 : kDefaultPanelTensor) : kDefaultPanelSimt);
  const int panel_unit = pl.tensor ? kBM * pl.cta : kBM;   // whole row tiles: the dz kernel zero-fills to the tile end
  panel = (panel + panel_unit - 1) / panel_unit * panel_unit;
  const int t_round = (T + panel_unit - 1) / panel_unit * panel_unit;
  if (panel > t_round) panel = t_round;
  if (panel < panel_unit) panel = panel_unit;
  pl.panel_tokens = panel;
  pl.dz_ld = pl.tensor ? align_up((size_t)V, 64) : (size_t)V;
  pl.decide_blocks = (T + kDecideTokens - 1) / kDecideTokens;
  size_t off = 0;
  pl.off_status = off;      off += 256;
  pl.off_batch_mean = pl.off_status + 16;
  pl.off_seq_sum = off;     off = align_up(off + sizeof(long long) * (size_t)(p->num_seqs > 0 ? p->num_seqs : 1), 256);
  pl.off_partials = off;    off = align_up(off + sizeof(float4) * (size_t)pl.n_split * (size_t)(T > 0 ? T : 1), 256);
  pl.off_acc_y = off;       off = align_up(off + sizeof(float) * (size_t)(T > 0 ? T : 1), 256);
  pl.off_decide = off;      off = align_up(off + sizeof(DecidePartial) * (size_t)(pl.decide_blocks > 0 ? pl.decide_blocks : 1), 1024);
  pl.off_dz = off;          off = align_up(off + (size_t)panel * pl.dz_ld * (pl.tensor ? 2 : 4), 1024);
  pl.compact = pl.tensor && p->compact_rows != 0;
  pl.compact_blocks = (T + kCompactThreads - 1) / kCompactThreads;
  pl.t_pad = align_up((size_t)(T > 0 ? T : 1), 256) + 256;
  if (pl.compact) {
    const size_t nb = (size_t)(pl.compact_blocks > 0 ? pl.compact_blocks : 1);
    pl.off_n_active = off;   off += 256;
    pl.off_blk_count = off;  off = align_up(off + 4 * nb, 256);
    pl.off_blk_offset = off; off = align_up(off + 4 * nb, 256);
    pl.off_position = off;   off = align_up(off + 4 * pl.t_pad, 256);
    pl.off_targets_c = off;  off = align_up(off + 4 * pl.t_pad, 256);
    pl.off_lse_c = off;      off = align_up(off + 4 * pl.t_pad, 256);
    pl.off_coef_c = off;     off = align_up(off + 4 * pl.t_pad, 256);
    pl.off_hidden_c = off;   off = align_up(off + 2 * pl.t_pad * (size_t)p->H, 1024);
    pl.off_dh_c = off;       off = align_up(off + 2 * pl.t_pad * (size_t)p->H, 1024);
  }
  pl.dw_bf16 = p->dw_dtype == ULORL_BF16;
  if (pl.dw_bf16) {
    pl.off_dw_acc = off;
    off = align_up(off + sizeof(float) * (size_t)V * (size_t)p->H, 1024);
  }
  pl.total = off;
  return pl;
}

static int check_launch() {
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    std::fprintf(stderr, "ulorl: CUDA launch error: %s\n", cudaGetErrorString(e));
    return ULORL_ERR_CUDA;
  }
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return ULORL_OK;
}

#define ULORL_LAUNCH_CHECK()                    \
  do {                                          \
    const int _st = check_launch();             \
    if (_st != ULORL_OK) return _st;            \
  } while (0)

// ------------------------------------------------------------------ tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!tried) {
    tried = true;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// bf16 matrix [rows][cols] with `ld` elements between rows; box = box_cols x box_rows, 128-byte swizzle,
// out-of-range elements read as zero.
static int make_map(CUtensorMap* map, CUtensorMapDataType dtype, size_t elem_bytes, const void* base, uint64_t rows,
                    uint64_t cols, uint64_t ld, uint32_t box_cols, uint32_t box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return ULORL_ERR_CUDA;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {ld * elem_bytes};
  const cuuint32_t box[2] = {box_cols, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(map, dtype, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    std::fprintf(stderr, "ulorl: cuTensorMapEncodeTiled failed (%d)\n", (int)r);
    return ULORL_ERR_CUDA;
  }
  return ULORL_OK;
}

static int make_map_bf16(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint64_t ld,
                         uint32_t box_cols, uint32_t box_rows) {
  return make_map(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, rows, cols, ld, box_cols, box_rows);
}

// Optional per-kernel timing of the tensor-core launches: when enabled, an event pair brackets
// every launch on its stream, so durations are measured inside whatever region the caller times.
struct KernelTiming {
  std::atomic<bool> enabled{false};
  std::vector<cudaEvent_t> ev[4];   // start/stop pairs per kernel kind
  size_t used[4] = {0, 0, 0, 0};
};
static KernelTiming g_timing;

static cudaEvent_t timing_event(int kind) {
  KernelTiming& t = g_timing;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (t.used[kind] == t.ev[kind].size()) {
    cudaEvent_t e;
    if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
    t.ev[kind].push_back(e);
  }
  return t.ev[kind][t.used[kind]++];
}

template <int kMode, int kCta, int kAcc>
static int launch_umma_impl(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const UmmaArgs& a,
                            int num_sms, cudaStream_t stream) {
  // the shared-memory opt-in is a property of the function on ONE device: set up once per device
  static bool opted_in[kMaxDevices] = {};
  constexpr size_t smem = PipeConfig<kCta, kAcc, KAtoms<kMode, kCta>::value>::smem_bytes;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ULORL_ERR_CUDA;
  {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!opted_in[dev]) {
      if (cudaFuncSetAttribute(umma_kernel<kMode, kCta, kAcc>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               (int)smem) != cudaSuccess)
        return ULORL_ERR_CUDA;
      opted_in[dev] = true;
    }
  }
  const int units = (kMode == kModeStats) ? a.m_tiles * a.n_split : a.m_tiles * a.n_tiles;
  if (units <= 0) return ULORL_OK;
  if (kMode != kModeStats && a.group_m <= 0) return ULORL_ERR_INVALID_ARG;
  // L2 policy of the tile loads: keep what is re-read for long (the hidden tile of the two logits
  // kernels, the slices of W / of the hidden panel that every pair sweeps in the gradient kernels).
  // The statistics kernel marks its W stream too: it starts in an L2 that the gradient kernels of the
  // step before left full of evict-last lines, which unmarked loads cannot displace.
  UmmaArgs a2 = a;
  a2.l2_a = (kMode == kModeStats || kMode == kModeDz) ? ptx::kL2EvictLast : ptx::kL2Normal;
  a2.l2_b = (kMode == kModeStats || kMode == kModeDHidden || kMode == kModeDW) ? ptx::kL2EvictLast : ptx::kL2Normal;
  const int max_workers = num_sms / kCta;
  const int workers = units < max_workers ? units : max_workers;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  if (g_timing.enabled.load(std::memory_order_relaxed)) {
    e0 = timing_event(kMode);
    e1 = timing_event(kMode);
    if (e0 && e1) cudaEventRecord(e0, stream);
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(workers * kCta), 1, 1);
  cfg.blockDim = dim3(kUmmaThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kCta;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t le = cudaLaunchKernelEx(&cfg, umma_kernel<kMode, kCta, kAcc>, ma, mb, mc, a2);
  if (le != cudaSuccess) {
    std::fprintf(stderr, "ulorl: cudaLaunchKernelEx failed: %s\n", cudaGetErrorString(le));
    return ULORL_ERR_CUDA;
  }
  const int st = check_launch();
  if (e0 && e1) cudaEventRecord(e1, stream);
  return st;
}

// Accumulators per unit: the gradient contractions on CTA pairs use two (256 x 512 outputs a unit).
template <int kMode>
static constexpr int acc_per_unit_pair() { return (kMode == kModeDHidden || kMode == kModeDW) ? 2 : 1; }
static int grad_unit_cols(const Plan& pl) { return pl.cta == 2 ? 2 * kBN : kBN; }

// mc is the output tensor map of the dz and d_W kernels; the other kernels get any valid map and ignore it.
template <int kMode>
static int launch_umma(const Plan& pl, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc,
                       const UmmaArgs& a, cudaStream_t stream) {
  return pl.cta == 2 ? launch_umma_impl<kMode, 2, acc_per_unit_pair<kMode>()>(ma, mb, mc, a, pl.sms, stream)
                     : launch_umma_impl<kMode, 1, 1>(ma, mb, mc, a, pl.sms, stream);
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ------------------------------------------------------------------ decision stage
static DecideConsts make_decide_consts(const ulorl_params_t* p) {
  DecideConsts c{};
  c.ln_tau = (float)std::log((double)p->mpt_tau);
  c.ln_hi = (float)std::log1p((double)p->clip_eps_high);
  c.ln_lo = p->clip_eps_low < 1.f ? (float)std::log1p(-(double)p->clip_eps_low) : -INFINITY;
  c.sigma = p->entropy_target;
  c.eps_lo = (double)p->clip_eps_low;
  c.eps_hi = (double)p->clip_eps_high;
  double N = p->norm_tokens > 0 ? (double)p->norm_tokens : (double)p->T;
  if (p->loss_norm == ULORL_NORM_SEQUENCE) N = p->norm_seqs > 0 ? (double)p->norm_seqs : (double)p->num_seqs;
  c.inv_N = N > 0 ? 1.0 / N : 0.0;
  c.is_mode = p->is_mode;
  c.mpt_mode = p->mpt_mode;
  c.ent_scope = p->ent_scope;
  c.adv_per_token = p->adv_per_token;
  c.current_version = p->current_version;
  c.loss_norm = p->loss_norm;
  c.kl_beta = (double)p->kl_beta;
  return c;
}

static int run_decide(const ulorl_params_t* p, const Plan& pl, const float* logp, const float* entropy,
                      const float* old_logp, const float* ref_logp, const int32_t* segment_version,
                      const float* advantages,
                      const int32_t* seq_offsets, const float* entropy_supplied, float* grad_coef, uint8_t* flags,
                      float* seq_entropy, float* loss, void* stats, uint8_t* ws, cudaStream_t stream) {
  TraceRange trace("ulorl decision stage");
  const int T = p->T, S = p->num_seqs;
  int* status = reinterpret_cast<int*>(ws + pl.off_status);
  float* batch_mean = reinterpret_cast<float*>(ws + pl.off_batch_mean);
  long long* seq_sum = reinterpret_cast<long long*>(ws + pl.off_seq_sum);
  DecidePartial* partials = reinterpret_cast<DecidePartial*>(ws + pl.off_decide);
  // the gate needs a float array of per-sequence means even when the caller does not want it back
  float* seq_ent_out = seq_entropy;
  if (cudaMemsetAsync(seq_sum, 0, sizeof(long long) * (size_t)S, stream) != cudaSuccess) return ULORL_ERR_CUDA;
  seq_entropy_sum_kernel<<<(T + kSeqChunk - 1) / kSeqChunk, kSeqThreads, 0, stream>>>(S, T, seq_offsets, entropy, seq_sum);
  ULORL_LAUNCH_CHECK();
  seq_entropy_mean_kernel<<<1, kSeqThreads, 0, stream>>>(S, T, seq_offsets, seq_sum, seq_ent_out, batch_mean, status);
  ULORL_LAUNCH_CHECK();
  const DecideConsts c = make_decide_consts(p);
  const float* gate = (p->ent_scope == ULORL_ENT_SUPPLIED) ? entropy_supplied : seq_ent_out;
  // 128-bit accesses when every per-token array starts on a 16-byte boundary (flags: 4 bytes)
  auto al = [](const void* p, uintptr_t a) { return p == nullptr || (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; };
  const bool vec = al(logp, 16) && al(old_logp, 16) && al(segment_version, 16) && al(grad_coef, 16) && al(flags, 4) &&
                   (!p->adv_per_token || al(advantages, 16)) && (!(p->kl_beta > 0.f) || al(ref_logp, 16));
  if (vec)
    decide_kernel<true><<<pl.decide_blocks, kDecideThreads, 0, stream>>>(T, S, c, logp, old_logp, ref_logp,
                                                                         segment_version, advantages, seq_offsets, gate,
                                                                         batch_mean, grad_coef, flags, partials);
  else
    decide_kernel<false><<<pl.decide_blocks, kDecideThreads, 0, stream>>>(T, S, c, logp, old_logp, ref_logp,
                                                                          segment_version, advantages, seq_offsets, gate,
                                                                          batch_mean, grad_coef, flags, partials);
  ULORL_LAUNCH_CHECK();
  finalize_kernel<<<1, kFinalThreads, 0, stream>>>(T, pl.decide_blocks, c.inv_N, partials, batch_mean, status, loss,
                                                   reinterpret_cast<ulorl_stats_t*>(stats));
  ULORL_LAUNCH_CHECK();
  return ULORL_OK;
}

static int validate_decide_args(const ulorl_params_t* p, const float* old_logp, const float* ref_logp,
                                const float* advantages,
                                const int32_t* seq_offsets, const float* entropy_supplied, float* seq_entropy,
                                float* loss) {
  if (!advantages || !seq_offsets || !loss || !seq_entropy) return ULORL_ERR_INVALID_ARG;
  if (p->is_mode == ULORL_IS_SAIS && !old_logp) return ULORL_ERR_INVALID_ARG;
  if (p->kl_beta > 0.f && !ref_logp) return ULORL_ERR_INVALID_ARG;
  if (p->mpt_mode == ULORL_MPT_DYNAMIC && p->ent_scope == ULORL_ENT_SUPPLIED && !entropy_supplied)
    return ULORL_ERR_INVALID_ARG;
  return ULORL_OK;
}

// T == 0: nothing to compute; the loss and the statistics are zero.
static int empty_forward(void* workspace, size_t workspace_bytes, float* loss, void* stats, cudaStream_t stream) {
  if (!loss) return ULORL_ERR_INVALID_ARG;
  if (workspace && workspace_bytes >= 256 && cudaMemsetAsync(workspace, 0, 256, stream) != cudaSuccess)
    return ULORL_ERR_CUDA;
  if (cudaMemsetAsync(loss, 0, sizeof(float), stream) != cudaSuccess) return ULORL_ERR_CUDA;
  if (stats && cudaMemsetAsync(stats, 0, sizeof(ulorl_stats_t), stream) != cudaSuccess) return ULORL_ERR_CUDA;
  return ULORL_OK;
}

// Vocabulary tiles of each split that one of `w_slabs` cuts of a sweep covers.
static int w_slab_tiles(const Plan& pl, int w_slabs) {
  return std::max(1, (pl.tiles_per_split + w_slabs - 1) / std::max(w_slabs, 1));
}

// Points at which the host-buffer step interleaves its copies with the two passes.  The forward
// launches the statistics kernel once per chunk of tokens (all at once without hooks), the backward
// reports every token panel whose d_hidden rows are final.
struct StepHooks {
  // Forward, tensor path: the statistics kernel is launched once per chunk of tokens; chunk c covers tokens
  // [chunk_starts[c], chunk_starts[c + 1]) (the last one runs to T; empty = one chunk).  With w_slabs > 1 the
  // sweep of the FIRST chunk is cut into w_slabs launches: launch j covers, of every vocabulary split, the j-th
  // run of tiles (w_slab_tiles(plan) of them), and before_w_slab(j) is called before it -- W may still be
  // arriving while the chunk's first launches run.  The cut does not change the results.
  std::vector<int> chunk_starts;
  int w_slabs = 0;
  std::function<int(int)> before_w_slab;
  std::function<int(int, int)> before_stats_chunk;    // (first token, tokens) -> status
  std::function<int(int, int)> after_dhidden_panel;   // (first token, tokens) -> status; dense backward only
  // Tensor path: when set, the last panel computes d_W before d_hidden and in slabs of vocabulary rows,
  // and this is called after each slab (first row, rows): those rows of d_W are final from then on.
  std::function<int(int, int)> after_dw_slab;
  // Tensor path, with after_dw_slab: device memory for a second dz panel (same size as the workspace's), or
  // NULL.  With it the last two panels are reordered so that more work follows the point where d_W is final.
  void* dz_second_buffer = nullptr;
};

}  // namespace ulorl

using namespace ulorl;

extern "C" {

size_t ulorl_workspace_bytes(const ulorl_params_t* params) {
  if (validate_params(params) != ULORL_OK) return 0;
  return make_plan(params).total;
}

int ulorl_selftest_bounded_wait(void* workspace, int64_t limit_cycles, void* cuda_stream) {
  if (!workspace) return ULORL_ERR_INVALID_ARG;
  if (limit_cycles < 1000 || limit_cycles > 100000000) return ULORL_ERR_INVALID_ARG;   // at most ~0.1 s of SM clocks
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  bounded_wait_selftest_kernel<<<1, 32, 0, stream>>>((long long)limit_cycles, reinterpret_cast<int*>(workspace));
  return check_launch();
}

int ulorl_decision_thresholds(const ulorl_params_t* params, float* out) {
  const int st = validate_params(params);
  if (st != ULORL_OK) return st;
  if (!out) return ULORL_ERR_INVALID_ARG;
  const DecideConsts c = make_decide_consts(params);
  out[0] = c.ln_tau;
  out[1] = c.ln_hi;
  out[2] = c.ln_lo;
  return ULORL_OK;
}

int64_t ulorl_launch_count(void) { return (int64_t)g_launches.load(std::memory_order_relaxed); }

const char* ulorl_status_string(int status) {
  switch (status) {
    case ULORL_OK: return "ok";
    case ULORL_ERR_INVALID_ARG: return "invalid argument";
    case ULORL_ERR_UNSUPPORTED: return "unsupported shape, dtype or alignment";
    case ULORL_ERR_WORKSPACE: return "workspace too small";
    case ULORL_ERR_CUDA: return "CUDA call failed";
    case ULORL_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
    case ULORL_ERR_BAD_TARGET: return "a target id was outside [0, V)";
    case ULORL_ERR_STATIC_LIMIT: return "batch larger than the built-in scratch of the no-allocation entry point";
    default: return "unknown status";
  }
}

static int static_scratch_address(uint8_t** out);

int ulorl_check_status(void* workspace, void* cuda_stream) {
  if (!workspace) {   // the status word of the built-in scratch of ulorl_token_loss_decide_static on this device
    uint8_t* builtin = nullptr;
    const int st = static_scratch_address(&builtin);
    if (st != ULORL_OK) return st;
    workspace = builtin;
  }
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  int word = 0;
  if (cudaMemcpyAsync(&word, workspace, sizeof(int), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return ULORL_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return ULORL_ERR_CUDA;
  if (word & kStatusTimeout) return ULORL_ERR_DEVICE_TIMEOUT;
  if (word & kStatusBadOffsets) return ULORL_ERR_INVALID_ARG;
  if (word & kStatusBadTarget) return ULORL_ERR_BAD_TARGET;
  return ULORL_OK;
}

int ulorl_token_loss_decide(const ulorl_params_t* params, const float* logp, const float* entropy,
                            const float* old_logp, const float* ref_logp, const int32_t* segment_version,
                            const float* advantages,
                            const int32_t* seq_offsets, const float* entropy_supplied, float* grad_coef,
                            uint8_t* flags, float* seq_entropy, float* loss, void* stats, void* workspace,
                            size_t workspace_bytes, void* cuda_stream) {
  int st = validate_params(params);
  if (st != ULORL_OK) return st;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (params->T == 0) return empty_forward(workspace, workspace_bytes, loss, stats, stream);
  if (!logp || !entropy || !workspace) return ULORL_ERR_INVALID_ARG;
  st = validate_decide_args(params, old_logp, ref_logp, advantages, seq_offsets, entropy_supplied, seq_entropy, loss);
  if (st != ULORL_OK) return st;
  const Plan pl = make_plan(params);
  if (workspace_bytes < pl.total) return ULORL_ERR_WORKSPACE;
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  if (cudaMemsetAsync(ws + pl.off_status, 0, 256, stream) != cudaSuccess) return ULORL_ERR_CUDA;
  return run_decide(params, pl, logp, entropy, old_logp, ref_logp, segment_version, advantages, seq_offsets, entropy_supplied,
                    grad_coef, flags, seq_entropy, loss, stats, ws, stream);
}

static int fwd_impl(const ulorl_params_t* params, const void* hidden, const void* W, const int32_t* targets,
                    const float* old_logp, const float* ref_logp, const int32_t* segment_version,
                    const float* advantages,
                    const int32_t* seq_offsets, const float* entropy_supplied, float* logp, float* entropy,
                    float* lse, float* grad_coef, uint8_t* flags, float* seq_entropy, float* loss, void* stats,
                    void* workspace, size_t workspace_bytes, void* cuda_stream, const StepHooks* hooks) {
  TraceRange trace("ulorl forward");
  int st = validate_params(params);
  if (st != ULORL_OK) return st;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (params->T == 0) return empty_forward(workspace, workspace_bytes, loss, stats, stream);
  if (!hidden || !W || !targets || !logp || !entropy || !lse || !workspace) return ULORL_ERR_INVALID_ARG;
  st = validate_decide_args(params, old_logp, ref_logp, advantages, seq_offsets, entropy_supplied, seq_entropy, loss);
  if (st != ULORL_OK) return st;
  if (!aligned16(hidden) || !aligned16(W) || !aligned16(workspace)) return ULORL_ERR_UNSUPPORTED;
  const Plan pl = make_plan(params);
  if (workspace_bytes < pl.total) return ULORL_ERR_WORKSPACE;
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  const int T = params->T, H = params->H, V = params->V;
  if (cudaMemsetAsync(ws + pl.off_status, 0, 256, stream) != cudaSuccess) return ULORL_ERR_CUDA;
  int* status = reinterpret_cast<int*>(ws + pl.off_status);
  float4* partials = reinterpret_cast<float4*>(ws + pl.off_partials);
  float* acc_y = reinterpret_cast<float*>(ws + pl.off_acc_y);
  const float kappa = params->inv_temperature;

  if (pl.tensor) {
    CUtensorMap map_a, map_b;
    st = make_map_bf16(&map_a, hidden, (uint64_t)T, (uint64_t)H, (uint64_t)H, kBK, kBM);
    if (st != ULORL_OK) return st;
    st = make_map_bf16(&map_b, W, (uint64_t)V, (uint64_t)H, (uint64_t)H, kBK, kBN / pl.cta);
    if (st != ULORL_OK) return st;
    const int tile_m = kBM * pl.cta;
    const int n_tiles = (V + kBN - 1) / kBN;
    std::vector<int> starts = (hooks && !hooks->chunk_starts.empty()) ? hooks->chunk_starts : std::vector<int>{0};
    starts.push_back(T);
    auto launch_stats = [&](int t0, int rows, int tile_base, int tiles, int resume) -> int {
      UmmaArgs a{};
      a.M = rows; a.N = V; a.K = H;
      a.m_tiles = (rows + tile_m - 1) / tile_m;
      a.n_tiles = n_tiles;
      a.n_split = pl.n_split;
      a.split_stride = pl.tiles_per_split;
      a.tiles_per_split = tiles;
      a.tile_base = tile_base;
      a.resume = resume;
      a.a_mn0 = t0;
      a.row0 = t0;
      a.kappa = kappa;
      a.targets = targets;
      a.partials = partials;
      a.acc_y = acc_y;
      a.T_total = T;
      a.status = status;
      return launch_umma<kModeStats>(pl, map_a, map_b, map_a, a, stream);
    };
    for (size_t c = 0; c + 1 < starts.size(); ++c) {
      const int t0 = starts[c], rows = starts[c + 1] - starts[c];
      if (rows <= 0 || t0 % tile_m != 0) return ULORL_ERR_INVALID_ARG;
      if (hooks && hooks->before_stats_chunk) {
        st = hooks->before_stats_chunk(t0, rows);
        if (st != ULORL_OK) return st;
      }
      const int w_slabs = (c == 0 && hooks && hooks->before_w_slab) ? hooks->w_slabs : 0;
      if (w_slabs > 1) {
        const int q = w_slab_tiles(pl, w_slabs);
        for (int j = 0; j * q < pl.tiles_per_split; ++j) {
          st = hooks->before_w_slab(j);
          if (st != ULORL_OK) return st;
          st = launch_stats(t0, rows, j * q, q, j > 0 ? 1 : 0);
          if (st != ULORL_OK) return st;
        }
      } else {
        st = launch_stats(t0, rows, 0, pl.tiles_per_split, 0);
        if (st != ULORL_OK) return st;
      }
    }
    merge_splits_kernel<<<(T + 255) / 256, 256, 0, stream>>>(T, 0, T, pl.n_split, kappa, partials, acc_y, logp, entropy,
                                                             lse);
    ULORL_LAUNCH_CHECK();
  } else {
    if (hooks && hooks->before_stats_chunk) {
      st = hooks->before_stats_chunk(0, T);
      if (st != ULORL_OK) return st;
    }
    const dim3 grid((T + kSimtTile - 1) / kSimtTile, pl.n_split);
    if (params->dtype == ULORL_F32)
      simt_stats_kernel<float><<<grid, kSimtThreads, 0, stream>>>(
          static_cast<const float*>(hidden), static_cast<const float*>(W), targets, T, V, H, kappa, pl.tiles_per_split,
          partials, acc_y, status);
    else
      simt_stats_kernel<__nv_bfloat16><<<grid, kSimtThreads, 0, stream>>>(
          static_cast<const __nv_bfloat16*>(hidden), static_cast<const __nv_bfloat16*>(W), targets, T, V, H, kappa,
          pl.tiles_per_split, partials, acc_y, status);
    ULORL_LAUNCH_CHECK();
    merge_splits_kernel<<<(T + 255) / 256, 256, 0, stream>>>(T, 0, T, pl.n_split, kappa, partials, acc_y, logp, entropy,
                                                             lse);
    ULORL_LAUNCH_CHECK();
  }
  return run_decide(params, pl, logp, entropy, old_logp, ref_logp, segment_version, advantages, seq_offsets, entropy_supplied,
                    grad_coef, flags, seq_entropy, loss, stats, ws, stream);
}

int ulorl_token_loss_fwd(const ulorl_params_t* params, const void* hidden, const void* W, const int32_t* targets,
                         const float* old_logp, const float* ref_logp, const int32_t* segment_version,
                         const float* advantages,
                         const int32_t* seq_offsets, const float* entropy_supplied, float* logp, float* entropy,
                         float* lse, float* grad_coef, uint8_t* flags, float* seq_entropy, float* loss, void* stats,
                         void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return fwd_impl(params, hidden, W, targets, old_logp, ref_logp, segment_version, advantages, seq_offsets, entropy_supplied, logp,
                  entropy, lse, grad_coef, flags, seq_entropy, loss, stats, workspace, workspace_bytes, cuda_stream,
                  nullptr);
}

// d_W rows [v0, v0 + v_rows) are final in the float32 accumulator: round them into the caller's bf16 d_W.
static int round_dw_rows(const float* acc, void* d_W, int v0, int v_rows, int H, int accumulate, cudaStream_t stream) {
  const size_t n8 = (size_t)v_rows * (size_t)H / 8;            // H is a multiple of 8
  if (n8 == 0) return ULORL_OK;
  const size_t first = (size_t)v0 * (size_t)H;
  const unsigned blocks = (unsigned)std::min<size_t>((n8 + 255) / 256, 148u * 16u);
  dw_round_kernel<<<blocks, 256, 0, stream>>>(acc + first, static_cast<__nv_bfloat16*>(d_W) + first, n8, accumulate);
  return check_launch();
}

static int bwd_impl(const ulorl_params_t* params, const void* hidden, const void* W, const int32_t* targets,
                    const float* lse, const float* grad_coef, const float* grad_loss, void* d_hidden, void* d_W_out,
                    void* workspace, size_t workspace_bytes, void* cuda_stream, const StepHooks* hooks) {
  TraceRange trace("ulorl backward");
  int st = validate_params(params);
  if (st != ULORL_OK) return st;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  const int T = params->T, H = params->H, V = params->V;
  const size_t dw_elem = params->dw_dtype == ULORL_BF16 ? 2 : 4;
  if (T == 0) {
    if (!d_W_out) return ULORL_ERR_INVALID_ARG;
    if (!params->dw_accumulate && cudaMemsetAsync(d_W_out, 0, dw_elem * (size_t)V * H, stream) != cudaSuccess)
      return ULORL_ERR_CUDA;
    if (hooks && hooks->after_dw_slab) return hooks->after_dw_slab(0, V);
    return ULORL_OK;
  }
  if (!hidden || !W || !targets || !lse || !grad_coef || !d_hidden || !d_W_out || !workspace) return ULORL_ERR_INVALID_ARG;
  if (!aligned16(hidden) || !aligned16(W) || !aligned16(d_hidden) || !aligned16(d_W_out) || !aligned16(workspace))
    return ULORL_ERR_UNSUPPORTED;
  const Plan pl = make_plan(params);
  if (workspace_bytes < pl.total) return ULORL_ERR_WORKSPACE;
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  const float kappa = params->inv_temperature;
  int* status = reinterpret_cast<int*>(ws + pl.off_status);
  // The contractions sum d_W in float32: straight into the caller's array, or, for a bf16 d_W, into the
  // workspace, from where rows are rounded (and added to the caller's values, if asked) once they are final.
  float* d_W = pl.dw_bf16 ? reinterpret_cast<float*>(ws + pl.off_dw_acc) : static_cast<float*>(d_W_out);
  const int acc_into = pl.dw_bf16 ? 0 : params->dw_accumulate;
  auto dw_rows_final = [&](int v0, int v_rows) -> int {
    if (pl.dw_bf16) {
      const int rc = round_dw_rows(d_W, d_W_out, v0, v_rows, H, params->dw_accumulate, stream);
      if (rc != ULORL_OK) return rc;
    }
    return (hooks && hooks->after_dw_slab) ? hooks->after_dw_slab(v0, v_rows) : (int)ULORL_OK;
  };

  if (pl.tensor) {
    __nv_bfloat16* dz = reinterpret_cast<__nv_bfloat16*>(ws + pl.off_dz);
    const int tile_m = kBM * pl.cta;
    // With compaction the three contractions run on gathered copies of the active rows; how many
    // there are is only known on the device, so every launch is sized for the worst case and reads
    // the count itself.
    const int* n_active = nullptr;
    void* d_hidden_out = d_hidden;
    if (pl.compact) {
      int* blk_count = reinterpret_cast<int*>(ws + pl.off_blk_count);
      int* blk_offset = reinterpret_cast<int*>(ws + pl.off_blk_offset);
      int* position = reinterpret_cast<int*>(ws + pl.off_position);
      int* n_act = reinterpret_cast<int*>(ws + pl.off_n_active);
      int* targets_c = reinterpret_cast<int*>(ws + pl.off_targets_c);
      float* lse_c = reinterpret_cast<float*>(ws + pl.off_lse_c);
      float* coef_c = reinterpret_cast<float*>(ws + pl.off_coef_c);
      __nv_bfloat16* hidden_c = reinterpret_cast<__nv_bfloat16*>(ws + pl.off_hidden_c);
      compact_count_kernel<<<pl.compact_blocks, kCompactThreads, 0, stream>>>(T, grad_coef, blk_count);
      ULORL_LAUNCH_CHECK();
      compact_offsets_kernel<<<1, 1024, 0, stream>>>(pl.compact_blocks, blk_count, blk_offset, n_act);
      ULORL_LAUNCH_CHECK();
      compact_gather_kernel<__nv_bfloat16><<<pl.compact_blocks, kCompactThreads, 0, stream>>>(
          T, H, grad_coef, blk_offset, n_act, static_cast<const __nv_bfloat16*>(hidden), targets, lse, position,
          hidden_c, targets_c, lse_c, coef_c);
      ULORL_LAUNCH_CHECK();
      if (!acc_into && cudaMemsetAsync(d_W, 0, sizeof(float) * (size_t)V * H, stream) != cudaSuccess)
        return ULORL_ERR_CUDA;
      n_active = n_act;
      hidden = hidden_c;
      targets = targets_c;
      lse = lse_c;
      grad_coef = coef_c;
      d_hidden_out = ws + pl.off_dh_c;
    }
    const uint64_t hidden_rows = pl.compact ? (uint64_t)pl.t_pad : (uint64_t)T;
    CUtensorMap map_hidden_k, map_w_k, map_w_mn, map_hidden_mn;
    st = make_map_bf16(&map_hidden_k, hidden, hidden_rows, (uint64_t)H, (uint64_t)H, kBK, kBM);
    if (st != ULORL_OK) return st;
    st = make_map_bf16(&map_w_k, W, (uint64_t)V, (uint64_t)H, (uint64_t)H, kBK, kBN / pl.cta);
    if (st != ULORL_OK) return st;
    st = make_map_bf16(&map_w_mn, W, (uint64_t)V, (uint64_t)H, (uint64_t)H, 64, kBK);
    if (st != ULORL_OK) return st;
    st = make_map_bf16(&map_hidden_mn, hidden, hidden_rows, (uint64_t)H, (uint64_t)H, 64, kBK);
    if (st != ULORL_OK) return st;
    CUtensorMap map_dw_out;   // d_W as the target of 128-row x 32-column float tiles
    st = make_map(&map_dw_out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, d_W, (uint64_t)V, (uint64_t)H, (uint64_t)H, 32, kBM);
    if (st != ULORL_OK) return st;
    // One token panel: its rows, its dz buffer and the tensor maps over that buffer.
    struct Panel {
      int t0, rows, index;
      CUtensorMap dz_out, dz_k, dz_mn;
    };
    auto make_panel = [&](int t0, int index, __nv_bfloat16* buf, Panel& pn) -> int {
      pn.t0 = t0;
      pn.rows = (T - t0) < pl.panel_tokens ? (T - t0) : pl.panel_tokens;
      pn.index = index;
      // the whole buffer as the target of 128-row x 64-column bf16 tiles; its valid rows as the operand of the
      // two gradient contractions (K-major for d_hidden, MN-major for d_W)
      int rc = make_map_bf16(&pn.dz_out, buf, (uint64_t)pl.panel_tokens, (uint64_t)pl.dz_ld, (uint64_t)pl.dz_ld, 64, kBM);
      if (rc != ULORL_OK) return rc;
      rc = make_map_bf16(&pn.dz_k, buf, (uint64_t)pn.rows, (uint64_t)pl.dz_ld, (uint64_t)pl.dz_ld, kBK, kBM);
      if (rc != ULORL_OK) return rc;
      return make_map_bf16(&pn.dz_mn, buf, (uint64_t)pn.rows, (uint64_t)pl.dz_ld, (uint64_t)pl.dz_ld, 64, kBK);
    };
    // dz panel: recompute logits, softmax minus one-hot scaled by the token's coefficient
    auto run_dz = [&](const Panel& pn) -> int {
      UmmaArgs a{};
      a.M = pn.rows; a.N = V; a.K = H;
      a.m_tiles = (pn.rows + tile_m - 1) / tile_m;
      a.n_tiles = (int)(pl.dz_ld / kBN) + ((pl.dz_ld % kBN) ? 1 : 0);
      a.group_m = kRasterGroup;
      a.a_mn0 = pn.t0;
      a.row0 = pn.t0;
      a.kappa = kappa;
      a.targets = targets; a.lse = lse; a.grad_coef = grad_coef; a.grad_loss = grad_loss;
      a.dz_cols = (int)pl.dz_ld;
      a.dyn_rows = n_active; a.dyn_base = pn.t0;
      a.status = status;
      return launch_umma<kModeDz>(pl, map_hidden_k, map_w_k, pn.dz_out, a, stream);
    };
    // d_hidden[t0 + m, h] = sum_v dz[m, v] W[v, h]
    auto run_d_hidden = [&](const Panel& pn) -> int {
      UmmaArgs a{};
      a.M = pn.rows; a.N = H; a.K = V;
      a.m_tiles = (pn.rows + tile_m - 1) / tile_m;
      a.n_tiles = (H + grad_unit_cols(pl) - 1) / grad_unit_cols(pl);
      a.group_m = kGradRasterGroup;
      a.row0 = pn.t0;
      a.d_hidden = static_cast<__nv_bfloat16*>(d_hidden_out);
      a.out_ld = (size_t)H;
      a.dyn_rows = n_active; a.dyn_base = pn.t0;
      a.status = status;
      int rc = launch_umma<kModeDHidden>(pl, pn.dz_k, map_w_mn, map_w_mn, a, stream);
      if (rc != ULORL_OK) return rc;
      if (hooks && hooks->after_dhidden_panel && !pl.compact) return hooks->after_dhidden_panel(pn.t0, pn.rows);
      return ULORL_OK;
    };
    // d_W[v, h] (+)= sum_m dz[m, v] hidden[t0 + m, h] for the vocabulary rows [v0, v0 + v_rows)
    auto run_d_W = [&](const Panel& pn, int v0, int v_rows) -> int {
      UmmaArgs a{};
      a.M = v_rows; a.N = H; a.K = pn.rows;
      a.m_tiles = (v_rows + tile_m - 1) / tile_m;
      a.n_tiles = (H + grad_unit_cols(pl) - 1) / grad_unit_cols(pl);
      a.group_m = kGradRasterGroup;
      a.a_mn0 = v0;
      a.b_k0 = pn.t0;
      a.row0 = v0;
      a.d_W = d_W;
      a.out_ld = (size_t)H;
      a.accumulate = (pn.index > 0 || acc_into || pl.compact) ? 1 : 0;
      a.dyn_rows = n_active; a.dyn_base = pn.t0;
      a.status = status;
      return launch_umma<kModeDW>(pl, pn.dz_mn, map_hidden_mn, map_dw_out, a, stream);
    };
    const int n_panels = (T + pl.panel_tokens - 1) / pl.panel_tokens;
    const bool by_slabs = hooks && hooks->after_dw_slab;
    // With a second dz buffer from the caller, the d_hidden contraction of the panel before the last is put off
    // until d_W is final: the last two panels then run dz, d_W, dz', d_W' (slab by slab), d_hidden, d_hidden', so
    // that two d_hidden contractions, not one, are still to come while the rows of d_W are already on their way out.
    __nv_bfloat16* dz_alt = (hooks && by_slabs && !pl.compact && n_panels >= 2)
                                ? static_cast<__nv_bfloat16*>(hooks->dz_second_buffer) : nullptr;
    Panel held{};
    for (int t0 = 0, panel = 0; t0 < T; t0 += pl.panel_tokens, ++panel) {
      const bool last_panel = panel == n_panels - 1;
      TraceRange panel_trace(last_panel ? "ulorl backward: last panel" : "ulorl backward: panel");
      Panel pn;
      st = make_panel(t0, panel, (dz_alt && last_panel) ? dz_alt : dz, pn);
      if (st != ULORL_OK) return st;
      st = run_dz(pn);
      if (st != ULORL_OK) return st;
      if (dz_alt && panel == n_panels - 2) {       // its d_hidden follows the last panel's d_W
        st = run_d_W(pn, 0, V);
        if (st != ULORL_OK) return st;
        held = pn;
        continue;
      }
      if (last_panel && by_slabs) {
        // d_W is final slab by slab, so the caller can start moving it while the rest is computed; a slab
        // is a whole number of waves of units (row tiles in multiples of the worker count), about eight
        const int workers = std::max(1, pl.sms / pl.cta);
        const int v_tiles = (V + tile_m - 1) / tile_m;
        const int slab_tiles = workers * ((v_tiles + 8 * workers - 1) / (8 * workers));
        const int slab_rows = slab_tiles * tile_m;
        for (int v0 = 0; v0 < V; v0 += slab_rows) {
          const int v_rows = (V - v0) < slab_rows ? (V - v0) : slab_rows;
          st = run_d_W(pn, v0, v_rows);
          if (st != ULORL_OK) return st;
          st = dw_rows_final(v0, v_rows);
          if (st != ULORL_OK) return st;
        }
        if (dz_alt) {
          st = run_d_hidden(held);
          if (st != ULORL_OK) return st;
        }
        st = run_d_hidden(pn);
        if (st != ULORL_OK) return st;
      } else {
        st = run_d_hidden(pn);
        if (st != ULORL_OK) return st;
        st = run_d_W(pn, 0, V);
        if (st != ULORL_OK) return st;
        if (last_panel) {
          st = dw_rows_final(0, V);
          if (st != ULORL_OK) return st;
        }
      }
    }
    if (pl.compact) {
      compact_scatter_kernel<__nv_bfloat16><<<(T + 7) / 8, 256, 0, stream>>>(
          T, H, reinterpret_cast<const int*>(ws + pl.off_position),
          reinterpret_cast<const __nv_bfloat16*>(ws + pl.off_dh_c), static_cast<__nv_bfloat16*>(d_hidden));
      ULORL_LAUNCH_CHECK();
    }
    return ULORL_OK;
  }

  // SIMT path: float32 dz panel, three CUDA-core contractions
  float* dz = reinterpret_cast<float*>(ws + pl.off_dz);
  for (int t0 = 0, panel = 0; t0 < T; t0 += pl.panel_tokens, ++panel) {
    const int rows = (T - t0) < pl.panel_tokens ? (T - t0) : pl.panel_tokens;
    const dim3 gdz((rows + kSimtTile - 1) / kSimtTile, (V + kSimtTile - 1) / kSimtTile);
    const dim3 gdh((H + kSimtTile - 1) / kSimtTile, (rows + kSimtTile - 1) / kSimtTile);
    const dim3 gdw((H + kSimtTile - 1) / kSimtTile, (V + kSimtTile - 1) / kSimtTile);
    const int acc = (panel > 0 || acc_into) ? 1 : 0;
    if (params->dtype == ULORL_F32) {
      const float* h = static_cast<const float*>(hidden);
      const float* w = static_cast<const float*>(W);
      simt_dz_kernel<float><<<gdz, kSimtThreads, 0, stream>>>(h, w, targets, lse, grad_coef, grad_loss, T, V, H, kappa,
                                                               t0, t0 + rows, dz, pl.dz_ld);
      ULORL_LAUNCH_CHECK();
      simt_gemm_kernel<float, float, float><<<gdh, kSimtThreads, 0, stream>>>(
          dz, pl.dz_ld, 1, w, (size_t)H, 1, static_cast<float*>(d_hidden) + (size_t)t0 * H, (size_t)H, rows, H, V, 0);
      ULORL_LAUNCH_CHECK();
      simt_gemm_kernel<float, float, float><<<gdw, kSimtThreads, 0, stream>>>(
          dz, 1, pl.dz_ld, h + (size_t)t0 * H, (size_t)H, 1, d_W, (size_t)H, V, H, rows, acc);
      ULORL_LAUNCH_CHECK();
    } else {
      const __nv_bfloat16* h = static_cast<const __nv_bfloat16*>(hidden);
      const __nv_bfloat16* w = static_cast<const __nv_bfloat16*>(W);
      simt_dz_kernel<__nv_bfloat16><<<gdz, kSimtThreads, 0, stream>>>(h, w, targets, lse, grad_coef, grad_loss, T, V, H,
                                                                       kappa, t0, t0 + rows, dz, pl.dz_ld);
      ULORL_LAUNCH_CHECK();
      simt_gemm_kernel<float, __nv_bfloat16, __nv_bfloat16><<<gdh, kSimtThreads, 0, stream>>>(
          dz, pl.dz_ld, 1, w, (size_t)H, 1, static_cast<__nv_bfloat16*>(d_hidden) + (size_t)t0 * H, (size_t)H, rows, H,
          V, 0);
      ULORL_LAUNCH_CHECK();
      simt_gemm_kernel<float, __nv_bfloat16, float><<<gdw, kSimtThreads, 0, stream>>>(
          dz, 1, pl.dz_ld, h + (size_t)t0 * H, (size_t)H, 1, d_W, (size_t)H, V, H, rows, acc);
      ULORL_LAUNCH_CHECK();
    }
    if (hooks && hooks->after_dhidden_panel) {
      st = hooks->after_dhidden_panel(t0, rows);
      if (st != ULORL_OK) return st;
    }
  }
  return dw_rows_final(0, V);
}

int ulorl_token_loss_bwd(const ulorl_params_t* params, const void* hidden, const void* W, const int32_t* targets,
                         const float* lse, const float* grad_coef, const float* grad_loss, void* d_hidden, void* d_W,
                         void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return bwd_impl(params, hidden, W, targets, lse, grad_coef, grad_loss, d_hidden, d_W, workspace, workspace_bytes,
                  cuda_stream, nullptr);
}

int ulorl_token_loss_bwd_slabs(const ulorl_params_t* params, const void* hidden, const void* W, const int32_t* targets,
                               const float* lse, const float* grad_coef, const float* grad_loss, void* d_hidden,
                               void* d_W, ulorl_dw_slab_fn on_slab, void* user, void* workspace,
                               size_t workspace_bytes, void* cuda_stream) {
  if (!on_slab)
    return bwd_impl(params, hidden, W, targets, lse, grad_coef, grad_loss, d_hidden, d_W, workspace, workspace_bytes,
                    cuda_stream, nullptr);
  StepHooks hooks;
  hooks.after_dw_slab = [&](int v0, int v_rows) { return on_slab(user, (int32_t)v0, (int32_t)v_rows); };
  return bwd_impl(params, hidden, W, targets, lse, grad_coef, grad_loss, d_hidden, d_W, workspace, workspace_bytes,
                  cuda_stream, &hooks);
}

// ------------------------------------------------------------------ decision stage without a workspace
// Scratch of ulorl_token_loss_decide_static: a fixed array in the library's own device image,
// resident on every GPU that loads the library until the process exits.
//   [0, 256)                       status word and batch-mean slot
//   [256, 256 + 8 * max seqs)      64-bit integer entropy sum per sequence
//   rest                           one DecidePartial per block of 256 tokens
constexpr size_t kStaticSeqBytes = sizeof(long long) * (size_t)ULORL_STATIC_MAX_SEQS;
constexpr size_t kStaticDecideBlocks = ((size_t)ULORL_STATIC_MAX_TOKENS + kDecideTokens - 1) / kDecideTokens;
constexpr size_t kStaticScratchBytes = 256 + kStaticSeqBytes + sizeof(DecidePartial) * kStaticDecideBlocks;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device address of g_static_scratch on the current device.  In host code the array's name is only
// a handle for the runtime; the address a kernel can use comes from cudaGetSymbolAddress, asked once
// per device with that device current.
static int static_scratch_address(uint8_t** out) {
  constexpr int kMaxDevices = 64;
  static uint8_t* cached[kMaxDevices] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ULORL_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!cached[dev]) {
    void* ptr = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess || !ptr) {
      std::fprintf(stderr, "ulorl: cudaGetSymbolAddress failed: %s\n", cudaGetErrorString(e));
      return ULORL_ERR_CUDA;
    }
    cached[dev] = static_cast<uint8_t*>(ptr);
  }
  *out = cached[dev];
  return ULORL_OK;
}

int ulorl_token_loss_decide_static(const ulorl_params_t* params, const float* logp, const float* entropy,
                                   const float* old_logp, const float* ref_logp, const int32_t* segment_version,
                                   const float* advantages,
                                   const int32_t* seq_offsets, const float* entropy_supplied, float* grad_coef,
                                   uint8_t* flags, float* seq_entropy, float* loss, void* stats, void* cuda_stream) {
  int st = validate_params(params);
  if (st != ULORL_OK) return st;
  if (params->T > ULORL_STATIC_MAX_TOKENS || params->num_seqs > ULORL_STATIC_MAX_SEQS) {
    std::fprintf(stderr,
                 "ulorl_token_loss_decide_static: T=%d, num_seqs=%d exceed the built-in scratch (at most %d tokens, "
                 "%d sequences); use ulorl_token_loss_decide with a caller workspace\n",
                 params->T, params->num_seqs, ULORL_STATIC_MAX_TOKENS, ULORL_STATIC_MAX_SEQS);
    return ULORL_ERR_STATIC_LIMIT;
  }
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  uint8_t* ws = nullptr;
  st = static_scratch_address(&ws);
  if (st != ULORL_OK) return st;
  if (params->T == 0) return empty_forward(ws, 256, loss, stats, stream);
  if (!logp || !entropy) return ULORL_ERR_INVALID_ARG;
  st = validate_decide_args(params, old_logp, ref_logp, advantages, seq_offsets, entropy_supplied, seq_entropy, loss);
  if (st != ULORL_OK) return st;
  Plan pl{};
  pl.off_status = 0;
  pl.off_batch_mean = 16;
  pl.off_seq_sum = 256;
  pl.off_decide = 256 + kStaticSeqBytes;
  pl.decide_blocks = (params->T + kDecideTokens - 1) / kDecideTokens;
  pl.total = kStaticScratchBytes;
  // the array keeps whatever the previous call left: the status word must start at zero, every
  // other slot that this call reads is written by this call first
  if (cudaMemsetAsync(ws + pl.off_status, 0, 256, stream) != cudaSuccess) return ULORL_ERR_CUDA;
  return run_decide(params, pl, logp, entropy, old_logp, ref_logp, segment_version, advantages, seq_offsets, entropy_supplied,
                    grad_coef, flags, seq_entropy, loss, stats, ws, stream);
}

int ulorl_sequence_entropy_partials(const ulorl_params_t* params, const float* entropy, const int32_t* seq_offsets,
                                    const int32_t* seq_ids, int32_t total_seqs, int64_t* table, void* workspace,
                                    void* cuda_stream) {
  int st = validate_params(params);
  if (st != ULORL_OK) return st;
  if (total_seqs < 0 || (total_seqs > 0 && !table)) return ULORL_ERR_INVALID_ARG;
  if (!seq_ids && params->num_seqs > total_seqs) return ULORL_ERR_INVALID_ARG;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  if (total_seqs > 0 && cudaMemsetAsync(table, 0, 2 * sizeof(int64_t) * (size_t)total_seqs, stream) != cudaSuccess)
    return ULORL_ERR_CUDA;
  if (params->T == 0 || params->num_seqs == 0) return ULORL_OK;
  if (!entropy || !seq_offsets) return ULORL_ERR_INVALID_ARG;
  static_assert(sizeof(long long) == sizeof(int64_t), "64-bit sums");
  seq_entropy_partials_kernel<<<params->num_seqs, kSeqThreads, 0, stream>>>(
      params->num_seqs, params->T, seq_offsets, entropy, seq_ids, total_seqs, reinterpret_cast<long long*>(table),
      reinterpret_cast<int*>(workspace));
  return check_launch();
}

int ulorl_sequence_entropy_combine(const int64_t* table, int32_t total_seqs, const int32_t* seq_ids, int32_t num_seqs,
                                   float* seq_entropy, float* batch_entropy, void* cuda_stream) {
  if (total_seqs < 0 || num_seqs < 0) return ULORL_ERR_INVALID_ARG;
  if (!seq_ids && num_seqs > total_seqs) return ULORL_ERR_INVALID_ARG;
  if (num_seqs == 0 && !batch_entropy) return ULORL_OK;
  if (!table || (num_seqs > 0 && !seq_entropy)) return ULORL_ERR_INVALID_ARG;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  const int n = num_seqs > 0 ? num_seqs : 1;
  seq_entropy_combine_kernel<<<(n + 127) / 128, 128, 0, stream>>>(num_seqs, seq_ids, total_seqs,
                                                                 reinterpret_cast<const long long*>(table), seq_entropy,
                                                                 batch_entropy);
  return check_launch();
}

int ulorl_group_advantages(const float* rewards, int32_t num_responses, int32_t group_size, float* advantages,
                           uint8_t* keep, void* cuda_stream) {
  if (num_responses < 0 || group_size <= 0) return ULORL_ERR_INVALID_ARG;
  if (num_responses == 0) return ULORL_OK;
  if (!rewards || !advantages) return ULORL_ERR_INVALID_ARG;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  const int groups = (num_responses + group_size - 1) / group_size;
  group_advantage_kernel<<<(groups + 127) / 128, 128, 0, stream>>>(num_responses, group_size, rewards, advantages, keep);
  return check_launch();
}

int ulorl_kernel_timing_begin(void) {
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  for (int k = 0; k < 4; ++k) g_timing.used[k] = 0;
  g_timing.enabled.store(true);
  return ULORL_OK;
}

int ulorl_kernel_timing_end(float* total_ms, int64_t* launches) {
  g_timing.enabled.store(false);
  if (!total_ms || !launches) return ULORL_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  for (int k = 0; k < 4; ++k) {
    double tot = 0.0;
    int64_t n = 0;
    for (size_t i = 0; i + 1 < g_timing.used[k]; i += 2) {
      if (cudaEventSynchronize(g_timing.ev[k][i + 1]) != cudaSuccess) return ULORL_ERR_CUDA;
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, g_timing.ev[k][i], g_timing.ev[k][i + 1]) != cudaSuccess) return ULORL_ERR_CUDA;
      tot += ms;
      ++n;
    }
    total_ms[k] = (float)tot;
    launches[k] = n;
  }
  return ULORL_OK;
}

// ------------------------------------------------------------------ host-buffer step
namespace {
struct HostStepLayout {
  size_t hidden, W, targets, old_logp, ref_logp, segver, adv, seq_off, ent_sup;
  size_t logp, entropy, lse, grad_coef, flags, seq_entropy, loss, stats, d_hidden, d_W, ws, dz2, total;
  size_t elem;
};
// Two copy streams and a few events, created on the first host-buffer step and kept: the inbound
// copies run ahead of the forward, the outbound copies of d_hidden behind the backward.
struct HostStepStreams {
  std::mutex step_mutex;   // held while one host-buffer step is enqueued: the streams and events are shared
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t start = nullptr, out_done = nullptr;
  std::vector<cudaEvent_t> chunk_in, panel_out, slab_out;
  cudaEvent_t slab_event(size_t i) {   // grows on demand; nullptr on failure
    while (slab_out.size() <= i) {
      cudaEvent_t e;
      if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
      slab_out.push_back(e);
    }
    return slab_out[i];
  }
  bool reserve(size_t n) {
    while (chunk_in.size() < n) {
      cudaEvent_t e0, e1;
      if (cudaEventCreateWithFlags(&e0, cudaEventDisableTiming) != cudaSuccess ||
          cudaEventCreateWithFlags(&e1, cudaEventDisableTiming) != cudaSuccess)
        return false;
      chunk_in.push_back(e0);
      panel_out.push_back(e1);
    }
    return true;
  }
};
// Streams and events belong to the device that was current when they were made: one set per device.
HostStepStreams* host_step_streams() {
  static HostStepStreams per_device[kMaxDevices];
  static bool ready[kMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  HostStepStreams& hs = per_device[dev];
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!ready[dev]) {
    if (cudaStreamCreateWithFlags(&hs.in, cudaStreamNonBlocking) != cudaSuccess ||
        cudaStreamCreateWithFlags(&hs.out, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&hs.start, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&hs.out_done, cudaEventDisableTiming) != cudaSuccess)
      return nullptr;
    ready[dev] = true;
  }
  return &hs;
}

HostStepLayout host_step_layout(const ulorl_params_t* p) {
  HostStepLayout L{};
  const size_t T = (size_t)p->T, H = (size_t)p->H, V = (size_t)p->V, S = (size_t)(p->num_seqs > 0 ? p->num_seqs : 1);
  L.elem = p->dtype == ULORL_BF16 ? 2 : 4;
  size_t off = 0;
  auto take = [&](size_t bytes) { const size_t o = off; off = align_up(off + (bytes ? bytes : 16), 1024); return o; };
  L.hidden = take(T * H * L.elem);
  L.W = take(V * H * L.elem);
  L.targets = take(T * 4);
  L.old_logp = take(T * 4);
  L.ref_logp = take(p->kl_beta > 0.f ? T * 4 : 0);
  L.segver = take(T * 4);
  L.adv = take((p->adv_per_token ? T : S) * 4);
  L.seq_off = take((S + 1) * 4);
  L.ent_sup = take(S * 4);
  L.logp = take(T * 4);
  L.entropy = take(T * 4);
  L.lse = take(T * 4);
  L.grad_coef = take(T * 4);
  L.flags = take(T);
  L.seq_entropy = take(S * 4);
  L.loss = take(16);
  L.stats = take(sizeof(ulorl_stats_t));
  L.d_hidden = take(T * H * L.elem);
  L.d_W = take(V * H * (p->dw_dtype == ULORL_BF16 ? 2 : 4));
  const Plan pl = make_plan(p);
  L.ws = take(pl.total);
  // a second dz panel when the backward has several panels to reorder at its end (tensor path, dense backward)
  const bool two_dz = pl.tensor && !pl.compact && p->T > pl.panel_tokens;
  L.dz2 = two_dz ? take((size_t)pl.panel_tokens * pl.dz_ld * 2) : 0;
  L.total = off;
  return L;
}
}  // namespace

size_t ulorl_host_step_arena_bytes(const ulorl_params_t* params) {
  if (validate_params(params) != ULORL_OK) return 0;
  return host_step_layout(params).total;
}

int ulorl_token_loss_step_host(const ulorl_params_t* params, const void* h_hidden, const void* h_W,
                               const int32_t* h_targets, const float* h_old_logp, const float* h_ref_logp,
                               const int32_t* h_segment_version,
                               const float* h_advantages, const int32_t* h_seq_offsets,
                               const float* h_entropy_supplied, float* h_logp, float* h_entropy, uint8_t* h_flags,
                               float* h_seq_entropy, float* h_loss, void* h_stats, void* h_d_hidden, void* h_d_W,
                               void* d_arena, size_t arena_bytes, void* cuda_stream) {
  TraceRange trace("ulorl host-buffer step");
  int st = validate_params(params);
  if (st != ULORL_OK) return st;
  if (!d_arena || !h_loss) return ULORL_ERR_INVALID_ARG;
  if (params->T > 0 && (!h_hidden || !h_W || !h_targets || !h_advantages || !h_seq_offsets)) return ULORL_ERR_INVALID_ARG;
  const HostStepLayout L = host_step_layout(params);
  if (arena_bytes < L.total) return ULORL_ERR_WORKSPACE;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  uint8_t* a = reinterpret_cast<uint8_t*>(d_arena);
  const size_t T = (size_t)params->T, H = (size_t)params->H, V = (size_t)params->V, S = (size_t)params->num_seqs;
  HostStepStreams* hs = host_step_streams();
  if (!hs) return ULORL_ERR_CUDA;
  std::lock_guard<std::mutex> step_lock(hs->step_mutex);
  const Plan pl = make_plan(params);
  const size_t row_bytes = H * L.elem;
  auto ok = [](cudaError_t e) { return e == cudaSuccess; };

  // copies in, on their own stream, ordered after whatever the caller's stream did to the arena before
  if (!ok(cudaEventRecord(hs->start, stream)) || !ok(cudaStreamWaitEvent(hs->in, hs->start, 0))) return ULORL_ERR_CUDA;
  auto h2d = [&](size_t off, const void* src, size_t bytes) {
    return (!src || !bytes) ? cudaSuccess : cudaMemcpyAsync(a + off, src, bytes, cudaMemcpyHostToDevice, hs->in);
  };
  if (!ok(h2d(L.targets, h_targets, T * 4)) || !ok(h2d(L.old_logp, h_old_logp, T * 4)) ||
      !ok(h2d(L.ref_logp, h_ref_logp, params->kl_beta > 0.f ? T * 4 : 0)) ||   // unread without the KL term
      !ok(h2d(L.segver, h_segment_version, T * 4)) ||
      !ok(h2d(L.adv, h_advantages, (params->adv_per_token ? T : S) * 4)) ||
      !ok(h2d(L.seq_off, h_seq_offsets, (S + 1) * 4)) || !ok(h2d(L.ent_sup, h_entropy_supplied, S * 4)))
    return ULORL_ERR_CUDA;
  // Order on the inbound stream: the first chunk of hidden states, then W in slabs of vocabulary rows, then
  // the other chunks, one event each.  The statistics kernel sweeps the first chunk slab by slab as W lands
  // (tensor path), and every later chunk as soon as its rows are there, while the rest is still on the bus.
  // The first chunk is sized so that one of its slab sweeps takes about as long as a slab's copy.
  const int chunk = pl.panel_tokens;
  const int tile_m = pl.tensor ? kBM * pl.cta : kBM;
  StepHooks hooks;
  if (params->T > 0) {
    int first = (int)align_up((size_t)chunk * 11 / 8, (size_t)tile_m);
    if (first >= params->T) first = params->T;
    hooks.chunk_starts.push_back(0);
    for (int t0 = first; t0 < params->T; t0 += chunk) hooks.chunk_starts.push_back(t0);
  }
  const int n_chunks = (int)hooks.chunk_starts.size();
  constexpr int kWSlabs = 8;
  const int n_tiles_v = (params->V + kBN - 1) / kBN;
  const int w_slabs = pl.tensor ? std::max(1, std::min(kWSlabs, pl.tiles_per_split)) : 1;
  const size_t n_panels = params->T > 0 ? ((size_t)params->T + chunk - 1) / chunk : 0;   // events of the backward's panels
  if (!hs->reserve(std::max((size_t)std::max(n_chunks, 1) + (size_t)w_slabs, n_panels))) return ULORL_ERR_CUDA;
  const size_t w_event0 = (size_t)std::max(n_chunks, 1);   // W-slab events sit behind the chunk events in the same table
  auto chunk_rows = [&](int c) {
    const size_t t0 = (size_t)hooks.chunk_starts[c];
    const size_t t1 = c + 1 < n_chunks ? (size_t)hooks.chunk_starts[c + 1] : T;
    return std::make_pair(t0, t1 - t0);
  };
  auto send_chunk = [&](int c) {
    const auto [t0, rows] = chunk_rows(c);
    return ok(h2d(L.hidden + t0 * row_bytes, static_cast<const uint8_t*>(h_hidden) + t0 * row_bytes, rows * row_bytes)) &&
           ok(cudaEventRecord(hs->chunk_in[c], hs->in));
  };
  if (n_chunks > 0 && !send_chunk(0)) return ULORL_ERR_CUDA;
  int n_w_events = 0;
  {
    // W slab j = of every vocabulary split of the statistics kernel, its j-th run of tiles: exactly what cut j
    // of the first chunk's sweep reads
    const int q = pl.tensor ? w_slab_tiles(pl, w_slabs) : n_tiles_v;
    const int stride = pl.tensor ? pl.tiles_per_split : n_tiles_v;
    const int splits = pl.tensor ? pl.n_split : 1;
    for (int j = 0; j * q < stride; ++j) {
      for (int sp = 0; sp < splits; ++sp) {
        const int tile0 = sp * stride + j * q;
        const int tile1 = std::min(std::min(tile0 + q, (sp + 1) * stride), n_tiles_v);
        if (tile1 <= tile0) continue;
        const size_t v0 = (size_t)tile0 * kBN, v1 = std::min(V, (size_t)tile1 * kBN);
        if (!ok(h2d(L.W + v0 * row_bytes, static_cast<const uint8_t*>(h_W) + v0 * row_bytes, (v1 - v0) * row_bytes)))
          return ULORL_ERR_CUDA;
      }
      if (j < w_slabs && !ok(cudaEventRecord(hs->chunk_in[w_event0 + j], hs->in))) return ULORL_ERR_CUDA;
      n_w_events = std::min(j + 1, w_slabs);
    }
  }
  for (int c = 1; c < n_chunks; ++c)
    if (!send_chunk(c)) return ULORL_ERR_CUDA;
  auto chunk_of = [&](int t) {       // index of the chunk that holds token t
    int c = 0;
    while (c + 1 < n_chunks && hooks.chunk_starts[c + 1] <= t) ++c;
    return c;
  };
  const bool sweep_by_slabs = pl.tensor && w_slabs > 1;
  hooks.before_stats_chunk = [&](int t0, int rows) {   // the last chunk that [t0, t0 + rows) touches has landed
    if (!ok(cudaStreamWaitEvent(stream, hs->chunk_in[chunk_of(t0 + rows - 1)], 0))) return (int)ULORL_ERR_CUDA;
    // W follows the first chunk on the inbound stream: without the slab-wise sweep all of it must be there
    if (!sweep_by_slabs && n_w_events > 0 &&
        !ok(cudaStreamWaitEvent(stream, hs->chunk_in[w_event0 + n_w_events - 1], 0)))
      return (int)ULORL_ERR_CUDA;
    return (int)ULORL_OK;
  };
  if (sweep_by_slabs) {
    hooks.w_slabs = w_slabs;
    hooks.before_w_slab = [&](int j) {
      return ok(cudaStreamWaitEvent(stream, hs->chunk_in[w_event0 + j], 0)) ? ULORL_OK : ULORL_ERR_CUDA;
    };
  }
  // d_hidden rows of a panel go back on the outbound stream while the next panel is computed
  hooks.after_dhidden_panel = [&](int t0, int rows) {
    if (!h_d_hidden) return (int)ULORL_OK;
    const int c = t0 / chunk;
    if (!ok(cudaEventRecord(hs->panel_out[c], stream)) || !ok(cudaStreamWaitEvent(hs->out, hs->panel_out[c], 0)) ||
        !ok(cudaMemcpyAsync(static_cast<uint8_t*>(h_d_hidden) + (size_t)t0 * row_bytes,
                            a + L.d_hidden + (size_t)t0 * row_bytes, (size_t)rows * row_bytes, cudaMemcpyDeviceToHost,
                            hs->out)))
      return (int)ULORL_ERR_CUDA;
    return (int)ULORL_OK;
  };
  // d_W rows go back slab by slab while the last panel is still being computed
  size_t n_slabs = 0;
  bool dw_by_slabs = false;
  const size_t dw_elem = params->dw_dtype == ULORL_BF16 ? 2 : 4;
  if (pl.tensor && h_d_W) {
    hooks.after_dw_slab = [&](int v0, int v_rows) {
      cudaEvent_t e = hs->slab_event(n_slabs++);
      if (!e || !ok(cudaEventRecord(e, stream)) || !ok(cudaStreamWaitEvent(hs->out, e, 0)) ||
          !ok(cudaMemcpyAsync(static_cast<uint8_t*>(h_d_W) + (size_t)v0 * H * dw_elem,
                              a + L.d_W + (size_t)v0 * H * dw_elem, (size_t)v_rows * H * dw_elem,
                              cudaMemcpyDeviceToHost, hs->out)))
        return (int)ULORL_ERR_CUDA;
      dw_by_slabs = true;
      return (int)ULORL_OK;
    };
    if (L.dz2) hooks.dz_second_buffer = a + L.dz2;
  }
  st = fwd_impl(params, a + L.hidden, a + L.W, reinterpret_cast<const int32_t*>(a + L.targets),
                h_old_logp ? reinterpret_cast<const float*>(a + L.old_logp) : nullptr,
                (h_ref_logp && params->kl_beta > 0.f) ? reinterpret_cast<const float*>(a + L.ref_logp) : nullptr,
                h_segment_version ? reinterpret_cast<const int32_t*>(a + L.segver) : nullptr,
                reinterpret_cast<const float*>(a + L.adv), reinterpret_cast<const int32_t*>(a + L.seq_off),
                h_entropy_supplied ? reinterpret_cast<const float*>(a + L.ent_sup) : nullptr,
                reinterpret_cast<float*>(a + L.logp), reinterpret_cast<float*>(a + L.entropy),
                reinterpret_cast<float*>(a + L.lse), reinterpret_cast<float*>(a + L.grad_coef), a + L.flags,
                reinterpret_cast<float*>(a + L.seq_entropy), reinterpret_cast<float*>(a + L.loss), a + L.stats, a + L.ws,
                L.total - L.ws, stream, &hooks);
  if (st != ULORL_OK) return st;
  // the host buffers are free again once the inbound stream has read them
  if (!ok(cudaEventRecord(hs->start, hs->in)) || !ok(cudaStreamWaitEvent(stream, hs->start, 0))) return ULORL_ERR_CUDA;
  auto d2h = [&](void* dst, size_t off, size_t bytes) {
    return (!dst || !bytes) ? cudaSuccess : cudaMemcpyAsync(dst, a + off, bytes, cudaMemcpyDeviceToHost, stream);
  };
  if (!ok(d2h(h_logp, L.logp, T * 4)) || !ok(d2h(h_entropy, L.entropy, T * 4)) || !ok(d2h(h_flags, L.flags, T)) ||
      !ok(d2h(h_seq_entropy, L.seq_entropy, S * 4)) || !ok(d2h(h_loss, L.loss, 4)) ||
      !ok(d2h(h_stats, L.stats, sizeof(ulorl_stats_t))))
    return ULORL_ERR_CUDA;
  st = bwd_impl(params, a + L.hidden, a + L.W, reinterpret_cast<const int32_t*>(a + L.targets),
                reinterpret_cast<const float*>(a + L.lse), reinterpret_cast<const float*>(a + L.grad_coef), nullptr,
                a + L.d_hidden, a + L.d_W, a + L.ws, L.total - L.ws, stream, &hooks);
  if (st != ULORL_OK) return st;
  // with compaction d_hidden is only final after the scatter at the end of the backward
  if (pl.compact && !ok(d2h(h_d_hidden, L.d_hidden, T * row_bytes))) return ULORL_ERR_CUDA;
  if (!dw_by_slabs && !ok(d2h(h_d_W, L.d_W, V * H * dw_elem))) return ULORL_ERR_CUDA;
  // the caller's stream is done only when the outbound copies are
  if (!ok(cudaEventRecord(hs->out_done, hs->out)) || !ok(cudaStreamWaitEvent(stream, hs->out_done, 0))) return ULORL_ERR_CUDA;
  return ULORL_OK;
}

}  // extern "C"
