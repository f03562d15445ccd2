// libgbmuf: the random-gossip BMUF synchronisation round (Algorithm 1 of "A Random Gossip BMUF
// Process for Neural Language Modeling") for K parameter replicas resident in one GPU's memory.
// CUDA for sm_100a.  The interface is include/gbmuf.h; this file holds the host side and the C
// ABI, the kernels live in the headers it includes:
//   philox.cuh           Philox4x32-10
//   round_setup.cuh      round_setup_kernel: neighbour draws for every (worker, component) of a
//                        round + the tile work-list prefix of the components that take part
//   primitives.cuh       bounded barrier waits, bulk copies, theta storage types
//   sync_fused.cuh       sync_fused_kernel: gather + average + block-momentum filter, one pass, in
//                        place, theta tile in shared memory (also gossip-MA)
//   sync_fused_tmem.cuh  sync_fused_tmem_kernel: the same with the theta tile in tensor memory and
//                        bulk stores (the default in gossip-BMUF mode); with many workers only a
//                        window of rows along the ring is resident; device self-tests
//   sync_ma_window.cuh   sync_ma_window_kernel: gossip-MA with many workers, a window of rows
//                        along the ring in shared memory
//   local_step.cuh       perturb_kernel (synthetic local steps), the Adagrad local step,
//                        init_stream_kernel (theta^k <- theta_0, omega^k <- theta_0, Delta^k <- 0),
//                        final_average_kernel (theta = (1/K) sum_k theta^k)
//   peer.cuh             one worker per GPU over peer-mapped buffers
//
// Floating point: every operation of Algorithm 1 is an explicit round-to-nearest intrinsic
// (__fadd_rn, __fmul_rn, ...) so that nothing is contracted into a fused multiply-add; the one
// fused multiply-add in use sits inside the averaging division (sync_fused.cuh), whose result is
// the correctly rounded quotient.

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <type_traits>
#include <vector>

#include "gbmuf.h"

#include "philox.cuh"
#include "round_setup.cuh"
#include "primitives.cuh"
#include "sync_fused.cuh"
#include "sync_fused_tmem.cuh"
#include "sync_ma_window.cuh"
#include "local_step.cuh"
#include "peer.cuh"

namespace {

// =================================================================================================
// Host side
// =================================================================================================
thread_local std::string g_create_error;

struct Tuning {
  int ncons = 0, T = 0, stages = 0, ring = 0, flags = 0;   // 0 = built-in choice
};

struct Launch {
  int ncons, stages, ring, T, BW, flags;
  uint32_t stage_stride, nbr_off, desc_off, ring_off, slot_stride, smem;
  int tmem_cols;                     // TMEM variant: columns to allocate (0 = shared-memory tile)
  uint32_t meta_off, meta_stride;
  // TMEM variant, which rows of a tile are resident: all K (win_rows = cell_rows = npos = K,
  // lead = K, pshift = 0) or a window along the ring plus the kept first p rows
  int win_rows, cell_rows, npos, lead, pshift, keep_lo;
  // gossip-MA ring window in shared memory (sync_ma_window_kernel): ring slots (0 = not in use),
  // offsets of the two kept-row sets and of the ring
  int ma_ring;
  uint32_t kept_off;
};

int host_candidates(int K, int p) {
  long long c = 2LL * p;
  if (c > K - 1) c = K - 1;
  return (int)c;
}

// Is `st` recording a stream capture?  (The legacy default stream never is.)
bool is_capturing(cudaStream_t st) {
  if (!st) return false;
  cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cs) != cudaSuccess) { cudaGetLastError(); return false; }
  return cs != cudaStreamCaptureStatusNone;
}

// Which streams a handle has put work into, as one event per stream recorded after the latest
// piece of work.  Re-partitioning and destruction wait for these events: for the handle's own
// work and nothing else on the device.  Events outlive the streams they were recorded in, so a
// stream the caller has destroyed in the meantime is no problem.  Work recorded into a stream
// capture is not tracked (an event recorded there cannot be waited for from the host); the
// caller keeps the handle alive while such a graph can still run.
struct WorkMarks {
  struct Mark { cudaStream_t s; cudaEvent_t ev; };
  std::vector<Mark> marks;
  static constexpr size_t kMaxStreams = 16;
  void note(cudaStream_t st) {
    if (is_capturing(st)) return;
    for (Mark& mk : marks)
      if (mk.s == st) { cudaEventRecord(mk.ev, st); return; }
    if (marks.size() == kMaxStreams) {               // many streams: retire the oldest mark
      cudaEventSynchronize(marks.front().ev);
      cudaEventDestroy(marks.front().ev);
      marks.erase(marks.begin());
    }
    Mark mk{st, nullptr};
    if (cudaEventCreateWithFlags(&mk.ev, cudaEventDisableTiming) != cudaSuccess) { cudaGetLastError(); return; }
    cudaEventRecord(mk.ev, st);
    marks.push_back(mk);
  }
  cudaError_t wait() {
    cudaError_t first = cudaSuccess;
    for (Mark& mk : marks) {
      const cudaError_t e = cudaEventSynchronize(mk.ev);
      if (e != cudaSuccess && first == cudaSuccess) first = e;
    }
    return first;
  }
  void release() {
    for (Mark& mk : marks) cudaEventDestroy(mk.ev);
    marks.clear();
  }
};

}  // namespace

struct gbmuf_ctx {
  gbmuf_config cfg;
  void* theta;
  float* omega;
  float* delta;
  int m = 0;
  int cand = 0;
  bool partitioned = false;
  std::vector<int64_t> off;
  std::vector<int32_t> periods;
  int64_t* d_off = nullptr;
  int32_t* d_periods = nullptr;
  uint8_t* d_mask = nullptr;
  int32_t* d_prefix = nullptr;
  int32_t* d_nbr = nullptr;
  int32_t* d_nbr_export = nullptr;
  int32_t* d_status = nullptr;
  double* d_norm_partial = nullptr;   // [K][kNormBlocks], local_adagrad
  float* d_clip_scale = nullptr;      // [K]
  cudaStream_t priv = nullptr;
  int num_sms = 0;
  int max_smem = 0;        // opt-in dynamic shared memory per block
  int smem_per_sm = 0;
  Tuning tuning;
  Launch launch;
  CUtensorMap map_theta;   // boxes [K rows][launch.BW columns] over theta
  std::vector<uint8_t> mask_stage;   // the library's own (pageable) copy of a caller's mask
  int cap_m = 0;                     // sizes the device tables were allocated for
  size_t cap_nbr_bytes = 0;
  WorkMarks work;
  std::string err;
};

namespace {

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { prev = -1; }
    if (prev != dev) ok = (cudaSetDevice(dev) == cudaSuccess);
  }
  ~DeviceGuard() {
    int cur = -1;
    if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
  }
};

gbmuf_status fail(gbmuf_ctx* ctx, gbmuf_status st, const std::string& msg) {
  if (ctx) ctx->err = msg; else g_create_error = msg;
  return st;
}

gbmuf_status cuda_fail(gbmuf_ctx* ctx, const char* what, cudaError_t e) {
  return fail(ctx, GBMUF_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

size_t theta_size(const gbmuf_ctx* c) { return c->cfg.theta_dtype == GBMUF_F32 ? 4 : 2; }

// The streaming kernels use more dynamic shared memory than a kernel gets by default; the limit
// is a per-device property of each kernel and is raised once per device (that device current),
// when a handle is created, not on every launch.
std::mutex g_attr_mutex;
constexpr int kAttrDevices = 64;
bool g_attr_done[kAttrDevices] = {};

cudaError_t ensure_kernel_attributes(int device, int max_smem) {
  std::lock_guard<std::mutex> lock(g_attr_mutex);
  if (device >= 0 && device < kAttrDevices && g_attr_done[device]) return cudaSuccess;
  const void* kernels[] = {
      (const void*)sync_fused_tmem_kernel<float, true, true>, (const void*)sync_fused_tmem_kernel<float, true, false>,
      (const void*)sync_fused_tmem_kernel<float, false, true>, (const void*)sync_fused_tmem_kernel<float, false, false>,
      (const void*)sync_fused_tmem_kernel<__nv_bfloat16, true, true>, (const void*)sync_fused_tmem_kernel<__nv_bfloat16, true, false>,
      (const void*)sync_fused_tmem_kernel<__nv_bfloat16, false, true>, (const void*)sync_fused_tmem_kernel<__nv_bfloat16, false, false>,
      (const void*)sync_fused_kernel<float>, (const void*)sync_fused_kernel<__nv_bfloat16>,
      (const void*)sync_ma_window_kernel<float, 1>, (const void*)sync_ma_window_kernel<__nv_bfloat16, 1>,
      (const void*)init_stream_kernel<float>, (const void*)init_stream_kernel<__nv_bfloat16>,
      (const void*)adagrad_stream_kernel<float>, (const void*)adagrad_stream_kernel<__nv_bfloat16>,
      (const void*)peer_round_kernel<float>, (const void*)peer_round_kernel<__nv_bfloat16>};
  for (const void* k : kernels) {
    const cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
    if (e != cudaSuccess) return e;
  }
  if (device >= 0 && device < kAttrDevices) g_attr_done[device] = true;
  return cudaSuccess;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Tensor map for boxes of K rows x BW columns over the [K][ld] theta array.
gbmuf_status build_tensor_maps(gbmuf_ctx* ctx, const Launch& L) {
  if (L.tmem_cols > 0 || L.ma_ring > 0) return GBMUF_OK;   // these variants stage rows by 1-D copies
  static EncodeTiledFn encode = nullptr;
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn)
      return fail(ctx, GBMUF_ERR_CUDA, "the driver does not provide cuTensorMapEncodeTiled");
    encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  const cuuint64_t ld = (cuuint64_t)ctx->cfg.ld;
  const cuuint64_t gdim[2] = {ld, (cuuint64_t)ctx->cfg.K};
  const cuuint32_t box[2] = {(cuuint32_t)L.BW, (cuuint32_t)ctx->cfg.K};
  const cuuint32_t estr[2] = {1, 1};
  const CUtensorMapL2promotion prom =
      (L.flags & 1) ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B;
  const cuuint64_t esz = (cuuint64_t)theta_size(ctx);
  const cuuint64_t gstride[1] = {ld * esz};
  CUresult r = encode(&ctx->map_theta,
                      ctx->cfg.theta_dtype == GBMUF_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                                        : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                      2, ctx->theta, gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                      CU_TENSOR_MAP_SWIZZLE_NONE, prom, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS)
    return fail(ctx, GBMUF_ERR_CUDA, "cuTensorMapEncodeTiled failed with code " + std::to_string((int)r));
  return GBMUF_OK;
}

// Choose (or check) the launch shape of the fused kernel for this K, q, mode and dtype.
// Shared memory: 256 bytes of barriers, `stages` theta stages of K*T elements (+ neighbour table
// and descriptor), and in BMUF mode `ring` slots of 2*T floats.
gbmuf_status plan_launch(gbmuf_ctx* ctx, const Tuning& t, Launch* out) {
  const int K = ctx->cfg.K, q = ctx->cfg.q;
  const int esz = (int)theta_size(ctx);
  const bool bmuf = ctx->cfg.mode == GBMUF_MODE_BMUF;
  Launch L;
  L.flags = t.flags;
  L.tmem_cols = 0; L.meta_off = 0; L.meta_stride = 0;
  L.win_rows = 0; L.cell_rows = 0; L.npos = 0; L.lead = 0; L.pshift = 0; L.keep_lo = 0;
  L.ma_ring = 0; L.kept_off = 0;
  const long long cap = ctx->max_smem < ctx->smem_per_sm - 1024 ? ctx->max_smem : ctx->smem_per_sm - 1024;
  // Variant: flags bit 3 forces the shared-memory theta tile, bit 1 forces the tensor-memory tile
  // (bit 2: with bulk stores); with neither, the tensor-memory tile with bulk stores is used
  // wherever it applies (gossip-BMUF, resident rows that fit) -- it is the faster one.  Bit 4
  // forces, bit 5 forbids the ring window of the tensor-memory tile.
  const int cw = esz == 4 ? 4 : 2;                       // TMEM columns per group of 4 elements
  const int in_rows = 8 / esz;                           // theta rows per load item
  // Rows resident in tensor memory: all K, or -- Definition 1's ring: a worker only averages with
  // workers within distance p -- a window of 2p + in_rows rows that slides along the ring plus
  // the first p rows kept for the last workers.  The window needs 2p + in_rows < K (then also
  // 2p < K - 1 and signed ring distances are unambiguous).
  const int p = ctx->cfg.p;
  // Window, kept rows: the first p rows always; the last p rows are either requested twice
  // (3p + in_rows cell rows) or kept too (4p + in_rows cell rows, every row read once).  The
  // second form is taken when it costs no tile width (or on request: flags bit 6).
  const int win_w = 2 * p + in_rows, cells_twice = win_w + p, cells_once = win_w + 2 * p;
  // widths whose element groups share out evenly over the consumer warps measured best for the
  // window (fp32, K = 64..256: 4096 x 4 slots, 3072 x 6, 2048 x 8 ahead of 3584 x 4; 2560 x 6 since a
  // thread's element groups are taken in pairs: 5 groups per row beat 4;
  // bf16: 5120 x 4 and 4096 x 4 ahead of 3584 x 6 and 3072 x 6), the ring as deep as fits
  static const int kWinF32[][2] = {{4096, 4}, {3072, 6}, {2560, 6}, {2048, 8}, {1024, 8}, {512, 8}};
  static const int kWinBf16[][2] = {{5120, 4}, {4096, 4}, {3584, 6}, {3072, 6}, {2048, 8}, {1024, 8}, {512, 8}};
  auto window_shape = [&](int rows, int* ring) {         // widest listed tile for `rows` cell rows
    const int (*tab)[2] = esz == 4 ? kWinF32 : kWinBf16;
    const int n = esz == 4 ? 6 : 7;
    for (int i = 0; i < n; ++i)
      if ((tab[i][0] / 512) * rows * cw <= 512) { if (ring) *ring = tab[i][1]; return tab[i][0]; }
    return 0;
  };
  const bool keep_both = (t.flags & 64) != 0 ||
                         (!t.T && window_shape(cells_once, nullptr) >= window_shape(cells_twice, nullptr) &&
                          window_shape(cells_once, nullptr) > 0);
  const int win_cells = keep_both ? cells_once : cells_twice;
  const bool win_possible = win_w < K;
  // measured with 16 replicas: fp32 3584 x 4 slots; bf16 4096 x 4 slots (3072 x 6 is as fast when
  // rounds are far apart but 4 % slower when they run back to back under the power cap)
  const int T_default = esz == 4 ? 3584 : 4096;
  auto fits_cols = [&](int T, int rows) { return T >= 512 && T % 512 == 0 && (T / 512) * rows * cw <= 512; };
  auto widest = [&](int rows) {                          // widest tile up to the default, 0 = none
    int T = T_default;
    while (T > 512 && !fits_cols(T, rows)) T -= 512;
    return fits_cols(T, rows) ? T : 0;
  };
  if ((t.flags & 16) && (t.flags & 32))
    return fail(ctx, GBMUF_ERR_INVALID_ARG, "flags bits 4 and 5 (force / forbid the ring window) exclude each other");
  if ((t.flags & 16) && bmuf && !win_possible)
    return fail(ctx, GBMUF_ERR_UNSUPPORTED, "the ring window needs 2p + rows per load item < K");
  bool use_win = false;
  if (win_possible && !(t.flags & 32)) {
    if (t.flags & 16) use_win = true;
    else if (t.T) use_win = !fits_cols(t.T, K) && fits_cols(t.T, win_cells);
    else use_win = widest(cells_twice) > widest(K);      // the window buys a wider tile
  }
  const int cells = use_win ? win_cells : K;
  const bool tmem_ok = bmuf && widest(cells) > 0;
  // (automatic choice only when the caller has not asked for anything specific to the
  // shared-memory tile: consumer threads, theta stages, or a tile width it cannot have)
  const bool auto_tmem = !(t.flags & 8) && tmem_ok && t.ncons == 0 && t.stages == 0 &&
                         (t.T == 0 || fits_cols(t.T, cells));
  const bool want_tmem = (t.flags & 2) || (bmuf && (t.flags & 16)) || auto_tmem;
  if (((t.flags & 2) || (bmuf && (t.flags & 16))) && !tmem_ok)
    return fail(ctx, GBMUF_ERR_UNSUPPORTED, "the tensor-memory variant needs gossip-BMUF mode and resident rows that fit 512 columns (K <= 128, or a ring window)");
  if (want_tmem) {
    const bool forced = (t.flags & 2) != 0 || (bmuf && (t.flags & 16) != 0);
    const bool bulk = (t.flags & 2) ? (t.flags & 4) != 0 : true;
    // theta tile in tensor memory: cells * (T/512) * cw <= 512 columns; T a multiple of 512
    int T = t.T ? t.T : widest(cells), ring_pref = 0;
    if (use_win && !t.T && bulk) {
      const int Tw = window_shape(cells, &ring_pref);
      if (Tw > 0) T = Tw; else ring_pref = 0;
    }
    const bool fits = fits_cols(T, cells);
    if (!fits && (forced || t.T))
      return fail(ctx, GBMUF_ERR_INVALID_ARG, "tensor-memory variant: tile_elems must be a multiple of 512 whose resident rows fit 512 columns of tensor memory");
    if (fits) {
      L.T = T; L.BW = 256; L.stages = 1;
      L.ncons = 512;
      L.flags = (t.flags & 1) | 2 | (bulk ? 4 : 0) | (use_win ? 16 : 0);
      L.win_rows = use_win ? win_w : K; L.cell_rows = cells;
      L.npos = use_win && !keep_both ? K + p : K; L.lead = use_win ? 2 * p : K; L.pshift = use_win ? p : 0;
      L.keep_lo = keep_both ? 0 : p;
      L.meta_off = 512;
      L.meta_stride = (uint32_t)(((long long)sizeof(TileDesc) + (long long)K * q * 4 + 127) / 128 * 128);
      L.ring_off = L.meta_off + 4 * L.meta_stride;
      L.slot_stride = (uint32_t)((bulk ? 8 + esz : 8) * T);
      // ring items per tile; the 4-entry descriptor ring needs the producer to stay within three
      // tiles of the consumers, i.e. a ring no deeper than three tiles' worth of items
      const int per_tile = (L.npos + in_rows - 1) / in_rows + K;
      const int ring_cap = 3 * per_tile < kMaxRing ? 3 * per_tile : kMaxRing;
      // Ring depth: 4 slots of the default width measured best (3 starve the pipeline, 5 and more
      // put too much in flight; even counts did better than odd ones); narrower slots: more of them.
      int R = t.ring ? t.ring : ring_pref ? ring_pref : (bulk ? 4 : 3);
      while (!t.ring && R > 2 && (long long)L.ring_off + (long long)R * L.slot_stride > cap) --R;
      while (!t.ring && !ring_pref && bulk && R + 2 <= ring_cap && (long long)R * L.slot_stride < 160 * 1024 &&
             (long long)L.ring_off + (long long)(R + 2) * L.slot_stride <= cap) R += 2;
      if (!t.ring && R > ring_cap) R = ring_cap;
      const bool ring_fits = (long long)L.ring_off + (long long)R * L.slot_stride <= cap && R >= 2 && R <= ring_cap;
      if (!ring_fits && (forced || t.ring))
        return fail(ctx, GBMUF_ERR_UNSUPPORTED, "tensor-memory variant: the ring does not fit shared memory (or is deeper than three tiles)");
      if (ring_fits) {
        L.ring = R;
        L.smem = (uint32_t)(L.ring_off + (long long)R * L.slot_stride);
        int cols = 32;
        while (cols < (T / 512) * cells * cw) cols <<= 1;
        L.tmem_cols = cols;
        L.stage_stride = 0; L.nbr_off = 0; L.desc_off = 0;
        *out = L;
        return GBMUF_OK;
      }
    }
  }
  L.flags = t.flags & 1;
  // gossip-MA with many workers: the ring window in shared memory (sync_ma_window_kernel).  Rows
  // of 8, 6, 4, 2 KB; two sets of p kept rows; a ring of 2p + 4 live rows (four workers are computed
  // at a time) plus rows in flight ahead of them.  Taken for fp32 theta from 192 workers on (the
  // only place where it measured faster than all K rows of a narrow tile: 3.3 against 2.6 TB/s
  // at K = 256; its consumers are bound by instruction latency), on request (flags bit 4),
  // never with bit 5.
  if (!bmuf && !(t.flags & (8 | 32)) && K >= 2 * p + 2 && t.ncons == 0 && t.stages == 0 &&
      ((t.flags & 16) || (K >= 192 && esz == 4))) {
    const int mv = 16 / esz;                                 // elements per 16 bytes
    const long long meta_stride = ((long long)sizeof(TileDesc) + (long long)K * q * 4 + 127) / 128 * 128;
    const long long fixed = (long long)kMwBarBytes + 2 * meta_stride;
    auto ring_for_rows = [&](int T) {                        // ring slots that fit beside the kept rows
      const long long rows = (cap - fixed) / ((long long)T * esz);
      long long R = rows - 2LL * p;
      if (R > kMaWinMaxRing) R = kMaWinMaxRing;
      return (int)R;
    };
    int T = 0, R = 0;
    if (t.T) {
      T = t.T;
      R = t.ring ? t.ring : ring_for_rows(T);
    } else {
      // The widest row whose ring still has two slots beyond the live ones: the round's time
      // turned out proportional to the number of rows, not to what is in flight (measured with
      // 64 workers: 8 KB rows with 4 rows ahead 4.3 TB/s, 4 KB rows with 31 ahead 2.5 TB/s).
      static const int kRowBytes[] = {8192, 6144, 4096, 2048};
      for (int i = 0; i < 4 && !T; ++i) {
        const int Tc = kRowBytes[i] / esz, Rc = t.ring ? t.ring : ring_for_rows(Tc);
        if (Rc >= 2 * p + kMwUnroll + 2) { T = Tc; R = Rc; }
      }
    }
    const bool shape_ok = T > 0 && T % (mv * 32) == 0 && T / mv <= 512 && R >= 2 * p + kMwUnroll + 2 && R <= kMaWinMaxRing &&
                          fixed + (2LL * p + R) * T * esz <= cap;
    if (!shape_ok && ((t.flags & 16) || t.T))
      return fail(ctx, GBMUF_ERR_UNSUPPORTED, "gossip-MA ring window: tile_elems must be a multiple of 32 16-byte vectors, "
                                              "at most 512 of them, with 2p kept rows and a ring of 2p + 6 .. 64 rows in shared memory");
    if (shape_ok) {
      L.T = T; L.BW = 256; L.stages = 1; L.ring = 0; L.ncons = T / mv;   // one 16-byte piece per thread and row
      L.flags = (t.flags & 1) | 16;
      L.ma_ring = R;
      L.meta_off = kMwBarBytes; L.meta_stride = (uint32_t)meta_stride;
      L.kept_off = (uint32_t)fixed;
      L.ring_off = (uint32_t)(fixed + 2LL * p * T * esz);
      L.slot_stride = (uint32_t)(T * esz);
      L.smem = (uint32_t)(L.ring_off + (long long)R * T * esz);
      L.stage_stride = 0; L.nbr_off = 0; L.desc_off = 0;
      *out = L;
      return GBMUF_OK;
    }
  } else if ((t.flags & 16) && !bmuf) {
    return fail(ctx, GBMUF_ERR_UNSUPPORTED, "the gossip-MA ring window needs K >= 2p + 2 and no consumer_threads / theta_stages setting");
  }
  auto stage_bytes = [&](int T, Launch* l) {
    long long at = ((long long)K * T * esz + 15) / 16 * 16;
    if (l) l->nbr_off = (uint32_t)at;
    at = (at + (long long)K * q * 4 + 15) / 16 * 16;
    if (l) l->desc_off = (uint32_t)at;
    at += (long long)sizeof(TileDesc);
    return (at + 127) / 128 * 128;
  };
  auto total_bytes = [&](int T, int S, int R) {
    return (long long)kBarBytes + S * stage_bytes(T, nullptr) + (bmuf ? (long long)R * 2 * T * 4 : 0);
  };
  // gossip-MA stages only theta, so it can afford (and needs) a second stage to overlap
  int want_stages = t.stages ? t.stages : (bmuf ? 1 : 2);
  auto ring_for = [&](int T) {   // slots used with tile T: the caller's, else as many as fit up to 4
    if (!bmuf) return 0;
    if (t.ring) return t.ring;
    int r = 4;
    while (r > 2 && total_bytes(T, want_stages, r) > cap) --r;
    return r;
  };
  if (t.T) {
    L.T = t.T;
    if (!t.stages && want_stages > 1 && total_bytes(L.T, want_stages, ring_for(L.T)) > cap) want_stages = 1;
  } else {
    // The widest power-of-two tile (longest contiguous run per row) that fits: measured DRAM
    // efficiency keeps growing with the run length up to 16 KB, and a tile that is a whole
    // number of consumer passes keeps every thread busy.
    int T = 4096;
    while (T > 8 && total_bytes(T, want_stages, ring_for(T)) > cap) T >>= 1;
    L.T = T;
  }
  L.ring = ring_for(L.T);
  if (L.T < kAlign || L.T % kAlign != 0)
    return fail(ctx, GBMUF_ERR_INVALID_ARG, "tile_elems must be a positive multiple of 8");
  if (L.T > 256 && L.T % 256 != 0)
    return fail(ctx, GBMUF_ERR_INVALID_ARG, "tile_elems above 256 must be a multiple of 256");
  L.BW = L.T < 256 ? L.T : 256;                // a tensor-map box is at most 256 elements wide
  L.stages = want_stages;
  if ((long long)K * L.T * esz >= (1 << 20) || total_bytes(L.T, L.stages, L.ring) > cap)
    return fail(ctx, GBMUF_ERR_UNSUPPORTED,
                "the theta stage(s) (K rows of the tile) and the omega/Delta ring do not fit the "
                "shared memory of one SM");
  const long long sb = stage_bytes(L.T, &L);
  L.stage_stride = (uint32_t)sb;
  L.ring_off = (uint32_t)(kBarBytes + L.stages * sb);
  L.slot_stride = (uint32_t)(2 * L.T * 4);
  L.smem = (uint32_t)total_bytes(L.T, L.stages, L.ring);
  if (t.ncons) {
    L.ncons = t.ncons;
  } else {
    int n = (L.T / 4 + 31) / 32 * 32;          // one quad per thread and row, within 128..992
    L.ncons = n < 128 ? 128 : n > 992 ? 992 : n;
    if (!bmuf) {                               // gossip-MA: 16 bytes of theta per thread and row,
      const int per = L.T / (16 / esz);        // and thread groups that share out the workers
      if (per >= 32 && per <= 496) L.ncons = per * (992 / per);
      else { n = (per + 31) / 32 * 32; L.ncons = n < 128 ? 128 : n > 992 ? 992 : n; }
    }
  }
  *out = L;
  return GBMUF_OK;
}

long long host_total_tiles(const gbmuf_ctx* ctx, uint64_t round, const uint8_t* mask, int T) {
  long long total = 0;
  for (int i = 0; i < ctx->m; ++i) {
    const bool due = mask ? mask[i] != 0 : (round % (uint64_t)ctx->periods[i] == 0);
    if (!due) continue;
    const int64_t lo = ctx->off[i], hi = ctx->off[i + 1];
    if (hi <= lo) continue;
    const int64_t start = lo & ~(int64_t)(kAlign - 1);
    total += (hi - start + T - 1) / T;
  }
  return total;
}

// Everything the fused kernel needs to know about one launch.
void fill_sync_params(const gbmuf_config& cfg, const Launch& L, void* theta, float* omega,
                      float* delta, long long ld, int m, const int64_t* off, const int32_t* prefix,
                      const int32_t* nbr, int32_t* status, SyncParams* P) {
  P->theta = theta; P->omega = omega; P->delta = delta;
  P->off = off; P->tile_prefix = prefix; P->nbr = nbr; P->status = status;
  P->ld = ld; P->K = cfg.K; P->m = m; P->q = cfg.q; P->mode = cfg.mode;
  P->eta = cfg.eta; P->zeta = cfg.zeta;
  const int qp1 = cfg.q + 1;
  P->qp1 = (float)qp1; P->inv_qp1 = 1.0f / (float)qp1; P->inv_exact = (qp1 & (qp1 - 1)) == 0;
  P->T = L.T; P->BW = L.BW; P->stages = L.stages; P->ring = L.ring; P->ncons = L.ncons;
  if (L.T > L.BW) { P->bw_shift = 8; P->bw_mask = 255; }          // several boxes of 256 columns
  else { P->bw_shift = 30; P->bw_mask = (1 << 30) - 1; }          // one box
  P->stage_stride = L.stage_stride; P->nbr_off = L.nbr_off; P->desc_off = L.desc_off;
  P->ring_off = L.ring_off; P->slot_stride = L.slot_stride;
}

// Launches the fused round in the variant the launch shape names.  `ctx` supplies the error
// slot, the device limits and (shared-memory variant) the tensor map of theta.  The kernels'
// shared-memory limit has been raised before (ensure_kernel_attributes).
gbmuf_status launch_round(gbmuf_ctx* ctx, const gbmuf_config& cfg, const Launch& L, void* theta,
                          float* omega, float* delta, long long ld, int m, const int64_t* off,
                          const int32_t* prefix, const int32_t* nbr, int32_t* status,
                          long long total, cudaStream_t st) {
  const int grid = (int)(total < ctx->num_sms ? total : ctx->num_sms);   // one persistent CTA per SM
  SyncParams P;
  fill_sync_params(cfg, L, theta, omega, delta, ld, m, off, prefix, nbr, status, &P);
  // Programmatic dependent launch: the kernel may start while the round set-up kernel before it
  // in the stream still runs; it waits for that kernel (grid_dependency_wait) before it reads the
  // tables.
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3((unsigned)grid, 1, 1);
  lc.dynamicSmemBytes = L.smem;
  lc.stream = st;
  lc.attrs = attr;
  lc.numAttrs = 1;
  cudaError_t e;
  if (L.tmem_cols > 0) {
    TmemParams Q;
    Q.theta_in = theta; Q.theta = theta; Q.omega = omega; Q.delta = delta;
    Q.off = off; Q.tile_prefix = prefix; Q.nbr = nbr; Q.status = status;
    Q.ld = ld; Q.K = cfg.K; Q.m = m; Q.q = cfg.q;
    Q.eta = P.eta; Q.zeta = P.zeta; Q.qp1 = P.qp1; Q.inv_qp1 = P.inv_qp1; Q.inv_exact = P.inv_exact;
    Q.T = L.T; Q.ring = L.ring; Q.ncols = L.tmem_cols;
    Q.W = L.win_rows; Q.wtot = L.cell_rows; Q.npos = L.npos; Q.lead = L.lead; Q.pshift = L.pshift; Q.keep_lo = L.keep_lo;
    Q.ring_off = L.ring_off; Q.meta_off = L.meta_off; Q.meta_stride = L.meta_stride; Q.slot_stride = L.slot_stride;
    const bool bulk = (L.flags & 4) != 0, bf = cfg.theta_dtype != GBMUF_F32, win = L.pshift > 0 || L.cell_rows < cfg.K;
    void (*kern)(const TmemParams);
    if (bf)
      kern = bulk ? (win ? sync_fused_tmem_kernel<__nv_bfloat16, true, true> : sync_fused_tmem_kernel<__nv_bfloat16, true, false>)
                  : (win ? sync_fused_tmem_kernel<__nv_bfloat16, false, true> : sync_fused_tmem_kernel<__nv_bfloat16, false, false>);
    else
      kern = bulk ? (win ? sync_fused_tmem_kernel<float, true, true> : sync_fused_tmem_kernel<float, true, false>)
                  : (win ? sync_fused_tmem_kernel<float, false, true> : sync_fused_tmem_kernel<float, false, false>);
    lc.blockDim = dim3(544, 1, 1);
    e = cudaLaunchKernelEx(&lc, kern, Q);
  } else if (L.ma_ring > 0) {
    MaWinParams M;
    M.theta = theta; M.off = off; M.tile_prefix = prefix; M.nbr = nbr; M.status = status;
    M.ld = ld; M.K = cfg.K; M.m = m; M.q = cfg.q; M.p = cfg.p;
    M.qp1 = P.qp1; M.inv_qp1 = P.inv_qp1; M.inv_exact = P.inv_exact;
    M.T = L.T; M.R = L.ma_ring; M.ncons = L.ncons; M.row_bytes = L.slot_stride;
    M.meta_off = L.meta_off; M.meta_stride = L.meta_stride; M.kept_off = L.kept_off; M.ring_off = L.ring_off;
    lc.blockDim = dim3((unsigned)(32 + L.ncons), 1, 1);
    if (cfg.theta_dtype == GBMUF_F32) e = cudaLaunchKernelEx(&lc, sync_ma_window_kernel<float, 1>, M);
    else e = cudaLaunchKernelEx(&lc, sync_ma_window_kernel<__nv_bfloat16, 1>, M);
  } else if (cfg.theta_dtype == GBMUF_F32) {
    lc.blockDim = dim3((unsigned)(32 + L.ncons), 1, 1);
    e = cudaLaunchKernelEx(&lc, sync_fused_kernel<float>, P, ctx->map_theta);
  } else {
    lc.blockDim = dim3((unsigned)(32 + L.ncons), 1, 1);
    e = cudaLaunchKernelEx(&lc, sync_fused_kernel<__nv_bfloat16>, P, ctx->map_theta);
  }
  if (e != cudaSuccess) return cuda_fail(ctx, "launch of the fused round kernel", e);
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, "launch of the fused round kernel", e);
  return GBMUF_OK;
}

// Launches the round set-up kernel as a programmatic dependent of whatever kernel precedes it in
// the stream: it may become resident early and waits (griddepcontrol.wait, its first
// instruction) for that kernel to finish before it touches anything.
cudaError_t launch_setup(const SetupParams& S, cudaStream_t st) {
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t lc = {};
  const long long items = (long long)S.K * S.m;
  lc.gridDim = dim3((unsigned)((items + 255) / 256), 1, 1);
  lc.blockDim = dim3(256, 1, 1);
  lc.dynamicSmemBytes = 0;
  lc.stream = st;
  lc.attrs = attr;
  lc.numAttrs = 1;
  return cudaLaunchKernelEx(&lc, round_setup_kernel, S);
}

void fill_setup(const gbmuf_ctx* ctx, uint64_t round, bool use_mask, bool plan, int32_t* nbr,
                SetupParams* S) {
  S->K = ctx->cfg.K; S->m = ctx->m; S->p = ctx->cfg.p; S->q = ctx->cfg.q;
  S->comp_base = ctx->cfg.comp_base; S->T = ctx->launch.T;
  S->use_mask = use_mask ? 1 : 0; S->plan = plan ? 1 : 0;
  S->seed = ctx->cfg.seed; S->round = round;
  S->off = ctx->d_off; S->periods = ctx->d_periods; S->mask = ctx->d_mask;
  S->nbr = nbr; S->tile_prefix = ctx->d_prefix;
}

int elementwise_grid(const gbmuf_ctx* ctx, long long work_items) {
  long long blocks = (work_items + 255) / 256;
  const long long cap = (long long)ctx->num_sms * 16;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  return (int)blocks;
}

// Blocks per worker row for the kernels that put the worker on blockIdx.y: enough to cover the
// row, capped so that the whole grid is about 16 blocks per SM.
int row_grid(const gbmuf_ctx* ctx, long long vectors_per_row, int K) {
  long long blocks = (vectors_per_row + 255) / 256;
  long long cap = ((long long)ctx->num_sms * 16 + K - 1) / K;
  if (cap < 1) cap = 1;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  return (int)blocks;
}

void free_tables(gbmuf_ctx* ctx) {
  cudaFree(ctx->d_off); cudaFree(ctx->d_periods); cudaFree(ctx->d_mask); cudaFree(ctx->d_prefix);
  cudaFree(ctx->d_nbr); cudaFree(ctx->d_nbr_export);
  ctx->d_off = nullptr; ctx->d_periods = nullptr; ctx->d_mask = nullptr; ctx->d_prefix = nullptr;
  ctx->d_nbr = nullptr; ctx->d_nbr_export = nullptr;
}

}  // namespace

// =================================================================================================
// C ABI
// =================================================================================================
extern "C" {

gbmuf_status gbmuf_create(const gbmuf_config* cfg, void* theta, float* omega, float* delta,
                          gbmuf_ctx** out) {
  if (!cfg || !out) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "cfg and out must not be NULL");
  if (cfg->K < 1) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "K must be >= 1");
  if (cfg->N < 1) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "N must be >= 1");
  if (cfg->ld < cfg->N || cfg->ld % 32 != 0)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "ld must be >= N and a multiple of 32");
  if (cfg->p < 0 || cfg->q < 0) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "p and q must be >= 0");
  if (cfg->mode != GBMUF_MODE_BMUF && cfg->mode != GBMUF_MODE_MA)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "unknown mode");
  if (cfg->theta_dtype != GBMUF_F32 && cfg->theta_dtype != GBMUF_BF16)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "unknown theta_dtype");
  if (cfg->comp_base < 0 || cfg->elem_base < 0)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "comp_base and elem_base must be >= 0");
  if (!(cfg->eta == cfg->eta) || !(cfg->zeta == cfg->zeta))
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "eta and zeta must not be NaN");
  const int cand = host_candidates(cfg->K, cfg->p);
  if (cfg->q > cand)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG,
                "q exceeds the number of ring neighbours min(2p, K-1) (Algorithm 1: q <= 2p)");
  if (cand > kMaxCand)
    return fail(nullptr, GBMUF_ERR_UNSUPPORTED, "more than 64 ring neighbours per worker");
  if (cfg->K > 256)
    return fail(nullptr, GBMUF_ERR_UNSUPPORTED, "more than 256 workers");
  if (cfg->ld > 0x7fffffffLL)
    return fail(nullptr, GBMUF_ERR_UNSUPPORTED, "ld above 2^31 - 1 elements");
  if (!theta || !omega || !delta)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "theta, omega and delta must not be NULL");
  if (((uintptr_t)theta | (uintptr_t)omega | (uintptr_t)delta) % 128 != 0)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "theta, omega and delta must be 128-byte aligned");
  if (cfg->device < 0) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "device must be >= 0");

  int ndev = 0;
  cudaError_t e = cudaGetDeviceCount(&ndev);
  if (e != cudaSuccess) return cuda_fail(nullptr, "cudaGetDeviceCount", e);
  if (cfg->device >= ndev) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "no such CUDA device");
  DeviceGuard guard(cfg->device);
  if (!guard.ok) return fail(nullptr, GBMUF_ERR_CUDA, "cudaSetDevice failed");

  gbmuf_ctx* ctx = new (std::nothrow) gbmuf_ctx();
  if (!ctx) return fail(nullptr, GBMUF_ERR_ALLOC, "out of host memory");
  ctx->cfg = *cfg; ctx->theta = theta; ctx->omega = omega; ctx->delta = delta; ctx->cand = cand;
  int v = 0;
  cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, cfg->device); ctx->num_sms = v;
  cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, cfg->device); ctx->max_smem = v;
  cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerMultiprocessor, cfg->device);
  ctx->smem_per_sm = v;
  gbmuf_status st = plan_launch(ctx, ctx->tuning, &ctx->launch);
  if (st == GBMUF_OK) st = build_tensor_maps(ctx, ctx->launch);
  if (st != GBMUF_OK) { g_create_error = ctx->err; delete ctx; return st; }
  e = ensure_kernel_attributes(cfg->device, ctx->max_smem);
  if (e != cudaSuccess) { delete ctx; return cuda_fail(nullptr, "raising the kernels' shared-memory limit", e); }
  e = cudaMalloc(&ctx->d_status, sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMemset(ctx->d_status, 0, sizeof(int32_t));
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->priv, cudaStreamNonBlocking);
  if (e != cudaSuccess) {
    st = e == cudaErrorMemoryAllocation ? fail(nullptr, GBMUF_ERR_ALLOC, "device status word")
                                        : cuda_fail(nullptr, "context set-up", e);
    cudaFree(ctx->d_status);
    delete ctx;
    return st;
  }
  *out = ctx;
  return GBMUF_OK;
}

gbmuf_status gbmuf_set_partition(gbmuf_ctx* ctx, int32_t m, const int64_t* offsets,
                                 const int32_t* periods) {
  if (!ctx) return GBMUF_ERR_INVALID_ARG;
  if (m < 1 || m > 65536 || !offsets) return fail(ctx, GBMUF_ERR_INVALID_ARG, "m must be in 1..65536 and offsets not NULL");
  if (offsets[0] != 0 || offsets[m] != ctx->cfg.N)
    return fail(ctx, GBMUF_ERR_INVALID_ARG, "offsets[0] must be 0 and offsets[m] must be N");
  for (int i = 0; i < m; ++i)
    if (offsets[i + 1] <= offsets[i]) return fail(ctx, GBMUF_ERR_INVALID_ARG, "offsets must be strictly increasing");
  if (periods)
    for (int i = 0; i < m; ++i)
      if (periods[i] < 1) return fail(ctx, GBMUF_ERR_INVALID_ARG, "periods must be >= 1");
  if ((long long)ctx->cfg.comp_base + m > 0x7fffffffLL)
    return fail(ctx, GBMUF_ERR_INVALID_ARG, "comp_base + m overflows");
  DeviceGuard guard(ctx->cfg.device);
  if (!guard.ok) return fail(ctx, GBMUF_ERR_CUDA, "cudaSetDevice failed");
  // the tables are about to be replaced: wait for the work this context has enqueued (and only
  // for that; other streams of the process keep running)
  cudaError_t e = ctx->work.wait();
  if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->priv);
  if (e != cudaSuccess) return cuda_fail(ctx, "waiting for the context's earlier work", e);
  ctx->partitioned = false;
  ctx->m = m;
  ctx->off.assign(offsets, offsets + m + 1);
  if (periods) ctx->periods.assign(periods, periods + m); else ctx->periods.assign(m, 1);
  const size_t nb = (size_t)ctx->cfg.K * m * (ctx->cfg.q > 0 ? ctx->cfg.q : 1) * sizeof(int32_t);
  if (m > ctx->cap_m || nb > ctx->cap_nbr_bytes) {
    // (tables that are already large enough are kept: freeing device memory stalls the device)
    free_tables(ctx);
    ctx->cap_m = 0; ctx->cap_nbr_bytes = 0;
    e = cudaMalloc(&ctx->d_off, (m + 1) * sizeof(int64_t));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->d_periods, m * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->d_mask, m);
    if (e == cudaSuccess) e = cudaMalloc(&ctx->d_prefix, (m + 1) * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->d_nbr, nb);
    if (e == cudaSuccess) e = cudaMalloc(&ctx->d_nbr_export, nb);
    if (e == cudaSuccess) { ctx->cap_m = m; ctx->cap_nbr_bytes = nb; }
  }
  // copies from the context's own vectors, complete when the private stream has been waited
  // for: nothing of the caller's is read later, and a round on any stream finds the tables
  if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->d_off, ctx->off.data(), (m + 1) * sizeof(int64_t), cudaMemcpyHostToDevice, ctx->priv);
  if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->d_periods, ctx->periods.data(), m * sizeof(int32_t), cudaMemcpyHostToDevice, ctx->priv);
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_mask, 1, m, ctx->priv);
  if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->priv);
  if (e != cudaSuccess) {
    free_tables(ctx);
    ctx->cap_m = 0; ctx->cap_nbr_bytes = 0;
    return e == cudaErrorMemoryAllocation ? fail(ctx, GBMUF_ERR_ALLOC, "partition tables") : cuda_fail(ctx, "partition upload", e);
  }
  ctx->partitioned = true;
  return GBMUF_OK;
}

gbmuf_status gbmuf_set_tuning(gbmuf_ctx* ctx, int32_t ncons, int32_t tile_elems, int32_t stages,
                              int32_t ring, int32_t flags) {
  if (!ctx) return GBMUF_ERR_INVALID_ARG;
  if (ncons < 0 || ncons > 992 || ncons % 32 != 0 || tile_elems < 0 || tile_elems > (1 << 16) ||
      stages < 0 || stages > kMaxThetaStages || ring < 0 || ring > kMaxRing || ring == 1 || flags < 0 || flags > 127 || ((flags & 4) && !(flags & 2)) || ((flags & 8) && (flags & (2 | 16))))
    return fail(ctx, GBMUF_ERR_INVALID_ARG, "tuning value out of range");
  Tuning t;
  t.ncons = ncons; t.T = tile_elems; t.stages = stages; t.ring = ring; t.flags = flags;
  Launch L;
  gbmuf_status st = plan_launch(ctx, t, &L);
  if (st != GBMUF_OK) return st;
  DeviceGuard guard(ctx->cfg.device);
  if (!guard.ok) return fail(ctx, GBMUF_ERR_CUDA, "cudaSetDevice failed");
  st = build_tensor_maps(ctx, L);
  if (st != GBMUF_OK) { build_tensor_maps(ctx, ctx->launch); return st; }
  ctx->tuning = t;
  ctx->launch = L;
  return GBMUF_OK;
}

gbmuf_status gbmuf_get_launch_info(gbmuf_ctx* ctx, int64_t* tiles, int32_t* grid, int32_t* block,
                                   int32_t* smem, int32_t* tile_elems, int32_t* stages) {
  if (!ctx) return GBMUF_ERR_INVALID_ARG;
  if (!ctx->partitioned) return fail(ctx, GBMUF_ERR_BAD_STATE, "set_partition has not been called");
  std::vector<uint8_t> all(ctx->m, 1);
  const long long total = host_total_tiles(ctx, 0, all.data(), ctx->launch.T);
  const long long cap = (long long)ctx->num_sms;
  if (tiles) *tiles = total;
  if (grid) *grid = (int32_t)(total < cap ? total : cap);
  if (block) *block = 32 + ctx->launch.ncons;
  if (smem) *smem = (int32_t)ctx->launch.smem;
  if (tile_elems) *tile_elems = ctx->launch.T;
  if (stages)
    *stages = ctx->launch.ma_ring > 0 ? 1000 + ctx->launch.ma_ring
              : ctx->launch.tmem_cols == 0 ? ctx->launch.stages
              : ctx->launch.pshift > 0 || ctx->launch.cell_rows < ctx->cfg.K ? -ctx->launch.cell_rows : 0;
  return GBMUF_OK;
}

gbmuf_status gbmuf_init(gbmuf_ctx* ctx, const void* theta0, void* stream) {
  if (!ctx) return GBMUF_ERR_INVALID_ARG;
  if (!theta0 || (uintptr_t)theta0 % 16 != 0)
    return fail(ctx, GBMUF_ERR_INVALID_ARG, "theta0 must be a 16-byte aligned device pointer");
  DeviceGuard guard(ctx->cfg.device);
  if (!guard.ok) return fail(ctx, GBMUF_ERR_CUDA, "cudaSetDevice failed");
  cudaStream_t st = (cudaStream_t)stream;
  const long long nchunks = (ctx->cfg.N + kInitChunk - 1) / kInitChunk;
  const int grid = (int)(nchunks < ctx->num_sms ? nchunks : ctx->num_sms);   // persistent CTAs
  const int esz = (int)theta_size(ctx);
  const size_t smem = 128 + (size_t)kInitChunk * 4 +
                      (size_t)kInitSlots * ((size_t)kInitChunk * esz + (esz != 4 ? (size_t)kInitChunk * 4 : 0));
  cudaError_t e;
  if (ctx->cfg.theta_dtype == GBMUF_F32) {
    init_stream_kernel<float><<<grid, 128, smem, st>>>((const float*)theta0, (float*)ctx->theta, ctx->omega,
                                                       ctx->delta, ctx->cfg.K, ctx->cfg.N, ctx->cfg.ld,
                                                       ctx->d_status);
  } else {
    init_stream_kernel<__nv_bfloat16><<<grid, 128, smem, st>>>((const __nv_bfloat16*)theta0,
                                                               (__nv_bfloat16*)ctx->theta, ctx->omega,
                                                               ctx->delta, ctx->cfg.K, ctx->cfg.N,
                                                               ctx->cfg.ld, ctx->d_status);
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, "launch of the init kernel", e);
  ctx->work.note(st);
  return GBMUF_OK;
}

gbmuf_status gbmuf_local_perturb(gbmuf_ctx* ctx, uint64_t step, float lr, float sigma,
                                 int32_t nsteps, void* stream) {
  if (!ctx) return GBMUF_ERR_INVALID_ARG;
  if (nsteps < 0 || step + (uint64_t)nsteps > 0xFFFFFFFFull || step > 0xFFFFFFFFull)
    return fail(ctx, GBMUF_ERR_INVALID_ARG, "nsteps must be >= 0 and step + nsteps <= 2^32 - 1");
  if (nsteps == 0) return GBMUF_OK;
  DeviceGuard guard(ctx->cfg.device);
  if (!guard.ok) return fail(ctx, GBMUF_ERR_CUDA, "cudaSetDevice failed");
  const uint32_t key0 = (uint32_t)ctx->cfg.seed;
  const uint32_t key1 = (uint32_t)(ctx->cfg.seed >> 32) ^ kTagPerturb;
  cudaStream_t st = (cudaStream_t)stream;
  const int K = ctx->cfg.K;
  if (ctx->cfg.theta_dtype == GBMUF_F32) {
    const dim3 grid(row_grid(ctx, (ctx->cfg.N + 3) / 4, K), K);
    perturb_kernel<float><<<grid, 256, 0, st>>>((float*)ctx->theta, K, ctx->cfg.N, ctx->cfg.ld, key0,
                                                key1, (uint32_t)step, nsteps, lr, sigma,
                                                ctx->cfg.elem_base);
  } else {
    const dim3 grid(row_grid(ctx, (ctx->cfg.N + 7) / 8, K), K);
    perturb_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((__nv_bfloat16*)ctx->theta, K, ctx->cfg.N,
                                                        ctx->cfg.ld, key0, key1, (uint32_t)step,
                                                        nsteps, lr, sigma, ctx->cfg.elem_base);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, "launch of the local-step kernel", e);
  ctx->work.note(st);
  return GBMUF_OK;
}

gbmuf_status gbmuf_local_adagrad(gbmuf_ctx* ctx, const float* grad, float* accum, float lr,
                                 float eps, float clip_norm, const uint8_t* clip_mask,
                                 void* stream) {
  if (!ctx) return GBMUF_ERR_INVALID_ARG;
  if (!grad || !accum || (((uintptr_t)grad | (uintptr_t)accum) % 128) != 0)
    return fail(ctx, GBMUF_ERR_INVALID_ARG, "grad and accum must be 128-byte aligned device pointers");
  if (!(lr == lr) || !(eps == eps) || !(clip_norm == clip_norm))
    return fail(ctx, GBMUF_ERR_INVALID_ARG, "lr, eps and clip_norm must not be NaN");
  ClipRanges R;
  R.n = 0;
  const bool clip = clip_mask != nullptr && clip_norm > 0.0f;
  if (clip) {
    if (!ctx->partitioned) return fail(ctx, GBMUF_ERR_BAD_STATE, "a clip mask needs set_partition first");
    for (int i = 0; i < ctx->m; ++i) {
      if (!clip_mask[i]) continue;
      if (R.n > 0 && R.end[R.n - 1] == ctx->off[i]) { R.end[R.n - 1] = ctx->off[i + 1]; continue; }
      if (R.n == kMaxClipRanges)
        return fail(ctx, GBMUF_ERR_UNSUPPORTED, "more than 16 separate runs of clipped components");
      R.begin[R.n] = ctx->off[i];
      R.end[R.n] = ctx->off[i + 1];
      ++R.n;
    }
  }
  DeviceGuard guard(ctx->cfg.device);
  if (!guard.ok) return fail(ctx, GBMUF_ERR_CUDA, "cudaSetDevice failed");
  cudaStream_t st = (cudaStream_t)stream;
  const int K = ctx->cfg.K;
  cudaError_t e;
  const float* scale = nullptr;
  if (clip && R.n > 0) {
    if (!ctx->d_norm_partial) {
      e = cudaMalloc(&ctx->d_norm_partial, (size_t)K * kNormBlocks * sizeof(double));
      if (e == cudaSuccess) e = cudaMalloc(&ctx->d_clip_scale, (size_t)K * sizeof(float));
      if (e != cudaSuccess) return fail(ctx, GBMUF_ERR_ALLOC, "scratch of the gradient-norm reduction");
    }
    sumsq_partial_kernel<<<dim3(kNormBlocks, K), 256, 0, st>>>(grad, ctx->cfg.ld, R, ctx->d_norm_partial);
    clip_scale_kernel<<<(K + 127) / 128, 128, 0, st>>>(ctx->d_norm_partial, K, kNormBlocks, clip_norm,
                                                       ctx->d_clip_scale);
    scale = ctx->d_clip_scale;
  }
  // streaming update: chunks of 4096 elements (16 KB of gradient and accumulator each), 4 slots
  AdagradParams A;
  const int esz = (int)theta_size(ctx);
  A.theta = ctx->theta; A.grad = grad; A.accum = accum; A.scale = scale; A.status = ctx->d_status;
  A.N = ctx->cfg.N; A.ld = ctx->cfg.ld; A.K = K; A.T = 4096; A.ring = 4; A.groups = 2;
  A.ring_off = 512; A.slot_stride = (uint32_t)((8 + esz) * A.T);
  A.lr = lr; A.eps = eps; A.R = R;
  const long long cpr = (ctx->cfg.N + A.T - 1) / A.T;
  if (cpr * K > 0x7fffffffLL) return fail(ctx, GBMUF_ERR_UNSUPPORTED, "more than 2^31 - 1 chunks");
  A.chunks_per_row = (int)cpr;
  const uint32_t smem_bytes = A.ring_off + (uint32_t)A.ring * A.slot_stride;
  const long long chunks = cpr * K;
  const int grid = (int)(chunks < ctx->num_sms ? chunks : ctx->num_sms);
  if (ctx->cfg.theta_dtype == GBMUF_F32) {
    adagrad_stream_kernel<float><<<grid, 544, smem_bytes, st>>>(A);
  } else {
    adagrad_stream_kernel<__nv_bfloat16><<<grid, 544, smem_bytes, st>>>(A);
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, "launch of the Adagrad local-step kernels", e);
  ctx->work.note(st);
  return GBMUF_OK;
}

gbmuf_status gbmuf_sync_round(gbmuf_ctx* ctx, uint64_t round, const uint8_t* comp_mask,
                              void* stream) {
  if (!ctx) return GBMUF_ERR_INVALID_ARG;
  if (!ctx->partitioned) return fail(ctx, GBMUF_ERR_BAD_STATE, "set_partition has not been called");
  DeviceGuard guard(ctx->cfg.device);
  if (!guard.ok) return fail(ctx, GBMUF_ERR_CUDA, "cudaSetDevice failed");
  const Launch& L = ctx->launch;
  const long long total = host_total_tiles(ctx, round, comp_mask, L.T);
  if (total == 0) return GBMUF_OK;
  if (total > 0x3fffffffLL) return fail(ctx, GBMUF_ERR_UNSUPPORTED, "more than 2^30 - 1 tiles");
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e;
  if (comp_mask) {
    // A mask is host data that must reach the device.  It cannot be recorded into a stream
    // capture (a replay would upload whatever the staging copy holds by then); rounds selected
    // by periods can.
    if (is_capturing(st))
      return fail(ctx, GBMUF_ERR_BAD_STATE,
                  "a component mask cannot be recorded into a stream capture; select components by periods there");
    // The caller's array may be page-locked, and a copy from page-locked memory really is
    // asynchronous.  The upload therefore starts from the library's own pageable copy: the
    // runtime moves pageable bytes into its staging area before cudaMemcpyAsync returns, so
    // neither the caller's array nor this copy is read after the call.
    ctx->mask_stage.assign(comp_mask, comp_mask + ctx->m);
    e = cudaMemcpyAsync(ctx->d_mask, ctx->mask_stage.data(), ctx->m, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(ctx, "upload of the component mask", e);
  }
  SetupParams S;
  fill_setup(ctx, round, comp_mask != nullptr, true, ctx->d_nbr, &S);
  e = launch_setup(S, st);
  if (e != cudaSuccess) return cuda_fail(ctx, "launch of the round set-up kernel", e);

  const gbmuf_status rc = launch_round(ctx, ctx->cfg, L, ctx->theta, ctx->omega, ctx->delta, ctx->cfg.ld, ctx->m,
                                       ctx->d_off, ctx->d_prefix, ctx->d_nbr, ctx->d_status, total, st);
  ctx->work.note(st);
  return rc;
}

gbmuf_status gbmuf_get_neighbors(gbmuf_ctx* ctx, uint64_t round, int32_t* out) {
  if (!ctx) return GBMUF_ERR_INVALID_ARG;
  if (!out) return fail(ctx, GBMUF_ERR_INVALID_ARG, "out must not be NULL");
  if (!ctx->partitioned) return fail(ctx, GBMUF_ERR_BAD_STATE, "set_partition has not been called");
  const int K = ctx->cfg.K, m = ctx->m, q = ctx->cfg.q;
  if (q == 0) return GBMUF_OK;
  DeviceGuard guard(ctx->cfg.device);
  if (!guard.ok) return fail(ctx, GBMUF_ERR_CUDA, "cudaSetDevice failed");
  SetupParams S;
  fill_setup(ctx, round, false, false, ctx->d_nbr_export, &S);
  const long long items = (long long)K * m;
  round_setup_kernel<<<(int)((items + 255) / 256), 256, 0, ctx->priv>>>(S);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, "launch of the round set-up kernel", e);
  std::vector<int32_t> tmp((size_t)K * m * q);
  e = cudaMemcpyAsync(tmp.data(), ctx->d_nbr_export, tmp.size() * sizeof(int32_t),
                      cudaMemcpyDeviceToHost, ctx->priv);
  if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->priv);
  if (e != cudaSuccess) return cuda_fail(ctx, "read-back of the neighbour table", e);
  for (int i = 0; i < m; ++i)          // device layout [m][K][q] -> caller's [K][m][q]
    for (int k = 0; k < K; ++k)
      for (int j = 0; j < q; ++j)
        out[((size_t)k * m + i) * q + j] = tmp[((size_t)i * K + k) * q + j];
  return GBMUF_OK;
}

gbmuf_status gbmuf_final_average(gbmuf_ctx* ctx, void* out, void* stream) {
  if (!ctx) return GBMUF_ERR_INVALID_ARG;
  if (!out || (uintptr_t)out % 16 != 0)
    return fail(ctx, GBMUF_ERR_INVALID_ARG, "out must be a 16-byte aligned device pointer");
  DeviceGuard guard(ctx->cfg.device);
  if (!guard.ok) return fail(ctx, GBMUF_ERR_CUDA, "cudaSetDevice failed");
  const int grid = elementwise_grid(ctx, (ctx->cfg.N + 3) / 4);
  cudaStream_t st = (cudaStream_t)stream;
  if (ctx->cfg.theta_dtype == GBMUF_F32)
    final_average_kernel<float><<<grid, 256, 0, st>>>((const float*)ctx->theta, (float*)out,
                                                      ctx->cfg.K, ctx->cfg.N, ctx->cfg.ld);
  else
    final_average_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)ctx->theta,
                                                              (__nv_bfloat16*)out, ctx->cfg.K,
                                                              ctx->cfg.N, ctx->cfg.ld);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, "launch of the final-average kernel", e);
  ctx->work.note(st);
  return GBMUF_OK;
}

gbmuf_status gbmuf_selftest_wait_timeout(gbmuf_ctx* ctx, void* stream, double* seconds_out) {
  if (!ctx) return GBMUF_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->cfg.device);
  if (!guard.ok) return fail(ctx, GBMUF_ERR_CUDA, "cudaSetDevice failed");
  cudaStream_t st = (cudaStream_t)stream;
  int32_t* d_ret = nullptr;
  cudaEvent_t a = nullptr, b = nullptr;
  cudaError_t e = cudaMalloc(&d_ret, sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMemsetAsync(d_ret, 0, sizeof(int32_t), st);
  if (e == cudaSuccess) e = cudaEventCreate(&a);
  if (e == cudaSuccess) e = cudaEventCreate(&b);
  if (e == cudaSuccess) e = cudaEventRecord(a, st);
  if (e == cudaSuccess) {
    wait_timeout_selftest_kernel<<<1, 32, 0, st>>>(ctx->d_status, d_ret);
    e = cudaGetLastError();
  }
  if (e == cudaSuccess) e = cudaEventRecord(b, st);
  int32_t ret = 0;
  if (e == cudaSuccess) e = cudaMemcpyAsync(&ret, d_ret, sizeof(ret), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  float ms = 0.f;
  if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, a, b);
  if (a) cudaEventDestroy(a);
  if (b) cudaEventDestroy(b);
  cudaFree(d_ret);
  if (e != cudaSuccess) return cuda_fail(ctx, "wait-timeout self-test", e);
  if (seconds_out) *seconds_out = ms / 1e3;
  if (ret != 2) return fail(ctx, GBMUF_ERR_BAD_STATE, "the self-test wait did not expire as it should");
  return GBMUF_OK;
}

gbmuf_status gbmuf_selftest_divide(gbmuf_ctx* ctx, int32_t divisor, void* stream,
                                   uint64_t* mismatches_out, uint32_t* first_bad_out) {
  if (!ctx) return GBMUF_ERR_INVALID_ARG;
  if (!mismatches_out) return fail(ctx, GBMUF_ERR_INVALID_ARG, "mismatches_out must not be NULL");
  if (divisor < 2 || divisor > 256)
    return fail(ctx, GBMUF_ERR_INVALID_ARG, "divisor must be in 2..256");
  DeviceGuard guard(ctx->cfg.device);
  if (!guard.ok) return fail(ctx, GBMUF_ERR_CUDA, "cudaSetDevice failed");
  cudaStream_t st = (cudaStream_t)stream;
  unsigned long long* d_buf = nullptr;             // [0] mismatches, [1] first bad pattern (low word)
  cudaError_t e = cudaMalloc(&d_buf, 2 * sizeof(unsigned long long));
  const unsigned long long init[2] = {0ull, 0xFFFFFFFFull};
  if (e == cudaSuccess) e = cudaMemcpyAsync(d_buf, init, sizeof(init), cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) {
    const float b = (float)divisor;
    divide_selftest_kernel<<<ctx->num_sms * 8, 256, 0, st>>>(b, 1.0f / b, d_buf,
                                                             reinterpret_cast<unsigned int*>(d_buf + 1));
    e = cudaGetLastError();
  }
  unsigned long long res[2] = {0ull, 0ull};
  if (e == cudaSuccess) e = cudaMemcpyAsync(res, d_buf, sizeof(res), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  cudaFree(d_buf);
  if (e != cudaSuccess) return cuda_fail(ctx, "divide self-test", e);
  *mismatches_out = (uint64_t)res[0];
  if (first_bad_out) *first_bad_out = (uint32_t)(res[1] & 0xFFFFFFFFull);
  return GBMUF_OK;
}

gbmuf_status gbmuf_device_status(gbmuf_ctx* ctx, void* stream, int32_t* out) {
  if (!ctx) return GBMUF_ERR_INVALID_ARG;
  if (!out) return fail(ctx, GBMUF_ERR_INVALID_ARG, "out must not be NULL");
  DeviceGuard guard(ctx->cfg.device);
  if (!guard.ok) return fail(ctx, GBMUF_ERR_CUDA, "cudaSetDevice failed");
  cudaStream_t st = (cudaStream_t)stream;
  int32_t v = 0;
  cudaError_t e = cudaMemcpyAsync(&v, ctx->d_status, sizeof(v), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_status, 0, sizeof(v), st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return cuda_fail(ctx, "read of the device status word", e);
  *out = v;
  return GBMUF_OK;
}

const char* gbmuf_last_error(const gbmuf_ctx* ctx) {
  return ctx ? ctx->err.c_str() : g_create_error.c_str();
}

gbmuf_status gbmuf_destroy(gbmuf_ctx* ctx) {
  if (!ctx) return GBMUF_OK;
  gbmuf_status rc = GBMUF_OK;
  {
    DeviceGuard guard(ctx->cfg.device);
    if (guard.ok) {
      // wait for this context's own work, not for the whole device
      if (ctx->work.wait() != cudaSuccess) rc = GBMUF_ERR_CUDA;
      if (ctx->priv && cudaStreamSynchronize(ctx->priv) != cudaSuccess) rc = GBMUF_ERR_CUDA;
      ctx->work.release();
      free_tables(ctx);
      cudaFree(ctx->d_status);
      cudaFree(ctx->d_norm_partial);
      cudaFree(ctx->d_clip_scale);
      if (ctx->priv) cudaStreamDestroy(ctx->priv);
    } else {
      rc = GBMUF_ERR_CUDA;
    }
  }
  delete ctx;
  return rc;
}


// -------------------------------------------------------------------------------------------------
// gbmuf_sync_round_noalloc: one round with every library-side table in a fixed device array.
// -------------------------------------------------------------------------------------------------
namespace {

constexpr int kNoAllocMaxM = 1024;            // components
constexpr int kNoAllocMaxDraws = 65536;       // K * m * q neighbour entries
constexpr size_t kNaStatusOff = 0;                                          // int32 status word
constexpr size_t kNaOffsetsOff = 256;                                       // int64 [m+1]
constexpr size_t kNaPrefixOff = kNaOffsetsOff + 8448;                       // int32 [m+1]
constexpr size_t kNaMaskOff = kNaPrefixOff + 4352;                          // uint8 [m]
constexpr size_t kNaNbrOff = kNaMaskOff + 1024;                             // int32 [m][K][q]
constexpr size_t kNoAllocBytes = kNaNbrOff + (size_t)kNoAllocMaxDraws * 4;  // 276,224 bytes

// The scratch itself.  Part of the loaded module: every GPU that loads this library holds these
// 270 KB until the process exits.  In HOST code this name is only a handle for
// cudaGetSymbolAddress; it is not a device address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

constexpr int kNoAllocMaxDevices = 64;
unsigned char* g_noalloc_ptr[kNoAllocMaxDevices] = {};   // device address of the array, per GPU

// Host-side staging of the two tables a call uploads, in ordinary (pageable) static memory: the
// caller's arrays may be page-locked, from which an asynchronous copy reads later, whereas the
// runtime has moved pageable bytes into its own staging area by the time cudaMemcpyAsync
// returns.  The mutex covers filling and handing over; it does not make overlapping calls
// safe on the GPU (they share the device array).
std::mutex g_noalloc_mutex;
int64_t g_noalloc_off_stage[kNoAllocMaxM + 1];
uint8_t g_noalloc_flag_stage[kNoAllocMaxM];

}  // namespace

gbmuf_status gbmuf_sync_round_noalloc(const gbmuf_config* cfg, void* theta, float* omega,
                                      float* delta, int32_t m, const int64_t* offsets,
                                      const uint8_t* comp_mask, uint64_t round, void* stream,
                                      int32_t* device_status_out) {
  if (!cfg) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "cfg must not be NULL");
  if (cfg->K < 1 || cfg->K > 256 || cfg->N < 1 || cfg->ld < cfg->N || cfg->ld % 32 != 0 ||
      cfg->ld > 0x7fffffffLL || cfg->p < 0 || cfg->q < 0 || cfg->comp_base < 0 ||
      (cfg->mode != GBMUF_MODE_BMUF && cfg->mode != GBMUF_MODE_MA) ||
      (cfg->theta_dtype != GBMUF_F32 && cfg->theta_dtype != GBMUF_BF16) ||
      !(cfg->eta == cfg->eta) || !(cfg->zeta == cfg->zeta))
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "configuration out of range (see gbmuf_create)");
  const int cand = host_candidates(cfg->K, cfg->p);
  if (cfg->q > cand || cand > kMaxCand)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "q exceeds the ring neighbours min(2p, K-1), or more than 64 of them");
  if (!theta || !omega || !delta || (((uintptr_t)theta | (uintptr_t)omega | (uintptr_t)delta) % 128) != 0)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "theta, omega and delta must be 128-byte aligned device pointers");
  if (m < 1 || !offsets) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "m must be >= 1 and offsets not NULL");
  if (m > kNoAllocMaxM)
    return fail(nullptr, GBMUF_ERR_UNSUPPORTED,
                "gbmuf_sync_round_noalloc handles at most 1024 components; use a context (gbmuf_create) for more");
  if ((long long)cfg->K * m * cfg->q > kNoAllocMaxDraws)
    return fail(nullptr, GBMUF_ERR_UNSUPPORTED,
                "gbmuf_sync_round_noalloc handles at most 65536 neighbour draws (K * m * q) per round; "
                "use a context (gbmuf_create) for more");
  if (offsets[0] != 0 || offsets[m] != cfg->N)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "offsets[0] must be 0 and offsets[m] must be N");
  for (int i = 0; i < m; ++i)
    if (offsets[i + 1] <= offsets[i]) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "offsets must be strictly increasing");
  if (cfg->device < 0 || cfg->device >= kNoAllocMaxDevices)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "device ordinal out of range");

  DeviceGuard guard(cfg->device);
  if (!guard.ok) return fail(nullptr, GBMUF_ERR_CUDA, "cudaSetDevice failed");
  cudaStream_t cs = (cudaStream_t)stream;
  // The call uploads host tables, so it cannot be part of a stream capture: the recorded copies
  // would read this library's staging arrays again at every replay, with whatever a later call
  // left there.  Refused before anything is enqueued.
  if (is_capturing(cs))
    return fail(nullptr, GBMUF_ERR_BAD_STATE,
                "gbmuf_sync_round_noalloc uploads host tables and cannot be recorded into a stream capture");
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  cudaError_t e;
  int v = 0;
  if (!g_noalloc_ptr[cfg->device]) {
    // once per device, with that device current: ask the runtime where the array lives there,
    // and raise the kernels' shared-memory limit
    unsigned char* ptr = nullptr;
    e = cudaGetSymbolAddress((void**)&ptr, g_noalloc_scratch);
    if (e != cudaSuccess || !ptr) return cuda_fail(nullptr, "cudaGetSymbolAddress of the fixed scratch array", e);
    cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, cfg->device);
    e = ensure_kernel_attributes(cfg->device, v);
    if (e != cudaSuccess) return cuda_fail(nullptr, "raising the kernels' shared-memory limit", e);
    g_noalloc_ptr[cfg->device] = ptr;
  }
  unsigned char* scratch = g_noalloc_ptr[cfg->device];

  // a context on the stack: it owns nothing, it only carries the description to the helpers
  gbmuf_ctx tmp;
  tmp.cfg = *cfg; tmp.theta = theta; tmp.omega = omega; tmp.delta = delta; tmp.m = m; tmp.cand = cand;
  cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, cfg->device); tmp.num_sms = v;
  cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, cfg->device); tmp.max_smem = v;
  cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerMultiprocessor, cfg->device); tmp.smem_per_sm = v;
  gbmuf_status st = plan_launch(&tmp, tmp.tuning, &tmp.launch);
  if (st == GBMUF_OK) st = build_tensor_maps(&tmp, tmp.launch);
  if (st != GBMUF_OK) { g_create_error = tmp.err; return st; }
  const Launch& L = tmp.launch;

  uint8_t* const flags = g_noalloc_flag_stage;
  long long total = 0;
  for (int i = 0; i < m; ++i) {
    flags[i] = comp_mask ? (comp_mask[i] != 0) : 1;
    g_noalloc_off_stage[i] = offsets[i];
    if (!flags[i]) continue;
    const int64_t start = offsets[i] & ~(int64_t)(kAlign - 1);
    total += (offsets[i + 1] - start + L.T - 1) / L.T;
  }
  g_noalloc_off_stage[m] = offsets[m];
  if (total > 0x3fffffffLL) return fail(nullptr, GBMUF_ERR_UNSUPPORTED, "more than 2^30 - 1 tiles");
  int32_t* d_status = reinterpret_cast<int32_t*>(scratch + kNaStatusOff);
  // the array keeps whatever the previous call left: the status word must start at zero, the
  // other tables are rewritten in full below for the sizes of this call
  e = cudaMemsetAsync(d_status, 0, sizeof(int32_t), cs);
  if (e == cudaSuccess && total > 0)
    e = cudaMemcpyAsync(scratch + kNaOffsetsOff, g_noalloc_off_stage, (size_t)(m + 1) * sizeof(int64_t), cudaMemcpyHostToDevice, cs);
  if (e == cudaSuccess && total > 0)
    e = cudaMemcpyAsync(scratch + kNaMaskOff, flags, (size_t)m, cudaMemcpyHostToDevice, cs);
  if (e != cudaSuccess) return cuda_fail(nullptr, "upload of offsets and mask into the fixed scratch array", e);
  if (total > 0) {
    SetupParams S;
    S.K = cfg->K; S.m = m; S.p = cfg->p; S.q = cfg->q; S.comp_base = cfg->comp_base; S.T = L.T;
    S.use_mask = 1; S.plan = 1; S.seed = cfg->seed; S.round = round;
    S.off = reinterpret_cast<const int64_t*>(scratch + kNaOffsetsOff);
    S.periods = nullptr;
    S.mask = scratch + kNaMaskOff;
    S.nbr = reinterpret_cast<int32_t*>(scratch + kNaNbrOff);
    S.tile_prefix = reinterpret_cast<int32_t*>(scratch + kNaPrefixOff);
    e = launch_setup(S, cs);
    if (e != cudaSuccess) return cuda_fail(nullptr, "launch of the round set-up kernel", e);

    st = launch_round(&tmp, *cfg, L, theta, omega, delta, cfg->ld, m, S.off, S.tile_prefix, S.nbr, d_status,
                      total, cs);
    if (st != GBMUF_OK) { g_create_error = tmp.err; return st; }
  }
  if (device_status_out) {
    int32_t word = 0;
    e = cudaMemcpyAsync(&word, d_status, sizeof(word), cudaMemcpyDeviceToHost, cs);
    if (e == cudaSuccess) e = cudaStreamSynchronize(cs);
    if (e != cudaSuccess) return cuda_fail(nullptr, "read of the device status word", e);
    *device_status_out = word;
  }
  return GBMUF_OK;
}


// -------------------------------------------------------------------------------------------------
// Replicas that live in HOST memory: gbmuf_host_* and the one-call form gbmuf_sync_round_host.
// -------------------------------------------------------------------------------------------------
}  // extern "C"

namespace {

struct HostChunk {             // one column chunk [c0, c1) of the model
  long long c0, c1;
  int first, mc;               // first component that reaches into it, and how many do
  size_t off_at, mask_at;      // where its local offsets (mc + 1) / flags (mc) start in the arenas
};

struct HostSet {               // one of the buffer sets the chunks rotate through
  gbmuf_ctx ctx;               // describes the device chunk buffers to the launch helpers
  unsigned char* tables = nullptr;   // prefix | nbr | mask | status
  cudaStream_t stream = nullptr;
};

constexpr int kHostSets = 3;

}  // namespace

struct gbmuf_host {
  gbmuf_config cfg;
  int m = 0, esz = 4, nsets = 0;
  long long chunk_cols = 0;
  int row_copies = 0;          // one cudaMemcpyAsync per row instead of one 2-D copy per array
  std::vector<int64_t> off;
  std::vector<HostChunk> chunks;
  HostSet sets[kHostSets];
  int64_t* d_chunk_off = nullptr;   // device: every chunk's local offsets, back to back
  uint8_t* h_flags = nullptr;       // page-locked: every chunk's participation flags of this round
  size_t t_nbr = 0, t_mask = 0, t_status = 0, t_bytes = 0;
};

namespace {

void free_host_handle(gbmuf_host* h) {
  for (int i = 0; i < kHostSets; ++i) {
    HostSet& s = h->sets[i];
    cudaFree(s.ctx.theta); cudaFree(s.ctx.omega); cudaFree(s.ctx.delta); cudaFree(s.tables);
    if (s.stream) cudaStreamDestroy(s.stream);
  }
  cudaFree(h->d_chunk_off);
  if (h->h_flags) cudaFreeHost(h->h_flags);
  delete h;
}

// rows [0, K) x columns of one array between host (row stride ld_h) and a chunk buffer (row
// stride ld_d), as one 2-D copy or as K row copies
cudaError_t copy_rows(void* dst, size_t dpitch, const void* src, size_t spitch, size_t width, int K,
                      cudaMemcpyKind kind, cudaStream_t st, bool row_copies) {
  if (!row_copies) return cudaMemcpy2DAsync(dst, dpitch, src, spitch, width, K, kind, st);
  for (int k = 0; k < K; ++k) {
    const cudaError_t e = cudaMemcpyAsync((char*)dst + (size_t)k * dpitch, (const char*)src + (size_t)k * spitch,
                                          width, kind, st);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace

extern "C" {

gbmuf_status gbmuf_host_create(const gbmuf_config* cfg, int32_t m, const int64_t* offsets,
                               int64_t chunk_cols, int32_t flags, gbmuf_host** out) {
  if (!cfg || !out) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "cfg and out must not be NULL");
  if (cfg->K < 1 || cfg->K > 256 || cfg->N < 1 || cfg->ld < cfg->N || cfg->p < 0 || cfg->q < 0 ||
      cfg->comp_base < 0 || (cfg->mode != GBMUF_MODE_BMUF && cfg->mode != GBMUF_MODE_MA) ||
      (cfg->theta_dtype != GBMUF_F32 && cfg->theta_dtype != GBMUF_BF16) ||
      !(cfg->eta == cfg->eta) || !(cfg->zeta == cfg->zeta) || cfg->device < 0)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "configuration out of range (see gbmuf_create)");
  const int cand = host_candidates(cfg->K, cfg->p);
  if (cfg->q > cand || cand > kMaxCand)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "q exceeds the ring neighbours min(2p, K-1), or more than 64 of them");
  if (m < 1 || m > 65536 || !offsets) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "m must be in 1..65536 and offsets not NULL");
  if (offsets[0] != 0 || offsets[m] != cfg->N)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "offsets[0] must be 0 and offsets[m] must be N");
  for (int i = 0; i < m; ++i)
    if (offsets[i + 1] <= offsets[i]) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "offsets must be strictly increasing");
  if (chunk_cols < 0 || (chunk_cols > 0 && chunk_cols % 32 != 0) || chunk_cols > (1LL << 30))
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "chunk_cols must be 0 or a multiple of 32 up to 2^30");
  if (flags < 0 || flags > 1) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "unknown flags");
  if (chunk_cols == 0) chunk_cols = 1 << 21;
  const long long N = cfg->N;
  if (chunk_cols > (N + 31) / 32 * 32) chunk_cols = (N + 31) / 32 * 32;
  const long long nchunks = (N + chunk_cols - 1) / chunk_cols;
  const int K = cfg->K, q = cfg->q;

  int ndev = 0;
  cudaError_t e = cudaGetDeviceCount(&ndev);
  if (e != cudaSuccess) return cuda_fail(nullptr, "cudaGetDeviceCount", e);
  if (cfg->device >= ndev) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "no such CUDA device");
  DeviceGuard guard(cfg->device);
  if (!guard.ok) return fail(nullptr, GBMUF_ERR_CUDA, "cudaSetDevice failed");

  gbmuf_host* h = new (std::nothrow) gbmuf_host();
  if (!h) return fail(nullptr, GBMUF_ERR_ALLOC, "out of host memory");
  h->cfg = *cfg; h->m = m; h->chunk_cols = chunk_cols; h->row_copies = flags & 1;
  h->esz = cfg->theta_dtype == GBMUF_F32 ? 4 : 2;
  h->off.assign(offsets, offsets + m + 1);
  h->nsets = nchunks < kHostSets ? (int)nchunks : kHostSets;

  // the chunks and their local partitions: fixed for the life of the handle
  std::vector<int64_t> all_off;
  size_t nflags = 0;
  int first = 0, mc_max = 1;
  for (long long ci = 0; ci < nchunks; ++ci) {
    HostChunk c;
    c.c0 = ci * chunk_cols;
    c.c1 = c.c0 + chunk_cols < N ? c.c0 + chunk_cols : N;
    while (offsets[first + 1] <= c.c0) ++first;
    c.first = first; c.off_at = all_off.size(); c.mask_at = nflags;
    all_off.push_back(0);
    int i = first;
    while (true) {
      all_off.push_back(offsets[i + 1] < c.c1 ? offsets[i + 1] - c.c0 : c.c1 - c.c0);
      if (offsets[i + 1] >= c.c1) break;
      ++i;
    }
    c.mc = i - first + 1;
    nflags += (size_t)c.mc;
    if (c.mc > mc_max) mc_max = c.mc;
    h->chunks.push_back(c);
  }
  // table block of one set: prefix int32 [mc_max + 1] | nbr int32 [K * mc_max * q] | mask | status
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  h->t_nbr = up((size_t)(mc_max + 1) * 4);
  h->t_mask = h->t_nbr + up((size_t)K * mc_max * (q > 0 ? q : 1) * 4);
  h->t_status = h->t_mask + up((size_t)mc_max);
  h->t_bytes = h->t_status + 256;

  gbmuf_status st = GBMUF_OK;
  for (int i = 0; i < h->nsets && st == GBMUF_OK; ++i) {
    gbmuf_ctx& c = h->sets[i].ctx;
    c.cfg = *cfg; c.cfg.N = chunk_cols; c.cfg.ld = chunk_cols; c.m = mc_max; c.cand = cand;
    c.theta = nullptr; c.omega = nullptr; c.delta = nullptr;
    int v = 0;
    cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, cfg->device); c.num_sms = v;
    cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, cfg->device); c.max_smem = v;
    cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerMultiprocessor, cfg->device); c.smem_per_sm = v;
    e = cudaMalloc(&c.theta, (size_t)K * chunk_cols * h->esz);
    if (e == cudaSuccess && cfg->mode == GBMUF_MODE_BMUF) e = cudaMalloc(&c.omega, (size_t)K * chunk_cols * 4);
    if (e == cudaSuccess && cfg->mode == GBMUF_MODE_BMUF) e = cudaMalloc(&c.delta, (size_t)K * chunk_cols * 4);
    if (e == cudaSuccess) e = cudaMalloc(&h->sets[i].tables, h->t_bytes);
    if (e == cudaSuccess) e = cudaMemset(h->sets[i].tables + h->t_status, 0, 256);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&h->sets[i].stream, cudaStreamNonBlocking);
    if (e == cudaSuccess && i == 0) e = ensure_kernel_attributes(cfg->device, c.max_smem);
    if (e != cudaSuccess) {
      st = e == cudaErrorMemoryAllocation ? fail(nullptr, GBMUF_ERR_ALLOC, "device chunk buffers")
                                          : cuda_fail(nullptr, "set-up of the chunk buffers", e);
      break;
    }
    st = plan_launch(&c, c.tuning, &c.launch);
    if (st == GBMUF_OK) st = build_tensor_maps(&c, c.launch);
    if (st != GBMUF_OK) g_create_error = c.err;
  }
  if (st == GBMUF_OK) {
    e = cudaMalloc(&h->d_chunk_off, all_off.size() * sizeof(int64_t));
    if (e == cudaSuccess)
      e = cudaMemcpyAsync(h->d_chunk_off, all_off.data(), all_off.size() * sizeof(int64_t), cudaMemcpyHostToDevice,
                          h->sets[0].stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->sets[0].stream);   // the table is in place
    if (e == cudaSuccess) e = cudaHostAlloc((void**)&h->h_flags, nflags, cudaHostAllocDefault);
    if (e != cudaSuccess)
      st = e == cudaErrorMemoryAllocation ? fail(nullptr, GBMUF_ERR_ALLOC, "chunk tables") : cuda_fail(nullptr, "chunk tables", e);
  }
  if (st != GBMUF_OK) { free_host_handle(h); return st; }
  *out = h;
  return GBMUF_OK;
}

gbmuf_status gbmuf_host_sync_round(gbmuf_host* h, void* theta, float* omega, float* delta,
                                   const uint8_t* comp_mask, uint64_t round) {
  if (!h) return GBMUF_ERR_INVALID_ARG;
  const gbmuf_config& cfg = h->cfg;
  const bool bmuf = cfg.mode == GBMUF_MODE_BMUF;
  if (!theta || (bmuf && (!omega || !delta)))
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "theta, omega and delta must not be NULL");
  DeviceGuard guard(cfg.device);
  if (!guard.ok) return fail(nullptr, GBMUF_ERR_CUDA, "cudaSetDevice failed");
  const int K = cfg.K, q = cfg.q, esz = h->esz;
  const long long chunk_cols = h->chunk_cols;
  const bool rc = h->row_copies != 0;
  gbmuf_status st = GBMUF_OK;
  cudaError_t e = cudaSuccess;
  for (size_t ci = 0; ci < h->chunks.size() && st == GBMUF_OK; ++ci) {
    const HostChunk& c = h->chunks[ci];
    HostSet& hs = h->sets[ci % (size_t)h->nsets];
    const int T = hs.ctx.launch.T;
    const int64_t* lo = h->off.data();
    uint8_t* fl = h->h_flags + c.mask_at;           // this chunk's own bytes: nothing reuses them
    long long total = 0;                            // before the call returns
    for (int j = 0; j < c.mc; ++j) {
      const int i = c.first + j;
      const long long b = lo[i] > c.c0 ? lo[i] - c.c0 : 0;
      const long long en = lo[i + 1] < c.c1 ? lo[i + 1] - c.c0 : c.c1 - c.c0;
      fl[j] = comp_mask ? (comp_mask[i] != 0) : 1;
      if (fl[j]) total += (en - (b & ~(long long)(kAlign - 1)) + T - 1) / T;
    }
    if (total == 0) continue;                       // nothing in this chunk takes part: leave it alone
    cudaStream_t cs = hs.stream;
    const long long c0 = c.c0;
    const size_t w_th = (size_t)(c.c1 - c0) * esz, w_f = (size_t)(c.c1 - c0) * 4;
    e = copy_rows(hs.ctx.theta, (size_t)chunk_cols * esz, (const char*)theta + (size_t)c0 * esz,
                  (size_t)cfg.ld * esz, w_th, K, cudaMemcpyHostToDevice, cs, rc);
    if (e == cudaSuccess && bmuf) {
      e = copy_rows(hs.ctx.omega, (size_t)chunk_cols * 4, omega + c0, (size_t)cfg.ld * 4, w_f, K,
                    cudaMemcpyHostToDevice, cs, rc);
      if (e == cudaSuccess)
        e = copy_rows(hs.ctx.delta, (size_t)chunk_cols * 4, delta + c0, (size_t)cfg.ld * 4, w_f, K,
                      cudaMemcpyHostToDevice, cs, rc);
    }
    if (e == cudaSuccess)
      e = cudaMemcpyAsync(hs.tables + h->t_mask, fl, (size_t)c.mc, cudaMemcpyHostToDevice, cs);
    if (e != cudaSuccess) { st = cuda_fail(nullptr, "host-to-device copy of a column chunk", e); break; }

    SetupParams S;
    S.K = K; S.m = c.mc; S.p = cfg.p; S.q = q; S.comp_base = cfg.comp_base + c.first; S.T = T;
    S.use_mask = 1; S.plan = 1; S.seed = cfg.seed; S.round = round;
    S.off = h->d_chunk_off + c.off_at;
    S.periods = nullptr;
    S.mask = hs.tables + h->t_mask;
    S.nbr = reinterpret_cast<int32_t*>(hs.tables + h->t_nbr);
    S.tile_prefix = reinterpret_cast<int32_t*>(hs.tables);
    e = launch_setup(S, cs);
    if (e != cudaSuccess) { st = cuda_fail(nullptr, "launch of the round set-up kernel", e); break; }
    st = launch_round(&hs.ctx, cfg, hs.ctx.launch, hs.ctx.theta, hs.ctx.omega, hs.ctx.delta, chunk_cols, c.mc,
                      S.off, S.tile_prefix, S.nbr, reinterpret_cast<int32_t*>(hs.tables + h->t_status), total, cs);
    if (st != GBMUF_OK) { g_create_error = hs.ctx.err; break; }
    e = copy_rows((char*)theta + (size_t)c0 * esz, (size_t)cfg.ld * esz, hs.ctx.theta, (size_t)chunk_cols * esz,
                  w_th, K, cudaMemcpyDeviceToHost, cs, rc);
    if (e == cudaSuccess && bmuf) {
      e = copy_rows(omega + c0, (size_t)cfg.ld * 4, hs.ctx.omega, (size_t)chunk_cols * 4, w_f, K,
                    cudaMemcpyDeviceToHost, cs, rc);
      if (e == cudaSuccess)
        e = copy_rows(delta + c0, (size_t)cfg.ld * 4, hs.ctx.delta, (size_t)chunk_cols * 4, w_f, K,
                      cudaMemcpyDeviceToHost, cs, rc);
    }
    if (e != cudaSuccess) { st = cuda_fail(nullptr, "device-to-host copy of a column chunk", e); break; }
  }
  // the call returns when the host arrays hold the result: wait for every set, read its status
  int32_t worst = 0;
  for (int i = 0; i < h->nsets; ++i) {
    int32_t word = 0;
    e = cudaMemcpyAsync(&word, h->sets[i].tables + h->t_status, 4, cudaMemcpyDeviceToHost, h->sets[i].stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->sets[i].stream);
    if (e != cudaSuccess && st == GBMUF_OK) st = cuda_fail(nullptr, "waiting for the column chunks", e);
    if (word != 0) {
      worst = word;
      cudaMemsetAsync(h->sets[i].tables + h->t_status, 0, 4, h->sets[i].stream);
    }
  }
  if (st == GBMUF_OK && worst != 0)
    st = fail(nullptr, GBMUF_ERR_TIMEOUT, "a bounded device-side wait expired; the host arrays are unspecified");
  return st;
}

gbmuf_status gbmuf_host_destroy(gbmuf_host* h) {
  if (!h) return GBMUF_OK;
  gbmuf_status rc = GBMUF_OK;
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) rc = GBMUF_ERR_CUDA;
  for (int i = 0; i < h->nsets && guard.ok; ++i)
    if (h->sets[i].stream && cudaStreamSynchronize(h->sets[i].stream) != cudaSuccess) rc = GBMUF_ERR_CUDA;
  free_host_handle(h);
  return rc;
}

gbmuf_status gbmuf_sync_round_host(const gbmuf_config* cfg, void* theta, float* omega, float* delta,
                                   int32_t m, const int64_t* offsets, const uint8_t* comp_mask,
                                   uint64_t round, int64_t chunk_cols) {
  gbmuf_host* h = nullptr;
  gbmuf_status st = gbmuf_host_create(cfg, m, offsets, chunk_cols, 0, &h);
  if (st != GBMUF_OK) return st;
  st = gbmuf_host_sync_round(h, theta, omega, delta, comp_mask, round);
  const gbmuf_status st2 = gbmuf_host_destroy(h);
  return st != GBMUF_OK ? st : st2;
}


// -------------------------------------------------------------------------------------------------
// One worker per GPU: gbmuf_peer_*
// -------------------------------------------------------------------------------------------------
}  // extern "C"

struct gbmuf_peer {
  gbmuf_config cfg;
  int rank = 0;
  void* theta_own[2] = {nullptr, nullptr};
  float* omega = nullptr;
  float* delta = nullptr;
  const void** d_theta_in[2] = {nullptr, nullptr};   // device arrays [K] of row pointers
  int m = 0;
  bool partitioned = false;
  std::vector<int64_t> off;
  std::vector<int32_t> periods;
  unsigned char* tables = nullptr;   // offsets | prefix | periods | mask | due | nbr
  size_t t_prefix = 0, t_periods = 0, t_mask = 0, t_due = 0, t_nbr = 0;
  int32_t* d_status = nullptr;
  long long total_tiles = 0;
  int num_sms = 0, max_smem = 0;
  int T = 0, stages = 0, ncons = 0;
  uint32_t stage_stride = 0, omega_off = 0, delta_off = 0, desc_off = 0, smem = 0;
  std::vector<uint8_t> mask_stage;   // the library's own (pageable) copy of a caller's mask
  size_t cap_bytes = 0;              // size the table block was allocated for
  WorkMarks work;
};

extern "C" {

gbmuf_status gbmuf_peer_create(const gbmuf_config* cfg, int32_t rank, void* const* theta_bufs,
                               float* omega, float* delta, gbmuf_peer** out) {
  if (!cfg || !out || !theta_bufs) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "cfg, theta_bufs and out must not be NULL");
  if (cfg->K < 1 || cfg->K > 65535 || rank < 0 || rank >= cfg->K)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "K must be in 1..65535 and 0 <= rank < K");
  if (cfg->N < 1 || cfg->ld < cfg->N || cfg->ld % 32 != 0 || cfg->p < 0 || cfg->q < 0 || cfg->comp_base < 0 ||
      (cfg->mode != GBMUF_MODE_BMUF && cfg->mode != GBMUF_MODE_MA) ||
      (cfg->theta_dtype != GBMUF_F32 && cfg->theta_dtype != GBMUF_BF16) ||
      !(cfg->eta == cfg->eta) || !(cfg->zeta == cfg->zeta) || cfg->device < 0)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "configuration out of range (see gbmuf_create)");
  const int cand = host_candidates(cfg->K, cfg->p);
  if (cfg->q > cand) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "q exceeds the ring neighbours min(2p, K-1)");
  if (cand > kMaxCand) return fail(nullptr, GBMUF_ERR_UNSUPPORTED, "more than 64 ring neighbours per worker");
  if (cfg->q > 15) return fail(nullptr, GBMUF_ERR_UNSUPPORTED, "more than 15 neighbours per draw in the peer form");
  if (!omega || !delta || (((uintptr_t)omega | (uintptr_t)delta) % 128) != 0)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "omega and delta must be 128-byte aligned device pointers");
  for (int b = 0; b < 2; ++b)
    for (int j = 0; j < cfg->K; ++j) {
      const void* ptr = theta_bufs[(size_t)b * cfg->K + j];
      if (!ptr || (uintptr_t)ptr % 128 != 0)
        return fail(nullptr, GBMUF_ERR_INVALID_ARG, "every theta buffer pointer must be non-NULL and 128-byte aligned");
    }
  if (theta_bufs[rank] == theta_bufs[(size_t)cfg->K + rank])
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "the worker's two theta buffers must be different");
  int ndev = 0;
  cudaError_t e = cudaGetDeviceCount(&ndev);
  if (e != cudaSuccess) return cuda_fail(nullptr, "cudaGetDeviceCount", e);
  if (cfg->device >= ndev) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "no such CUDA device");
  DeviceGuard guard(cfg->device);
  if (!guard.ok) return fail(nullptr, GBMUF_ERR_CUDA, "cudaSetDevice failed");
  gbmuf_peer* h = new (std::nothrow) gbmuf_peer();
  if (!h) return fail(nullptr, GBMUF_ERR_ALLOC, "out of host memory");
  h->cfg = *cfg; h->rank = rank; h->omega = omega; h->delta = delta;
  h->theta_own[0] = theta_bufs[rank];
  h->theta_own[1] = theta_bufs[(size_t)cfg->K + rank];
  int v = 0;
  cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, cfg->device); h->num_sms = v;
  cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, cfg->device); h->max_smem = v;
  // launch shape: the widest power-of-two tile whose stage ((q+1) theta rows + omega + Delta)
  // stays under 56 KB, so that four stages fit
  const int esz = cfg->theta_dtype == GBMUF_F32 ? 4 : 2;
  const bool bmuf = cfg->mode == GBMUF_MODE_BMUF;
  auto stage_bytes = [&](int T) {
    long long at = ((long long)(cfg->q + 1) * T * esz + 127) / 128 * 128;
    h->omega_off = (uint32_t)at;
    if (bmuf) at += (long long)T * 4;
    h->delta_off = (uint32_t)at;
    if (bmuf) at += (long long)T * 4;
    h->desc_off = (uint32_t)at;
    at += (long long)sizeof(TileDesc);
    return (at + 127) / 128 * 128;
  };
  int T = 4096;
  while (T > 64 && stage_bytes(T) > 56 * 1024) T >>= 1;
  h->T = T;
  h->stage_stride = (uint32_t)stage_bytes(T);
  h->stages = (int)((h->max_smem - 128) / h->stage_stride);
  if (h->stages > 4) h->stages = 4;
  if (h->stages < 1) { delete h; return fail(nullptr, GBMUF_ERR_UNSUPPORTED, "a stage does not fit shared memory"); }
  h->smem = 128 + (uint32_t)h->stages * h->stage_stride;
  int n = (T / 4 + 31) / 32 * 32;
  h->ncons = n < 128 ? 128 : n > 992 ? 992 : n;
  e = ensure_kernel_attributes(cfg->device, h->max_smem);
  if (e == cudaSuccess) e = cudaMalloc(&h->d_status, sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMemset(h->d_status, 0, sizeof(int32_t));
  for (int b = 0; b < 2 && e == cudaSuccess; ++b) {
    e = cudaMalloc(&h->d_theta_in[b], (size_t)cfg->K * sizeof(void*));
    if (e == cudaSuccess)
      e = cudaMemcpy(h->d_theta_in[b], theta_bufs + (size_t)b * cfg->K, (size_t)cfg->K * sizeof(void*),
                     cudaMemcpyHostToDevice);
  }
  if (e != cudaSuccess) {
    cudaFree(h->d_status); cudaFree(h->d_theta_in[0]); cudaFree(h->d_theta_in[1]);
    delete h;
    return e == cudaErrorMemoryAllocation ? fail(nullptr, GBMUF_ERR_ALLOC, "peer pointer tables")
                                          : cuda_fail(nullptr, "peer context set-up", e);
  }
  *out = h;
  return GBMUF_OK;
}

gbmuf_status gbmuf_peer_set_partition(gbmuf_peer* h, int32_t m, const int64_t* offsets,
                                      const int32_t* periods) {
  if (!h) return GBMUF_ERR_INVALID_ARG;
  if (m < 1 || m > 65536 || !offsets) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "m must be in 1..65536 and offsets not NULL");
  if (offsets[0] != 0 || offsets[m] != h->cfg.N)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "offsets[0] must be 0 and offsets[m] must be N");
  for (int i = 0; i < m; ++i) {
    if (offsets[i + 1] <= offsets[i]) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "offsets must be strictly increasing");
    if (periods && periods[i] < 1) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "periods must be >= 1");
  }
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return fail(nullptr, GBMUF_ERR_CUDA, "cudaSetDevice failed");
  cudaError_t e = h->work.wait();               // this worker's earlier rounds, nothing else
  if (e != cudaSuccess) return cuda_fail(nullptr, "waiting for the worker's earlier work", e);
  h->partitioned = false;
  h->m = m;
  h->off.assign(offsets, offsets + m + 1);
  if (periods) h->periods.assign(periods, periods + m); else h->periods.assign(m, 1);
  std::vector<int32_t> prefix((size_t)m + 1);
  long long total = 0;
  for (int i = 0; i < m; ++i) {              // every component has tiles: idle ones are copied through
    prefix[i] = (int32_t)total;
    const int64_t start = offsets[i] & ~(int64_t)(kAlign - 1);
    total += (offsets[i + 1] - start + h->T - 1) / h->T;
    if (total > 0x3fffffffLL) return fail(nullptr, GBMUF_ERR_UNSUPPORTED, "more than 2^30 - 1 tiles");
  }
  prefix[m] = (int32_t)total;
  h->total_tiles = total;
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  h->t_prefix = up((size_t)(m + 1) * 8);
  h->t_periods = h->t_prefix + up((size_t)(m + 1) * 4);
  h->t_mask = h->t_periods + up((size_t)m * 4);
  h->t_due = h->t_mask + up((size_t)m);
  h->t_nbr = h->t_due + up((size_t)m);
  const size_t bytes = h->t_nbr + up((size_t)m * (h->cfg.q > 0 ? h->cfg.q : 1) * 4);
  if (bytes > h->cap_bytes) {
    cudaFree(h->tables);
    h->tables = nullptr; h->cap_bytes = 0;
    e = cudaMalloc(&h->tables, bytes);
    if (e == cudaSuccess) h->cap_bytes = bytes;
  }
  if (e == cudaSuccess) e = cudaMemcpy(h->tables, h->off.data(), (size_t)(m + 1) * 8, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(h->tables + h->t_prefix, prefix.data(), (size_t)(m + 1) * 4, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(h->tables + h->t_periods, h->periods.data(), (size_t)m * 4, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaStreamSynchronize(nullptr);   // the copies above have landed
  if (e != cudaSuccess) {
    cudaFree(h->tables);
    h->tables = nullptr; h->cap_bytes = 0;
    return e == cudaErrorMemoryAllocation ? fail(nullptr, GBMUF_ERR_ALLOC, "partition tables") : cuda_fail(nullptr, "partition upload", e);
  }
  h->partitioned = true;
  return GBMUF_OK;
}

gbmuf_status gbmuf_peer_sync_round(gbmuf_peer* h, uint64_t round, const uint8_t* comp_mask,
                                   int32_t read_buffer, void* stream) {
  if (!h) return GBMUF_ERR_INVALID_ARG;
  if (!h->partitioned) return fail(nullptr, GBMUF_ERR_BAD_STATE, "gbmuf_peer_set_partition has not been called");
  if (read_buffer != 0 && read_buffer != 1) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "read_buffer must be 0 or 1");
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return fail(nullptr, GBMUF_ERR_CUDA, "cudaSetDevice failed");
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e;
  if (comp_mask) {
    // as in gbmuf_sync_round: no mask inside a stream capture, and the upload starts from the
    // library's own pageable copy so that the caller's (possibly page-locked) array is not read
    // after the call
    if (is_capturing(st))
      return fail(nullptr, GBMUF_ERR_BAD_STATE,
                  "a component mask cannot be recorded into a stream capture; select components by periods there");
    h->mask_stage.assign(comp_mask, comp_mask + h->m);
    e = cudaMemcpyAsync(h->tables + h->t_mask, h->mask_stage.data(), (size_t)h->m, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(nullptr, "upload of the component mask", e);
  }
  PeerPlanParams Q;
  Q.K = h->cfg.K; Q.m = h->m; Q.p = h->cfg.p; Q.q = h->cfg.q; Q.comp_base = h->cfg.comp_base;
  Q.rank = h->rank; Q.use_mask = comp_mask ? 1 : 0; Q.seed = h->cfg.seed; Q.round = round;
  Q.periods = reinterpret_cast<const int32_t*>(h->tables + h->t_periods);
  Q.mask = h->tables + h->t_mask;
  Q.nbr = reinterpret_cast<int32_t*>(h->tables + h->t_nbr);
  Q.due = h->tables + h->t_due;
  peer_plan_kernel<<<(h->m + 255) / 256, 256, 0, st>>>(Q);
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(nullptr, "launch of the peer plan kernel", e);
  PeerParams P;
  P.theta_in = h->d_theta_in[read_buffer];
  P.theta_out = h->theta_own[1 - read_buffer];
  P.omega = h->omega; P.delta = h->delta;
  P.off = reinterpret_cast<const int64_t*>(h->tables);
  P.tile_prefix = reinterpret_cast<const int32_t*>(h->tables + h->t_prefix);
  P.nbr = Q.nbr; P.due = Q.due; P.status = h->d_status;
  P.N = h->cfg.N; P.rank = h->rank; P.m = h->m; P.q = h->cfg.q; P.mode = h->cfg.mode;
  P.eta = h->cfg.eta; P.zeta = h->cfg.zeta;
  const int qp1 = h->cfg.q + 1;
  P.qp1 = (float)qp1; P.inv_qp1 = 1.0f / (float)qp1; P.inv_exact = (qp1 & (qp1 - 1)) == 0;
  P.T = h->T; P.stages = h->stages; P.ncons = h->ncons;
  P.stage_stride = h->stage_stride; P.omega_off = h->omega_off; P.delta_off = h->delta_off;
  P.desc_off = h->desc_off;
  const int grid = (int)(h->total_tiles < h->num_sms ? h->total_tiles : h->num_sms);
  if (h->cfg.theta_dtype == GBMUF_F32)
    peer_round_kernel<float><<<grid, 32 + h->ncons, h->smem, st>>>(P);
  else
    peer_round_kernel<__nv_bfloat16><<<grid, 32 + h->ncons, h->smem, st>>>(P);
  e = cudaGetLastError();
  h->work.note(st);
  if (e != cudaSuccess) return cuda_fail(nullptr, "launch of the peer round kernel", e);
  return GBMUF_OK;
}

gbmuf_status gbmuf_peer_device_status(gbmuf_peer* h, void* stream, int32_t* out) {
  if (!h || !out) return GBMUF_ERR_INVALID_ARG;
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return fail(nullptr, GBMUF_ERR_CUDA, "cudaSetDevice failed");
  cudaStream_t st = (cudaStream_t)stream;
  int32_t v = 0;
  cudaError_t e = cudaMemcpyAsync(&v, h->d_status, sizeof(v), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(h->d_status, 0, sizeof(v), st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return cuda_fail(nullptr, "read of the device status word", e);
  *out = v;
  return GBMUF_OK;
}

gbmuf_status gbmuf_peer_destroy(gbmuf_peer* h) {
  if (!h) return GBMUF_OK;
  gbmuf_status rc = GBMUF_OK;
  {
    DeviceGuard guard(h->cfg.device);
    if (guard.ok) {
      if (h->work.wait() != cudaSuccess) rc = GBMUF_ERR_CUDA;   // this worker's own rounds only
      h->work.release();
      cudaFree(h->tables); cudaFree(h->d_status); cudaFree(h->d_theta_in[0]); cudaFree(h->d_theta_in[1]);
    } else {
      rc = GBMUF_ERR_CUDA;
    }
  }
  delete h;
  return rc;
}

}  // extern "C"
