// libgbmuf: the random-gossip BMUF synchronisation round (Algorithm 1 of "A Random Gossip BMUF
// Process for Neural Language Modeling") for K parameter replicas resident in one GPU's memory.
// CUDA for sm_100a.  The interface is include/gbmuf.h; this file holds the kernels and the
// host-side C ABI.
//
// Kernels
//   round_setup_kernel   neighbour draws for every (worker, component) of a round + the tile
//                        work-list prefix of the components that take part
//   sync_fused_kernel    gather + average + block-momentum filter, one pass, in place
//   perturb_kernel       synthetic local steps (counter-based noise)
//   init_kernel          theta^k <- theta_0, omega^k <- theta_0, Delta^k <- 0
//   final_average_kernel theta = (1/K) sum_k theta^k
//
// Floating point: every operation is an explicit round-to-nearest intrinsic (__fadd_rn,
// __fmul_rn, __fdiv_rn) so that nothing is contracted into a fused multiply-add.

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <type_traits>
#include <vector>

#include "gbmuf.h"

namespace {

// =================================================================================================
// Philox4x32-10 (Salmon et al., SC'11), device side
// =================================================================================================
struct Philox4 { uint32_t x, y, z, w; };

__device__ __forceinline__ Philox4 philox4x32_10(Philox4 c, uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    Philox4 n;
    n.x = hi1 ^ c.y ^ k0;
    n.y = lo1;
    n.z = hi0 ^ c.w ^ k1;
    n.w = lo0;
    c = n;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return c;
}

constexpr uint32_t kTagSampler = 0x53414D50u;  // second key word of the neighbour-draw stream
constexpr uint32_t kTagPerturb = 0x50455254u;  // second key word of the local-step noise stream
constexpr int kMaxCand = 64;                   // largest candidate set min(2p, K-1)
constexpr int kAlign = 8;                      // tiles start on multiples of 8 elements (>= 16 B)

// =================================================================================================
// Round set-up: neighbour draws (Algorithm 1, the neighbour-choice line: k_1..k_q) and the
// work-list of this round.
// =================================================================================================
struct SetupParams {
  int K, m, p, q, comp_base, T, use_mask, plan;
  uint64_t seed, round;
  const int64_t* off;      // [m+1]
  const int32_t* periods;  // [m]
  const uint8_t* mask;     // [m] when use_mask
  int32_t* nbr;            // [m][K][q]
  int32_t* tile_prefix;    // [m+1]
};

// Ring neighbours of worker k (Definition 1): (k-1)%K..(k-p)%K then (k+1)%K..(k+p)%K, leaving
// out k itself and anything already listed.  Returns the count.
__device__ int ring_candidates(int k, int K, int p, int32_t* a) {
  int c = 0;
  for (int side = 0; side < 2; ++side) {
    for (int d = 1; d <= p && c < kMaxCand; ++d) {
      const int step = d % K;
      int node = side == 0 ? k - step : k + step;
      if (node < 0) node += K;
      if (node >= K) node -= K;
      if (node == k) continue;
      bool seen = false;
      for (int j = 0; j < c; ++j) seen |= (a[j] == node);
      if (!seen) a[c++] = node;
    }
  }
  return c;
}

__device__ __forceinline__ int tiles_of_component(int64_t lo, int64_t hi, int T) {
  if (hi <= lo) return 0;
  const int64_t start = lo & ~(int64_t)(kAlign - 1);
  return (int)((hi - start + T - 1) / T);
}

__global__ void __launch_bounds__(256) round_setup_kernel(SetupParams P) {
  const int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (g < (int64_t)P.K * P.m && P.q > 0) {
    const int i = (int)(g / P.K), k = (int)(g % P.K);
    int32_t a[kMaxCand];
    const int c = ring_candidates(k, P.K, P.p, a);
    int32_t* out = P.nbr + g * P.q;
    Philox4 r = {0, 0, 0, 0};
    for (int j = 0; j < P.q && j < c; ++j) {
      if ((j & 3) == 0) {
        Philox4 ctr = {(uint32_t)P.round, (uint32_t)(P.round >> 32), (uint32_t)(P.comp_base + i),
                       (uint32_t)k | ((uint32_t)(j >> 2) << 16)};
        r = philox4x32_10(ctr, (uint32_t)P.seed, (uint32_t)(P.seed >> 32) ^ kTagSampler);
      }
      const uint32_t u = (j & 3) == 0 ? r.x : (j & 3) == 1 ? r.y : (j & 3) == 2 ? r.z : r.w;
      const int t = j + (int)__umulhi(u, (uint32_t)(c - j));   // partial Fisher-Yates
      const int32_t tmp = a[j];
      a[j] = a[t];
      a[t] = tmp;
      out[j] = a[j];
    }
  }

  // Block 0 also lays out the work-list: tile_prefix[i] = number of tiles of the participating
  // components before i.  Block-wide exclusive scan, 256 components at a time.
  if (blockIdx.x == 0 && P.plan) {
    __shared__ int warp_tot[8];
    __shared__ int carry_s;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (int base = 0; base < P.m; base += 256) {
      const int i = base + threadIdx.x;
      int cnt = 0;
      if (i < P.m) {
        const bool due = P.use_mask ? (P.mask[i] != 0) : (P.round % (uint64_t)P.periods[i] == 0);
        if (due) cnt = tiles_of_component(P.off[i], P.off[i + 1], P.T);
      }
      int inc = cnt;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += n;
      }
      if (lane == 31) warp_tot[wid] = inc;
      __syncthreads();
      int before = 0;
      for (int w2 = 0; w2 < wid; ++w2) before += warp_tot[w2];
      const int carry = carry_s;
      if (i < P.m) P.tile_prefix[i] = carry + before + inc - cnt;
      __syncthreads();
      if (threadIdx.x == 255) carry_s = carry + before + inc;
      __syncthreads();
    }
    if (threadIdx.x == 0) P.tile_prefix[P.m] = carry_s;
  }
}

// =================================================================================================
// Shared-memory barrier and bulk-copy primitives (PTX).  Every wait is bounded.
// =================================================================================================
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // two seconds
// Wait for the phase with the given parity to complete.  Bounded in wall-clock time: after
// kWaitLimitNs it records GBMUF_ERR_TIMEOUT in the device status word and returns false; the
// caller then leaves its loop.  (try_wait may itself suspend the thread for a while, so the bound
// is on the timer, not on the number of tries.)
__device__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, int32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_timer_ns();
  for (uint32_t spin = 0;; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    if (spin > 32) __nanosleep(spin > 4096 ? 256 : 32);
    if ((spin & 63) == 63 && global_timer_ns() - t0 > kWaitLimitNs) break;
  }
  atomicExch(status, (int32_t)GBMUF_ERR_TIMEOUT);
  return false;
}
// Two-dimensional tiled TMA load: the box [rows 0..K) x [columns x, x + box width) of a row-major
// [K][ld] array lands in shared memory as K consecutive rows of box-width elements.  One request
// per box (no multicast); completion is counted in bytes on the mbarrier, out-of-range columns
// are zero-filled and still counted.  x * element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_box(uint32_t dst_smem, const CUtensorMap* map, int x, int y,
                                             uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], "
      "[%1, {%2, %3}], [%4];" ::"r"(dst_smem),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
      : "memory");
}

// One-dimensional bulk copy global -> shared through the copy engine (no multicast); completion
// is counted in bytes on the mbarrier.  Addresses and size are multiples of 16 bytes.
__device__ __forceinline__ void bulk_load_row(uint32_t dst_smem, const void* src, uint32_t bytes,
                                              uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          dst_smem),
      "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}

// =================================================================================================
// theta storage types
// =================================================================================================
template <typename TH> struct ThetaTraits;
template <> struct ThetaTraits<float> {
  static constexpr int VEC = 4;   // elements per 16-byte vector of theta
  static __device__ __forceinline__ float widen(float v) { return v; }
  static __device__ __forceinline__ float round_store(float v) { return v; }
  static __device__ __forceinline__ float narrow(float v) { return v; }
  static __device__ __forceinline__ void lds(const float* p, float (&x)[4]) {
    const float4 t = *reinterpret_cast<const float4*>(p);
    x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w;
  }
  static __device__ __forceinline__ void stg(float* p, const float (&x)[4]) {
    __stcs(reinterpret_cast<float4*>(p), make_float4(x[0], x[1], x[2], x[3]));
  }  // four consecutive elements (what one thread of the fused kernel handles per row)
  static __device__ __forceinline__ void lds_quad(const float* p, float (&x)[4]) { lds(p, x); }
  static __device__ __forceinline__ void stg_quad(float* p, const float (&x)[4]) { stg(p, x); }
};
template <> struct ThetaTraits<__nv_bfloat16> {
  static constexpr int VEC = 8;
  static __device__ __forceinline__ float widen(__nv_bfloat16 v) { return __bfloat162float(v); }
  // value of v after a round trip through bf16 storage (round to nearest, ties to even)
  static __device__ __forceinline__ float round_store(float v) {
    return __bfloat162float(__float2bfloat16_rn(v));
  }
  static __device__ __forceinline__ __nv_bfloat16 narrow(float v) { return __float2bfloat16_rn(v); }
  static __device__ __forceinline__ void lds(const __nv_bfloat16* p, float (&x)[8]) {
    const uint4 t = *reinterpret_cast<const uint4*>(p);
    x[0] = __uint_as_float(t.x << 16); x[1] = __uint_as_float(t.x & 0xFFFF0000u);
    x[2] = __uint_as_float(t.y << 16); x[3] = __uint_as_float(t.y & 0xFFFF0000u);
    x[4] = __uint_as_float(t.z << 16); x[5] = __uint_as_float(t.z & 0xFFFF0000u);
    x[6] = __uint_as_float(t.w << 16); x[7] = __uint_as_float(t.w & 0xFFFF0000u);
  }
  static __device__ __forceinline__ void stg(__nv_bfloat16* p, const float (&x)[8]) {
    uint4 t;
    __nv_bfloat162 h;
    h = __floats2bfloat162_rn(x[0], x[1]); t.x = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2bfloat162_rn(x[2], x[3]); t.y = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2bfloat162_rn(x[4], x[5]); t.z = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2bfloat162_rn(x[6], x[7]); t.w = *reinterpret_cast<uint32_t*>(&h);
    __stcs(reinterpret_cast<uint4*>(p), t);
  }
  // four consecutive elements = 8 bytes
  static __device__ __forceinline__ void lds_quad(const __nv_bfloat16* p, float (&x)[4]) {
    const uint2 t = *reinterpret_cast<const uint2*>(p);
    x[0] = __uint_as_float(t.x << 16); x[1] = __uint_as_float(t.x & 0xFFFF0000u);
    x[2] = __uint_as_float(t.y << 16); x[3] = __uint_as_float(t.y & 0xFFFF0000u);
  }
  static __device__ __forceinline__ void stg_quad(__nv_bfloat16* p, const float (&x)[4]) {
    uint2 t;
    __nv_bfloat162 h;
    h = __floats2bfloat162_rn(x[0], x[1]); t.x = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2bfloat162_rn(x[2], x[3]); t.y = *reinterpret_cast<uint32_t*>(&h);
    __stcs(reinterpret_cast<uint2*>(p), t);
  }
};

// =================================================================================================
// The fused round: gather + average + block-momentum filter, in place, one pass.
//
// Work item = one tile: up to T consecutive elements of ONE component, for all K workers.  A
// persistent CTA walks tiles blockIdx.x, blockIdx.x + gridDim.x, ...
//
// Shared memory holds (a) one or two theta stages, each the K replicas' slices of a tile -- every
// worker's average may need any other worker's slice, so the whole K-row tile must be resident --
// and (b) a small ring of row slots for omega and Delta, which are needed exactly once per
// (worker, element) and therefore only pass through.  Keeping omega and Delta out of the tile
// stage is what lets T, the contiguous run per row, be as long as 8 KB: measured DRAM efficiency
// grows with that run length far more than with pipeline depth.
//
// Warp 0 is the producer.  Per tile it looks the tile up in the work-list, has the copy engine
// fetch the theta stage (tiled TMA, one request per [K rows x 256 columns] box) and then, worker by
// worker, one row of omega and one of Delta into the next free ring slot (bulk copies).  The other
// warps are consumers: they wait for the theta stage, then for each worker k wait for its ring
// slot; each thread takes 16-byte vectors of the row, sums worker k's own slice and its q
// neighbours' slices out of shared memory (own first, then draw order), divides by q+1, applies the
// filter and writes Delta, omega and the restart point theta straight to global memory, then
// releases the slot.  All global reads are issued by the copy engine, so the bytes in flight do
// not depend on how many threads are resident.  Because the CTA is the only reader and writer of
// its tile in all K replicas and has staged the pre-round theta before writing any, every
// neighbour read sees the replica as it was before the round.  Unique traffic per
// replica-parameter: theta read once, omega and Delta read once, all three written once.
//
// Every wait is bounded; a wait that expires records GBMUF_ERR_TIMEOUT and the thread leaves.
// =================================================================================================
struct TileDesc {
  long long e0;   // first element of the staged range (multiple of kAlign)
  long long lo;   // first element this tile owns
  long long hi;   // one past the last element this tile owns
  int comp;
  int pad;
};

constexpr int kMaxRing = 8;
// barrier block at the start of shared memory (8 bytes each)
constexpr uint32_t kBarThetaFull = 0, kBarThetaEmpty = 32, kBarRingFull = 64, kBarRingEmpty = 128;
constexpr int kMaxThetaStages = 4;
constexpr uint32_t kBarBytes = 256;

struct SyncParams {
  void* theta;
  float* omega;
  float* delta;
  const int64_t* off;
  const int32_t* tile_prefix;
  const int32_t* nbr;   // [m][K][q]
  int32_t* status;
  long long ld;
  int K, m, q, mode;
  float eta, zeta, qp1, inv_qp1;
  int inv_exact;        // q+1 is a power of two: multiplying by 1/(q+1) equals dividing
  int T, BW, bw_shift, bw_mask;   // BW: columns per TMA box; column c of a tile is in box
                                  // c >> bw_shift at c & bw_mask
  int stages, ring, ncons;        // theta stages (1..4), ring slots, consumer threads
  uint32_t stage_stride, nbr_off, desc_off;   // theta stage: [theta boxes | nbr | desc]
  uint32_t ring_off, slot_stride;             // ring slot: [omega row T floats | Delta row T floats]
};

// The division of the gossip average, s / (q+1), for four elements.  The result is that of the
// IEEE-754 division rounded to nearest even, bit for bit, for every input; only the route differs:
//  - q+1 a power of two: multiplying by 1/(q+1) is exact;
//  - otherwise, for the small integer divisor b = q+1 and y = RN(1/b): q0 = RN(s*y), the exact
//    residual r = fma(-b, q0, s), then RN(q0 + r*y) (Markstein's correction step).  It is taken
//    only when the exponent of s is in the middle range, where no intermediate can overflow,
//    underflow or be subnormal; zeros, subnormals, huge values, infinities and NaNs go through the
//    division instruction sequence.  gbmuf_selftest_divide compares this routine with the plain
//    division over all 2^32 bit patterns for a given divisor.
// Costs 3 arithmetic instructions per element instead of about 10; gossip-MA with q+1 = 3 was
// limited by the divide.
// Exponent test: the result has one of its two top bits set iff the biased exponent of s is
// outside [64, 191], i.e. unless 2^-63 <= |s| < 2^65; results of several values may be OR-ed.
__device__ __forceinline__ uint32_t outside_mid_range(float s) {
  return (__float_as_uint(s) & 0x7F800000u) - 0x20000000u;
}
__device__ __forceinline__ float divide_corrected(float s, float b, float y) {
  const float q0 = __fmul_rn(s, y);
  const float r = __fmaf_rn(-b, q0, s);
  return __fmaf_rn(r, y, q0);
}
__device__ __forceinline__ void average_divide(float (&a)[4], float b, float y, int y_exact) {
  if (y_exact) {
#pragma unroll
    for (int x = 0; x < 4; ++x) a[x] = __fmul_rn(a[x], y);
  } else if (!((outside_mid_range(a[0]) | outside_mid_range(a[1]) | outside_mid_range(a[2]) |
                outside_mid_range(a[3])) & 0xC0000000u)) {
#pragma unroll
    for (int x = 0; x < 4; ++x) a[x] = divide_corrected(a[x], b, y);
  } else {
#pragma unroll
    for (int x = 0; x < 4; ++x) a[x] = __fdiv_rn(a[x], b);
  }
}

// Block-momentum filter for one element (Algorithm 1: G, Delta, omega, theta lines).  The
// block-start value is recomputed from the pre-round omega and Delta.
template <typename TH>
__device__ __forceinline__ void bmuf_filter(float avg, float& w, float& d, float& t, float eta,
                                            float zeta) {
  const float etad = __fmul_rn(eta, d);
  const float r = ThetaTraits<TH>::round_store(__fadd_rn(w, etad));
  const float g = __fsub_rn(avg, r);
  d = __fadd_rn(etad, __fmul_rn(zeta, g));
  w = __fadd_rn(w, d);
  t = __fadd_rn(w, __fmul_rn(eta, d));
}

template <typename TH>
__global__ void __launch_bounds__(1024, 1)
sync_fused_kernel(const SyncParams P, const __grid_constant__ CUtensorMap map_theta) {
  constexpr int VEC = 4;   // elements per thread and row: 16 bytes of omega / Delta, 16 or 8 of theta
  extern __shared__ __align__(128) unsigned char smem[];
  const uint32_t bars = smem_u32(smem);
  unsigned char* stage0 = smem + kBarBytes;
  unsigned char* ring0 = smem + P.ring_off;
  const int total = P.tile_prefix[P.m];
  const int S = P.stages, R = P.ring;
  const bool bmuf = P.mode == GBMUF_MODE_BMUF;
  const int my_tiles = (int)blockIdx.x < total ? (total - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(bars + kBarThetaFull + 8 * s, 1);          // the producer's arrival + bytes
      mbar_init(bars + kBarThetaEmpty + 8 * s, P.ncons);   // every consumer thread arrives
      reinterpret_cast<TileDesc*>(stage0 + (size_t)s * P.stage_stride + P.desc_off)->comp = -1;
    }
    for (int r = 0; r < R; ++r) {
      mbar_init(bars + kBarRingFull + 8 * r, 1);
      mbar_init(bars + kBarRingEmpty + 8 * r, P.ncons);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  if (threadIdx.x < 32) {
    // ------------------------------------------------------------------ producer warp
    const int lane = threadIdx.x;
    bool ok = true;
    // The tiles of this CTA come in increasing order, so the component only ever moves forward:
    // find the first one by bisection, then advance.  In the steady state the loop below touches
    // no global memory except through the copies it issues.
    int comp = 0, pfx_lo = 0, pfx_hi = 0;
    long long cb = 0, ce = 0;
    if (my_tiles > 0) {
      int lo_i = 0, hi_i = P.m;
      while (hi_i - lo_i > 1) {
        const int mid = (lo_i + hi_i) >> 1;
        if (__ldg(P.tile_prefix + mid) <= (int)blockIdx.x) lo_i = mid; else hi_i = mid;
      }
      comp = lo_i;
      pfx_lo = __ldg(P.tile_prefix + comp);
      pfx_hi = __ldg(P.tile_prefix + comp + 1);
      cb = __ldg(P.off + comp);
      ce = __ldg(P.off + comp + 1);
    }
    int theta_issued = 0;    // tiles whose theta stage has been requested
    int ring_issued = 0;     // ring slots requested so far (over all tiles)

    // request the theta stage of this CTA's j-th tile (j = theta_issued)
    auto issue_theta = [&]() -> bool {
      const int j = theta_issued;
      const int w = (int)blockIdx.x + j * (int)gridDim.x;
      const int s = j % S;
      if (j >= S) {
        bool fine = mbar_wait_bounded(bars + kBarThetaEmpty + 8 * s, ((j / S) - 1) & 1, P.status);
        if (!__all_sync(0xffffffffu, fine)) return false;
      }
      if (w >= pfx_hi) {
        while (w >= pfx_hi) {      // w < total = tile_prefix[m], so comp stays below m
          ++comp;
          pfx_lo = pfx_hi;
          pfx_hi = __ldg(P.tile_prefix + comp + 1);
        }
        cb = __ldg(P.off + comp);
        ce = __ldg(P.off + comp + 1);
      }
      const long long e0 = (cb & ~(long long)(kAlign - 1)) + (long long)(w - pfx_lo) * P.T;
      unsigned char* st = stage0 + (size_t)s * P.stage_stride;
      TileDesc* d = reinterpret_cast<TileDesc*>(st + P.desc_off);
      if (d->comp != comp) {       // the stage still holds the table of the component it last served
        int* snb = reinterpret_cast<int*>(st + P.nbr_off);
        const int32_t* gnb = P.nbr + (size_t)comp * P.K * P.q;
        for (int x = lane; x < P.K * P.q; x += 32) snb[x] = __ldg(gnb + x);
      }
      __syncwarp();
      if (lane == 0) {
        d->e0 = e0;
        d->lo = cb > e0 ? cb : e0;
        d->hi = ce < e0 + P.T ? ce : e0 + P.T;
        d->comp = comp;
      }
      __syncwarp();
      const uint32_t full = bars + kBarThetaFull + 8 * s;
      const uint32_t sbase = smem_u32(st);
      if (lane == 0) mbar_arrive_expect_tx(full, (uint32_t)P.K * (uint32_t)P.T * (uint32_t)sizeof(TH));
      __syncwarp();
      const uint32_t box_bytes = (uint32_t)P.K * (uint32_t)P.BW * (uint32_t)sizeof(TH);
      for (int b = lane; b < P.T / P.BW; b += 32)
        tma_load_box(sbase + (uint32_t)b * box_bytes, &map_theta, (int)e0 + b * P.BW, 0, full);
      ++theta_issued;
      return true;
    };

    for (int j = 0; j < S - 1 && j < my_tiles && ok; ++j) ok = issue_theta();
    for (int it = 0; it < my_tiles && ok; ++it) {
      if (it + S - 1 < my_tiles) ok = issue_theta();   // keeps S-1 tiles of theta ahead (S=1: this tile)
      if (!ok) break;
      if (bmuf) {
        const TileDesc* d = reinterpret_cast<const TileDesc*>(stage0 + (size_t)(it % S) * P.stage_stride + P.desc_off);
        const long long e0 = d->e0;
        long long run = P.ld - e0;                       // a row ends at ld: never read past it
        if (run > P.T) run = P.T;
        const uint32_t bytes = (uint32_t)run * 4u;
        for (int k = 0; k < P.K; ++k) {
          const int slot = ring_issued % R;
          if (ring_issued >= R) {
            bool fine = mbar_wait_bounded(bars + kBarRingEmpty + 8 * slot, ((ring_issued / R) - 1) & 1, P.status);
            ok = __all_sync(0xffffffffu, fine);
            if (!ok) break;
          }
          if (lane == 0) {
            const uint32_t full = bars + kBarRingFull + 8 * slot;
            const uint32_t dst = smem_u32(ring0 + (size_t)slot * P.slot_stride);
            const long long at = (long long)k * P.ld + e0;
            mbar_arrive_expect_tx(full, 2u * bytes);
            bulk_load_row(dst, P.omega + at, bytes, full);
            bulk_load_row(dst + (uint32_t)P.T * 4u, P.delta + at, bytes, full);
          }
          ++ring_issued;
        }
      }
    }
    if (!ok) {
      // leave only after the copies already requested into this CTA's shared memory have landed
      for (int j = theta_issued > S ? theta_issued - S : 0; j < theta_issued; ++j)
        mbar_wait_bounded(bars + kBarThetaFull + 8 * (j % S), (j / S) & 1, P.status);
      for (int j = ring_issued > R ? ring_issued - R : 0; j < ring_issued; ++j)
        mbar_wait_bounded(bars + kBarRingFull + 8 * (j % R), (j / R) & 1, P.status);
    }
    return;
  }

  // -------------------------------------------------------------------- consumer warps
  const int c = threadIdx.x - 32;
  const int nv = P.T / VEC;            // vectors per row of a tile
  const int q = P.q, BW = P.BW, box_elems = P.K * P.BW;
  TH* theta = static_cast<TH*>(P.theta);
  int ring_taken = 0;
  for (int it = 0; it < my_tiles; ++it) {
    const int s = it % S;
    if (!mbar_wait_bounded(bars + kBarThetaFull + 8 * s, (it / S) & 1, P.status)) return;
    unsigned char* st = stage0 + (size_t)s * P.stage_stride;
    const TH* sth = reinterpret_cast<const TH*>(st);
    const int* snb = reinterpret_cast<const int*>(st + P.nbr_off);
    const TileDesc* d = reinterpret_cast<const TileDesc*>(st + P.desc_off);
    const long long e0 = d->e0, lo = d->lo, hi = d->hi;
    if (!bmuf) {
      // gossip-MA: theta <- average.  No omega / Delta stream paces the workers, so each thread
      // walks all workers for its group of elements; unrolled so that the shared-memory loads
      // and the arithmetic of several workers overlap.
      // With more threads than element groups the workers are split between thread groups:
      // thread c takes group c % nv for workers c / nv, c / nv + kg, ...
      // The division (see average_divide) is kept free of branches inside the loop, which is
      // what lets the unrolled workers overlap: a pass either multiplies by an exact reciprocal
      // (DIV 0), or takes the corrected-product route for every element while OR-ing the exponent
      // tests (DIV 1), or divides plainly (DIV 2).  If a DIV 1 pass met a sum outside the middle
      // range, the thread repeats its share of the tile with DIV 2 from the still-staged theta,
      // overwriting what it stored.
      // Each thread takes 16 bytes of theta per row here: 4 fp32 or 8 bf16 elements.
      constexpr int MV = ThetaTraits<TH>::VEC;
      const int nvm = P.T / MV;
      const int kg = P.ncons > nvm ? P.ncons / nvm : 1;
      const int k_first = P.ncons > nvm ? c / nvm : 0;
      auto ma_pass = [&](auto div_tag) -> bool {
        constexpr int DIV = decltype(div_tag)::value;
        uint32_t oor = 0;
        for (int v = P.ncons > nvm ? c - k_first * nvm : c; v < nvm && k_first < kg; v += P.ncons) {
          const int col = v * MV;
          const long long e = e0 + col;
          if (e >= hi || e + MV <= lo) continue;
          const int b = col >> P.bw_shift, cin = col & P.bw_mask;
          const int boxbase = b * box_elems + cin;
          const bool whole = e >= lo && e + MV <= hi;
#pragma unroll 4
          for (int k = k_first; k < P.K; k += kg) {
            float a[MV], t[MV];
            ThetaTraits<TH>::lds(sth + boxbase + k * BW, a);
            for (int j = 0; j < q; ++j) {
              ThetaTraits<TH>::lds(sth + boxbase + snb[k * q + j] * BW, t);
#pragma unroll
              for (int x = 0; x < MV; ++x) a[x] = __fadd_rn(a[x], t[x]);
            }
#pragma unroll
            for (int x = 0; x < MV; ++x) {
              if (DIV == 0) {
                a[x] = __fmul_rn(a[x], P.inv_qp1);
              } else if (DIV == 1) {
                oor |= outside_mid_range(a[x]);
                a[x] = divide_corrected(a[x], P.qp1, P.inv_qp1);
              } else {
                a[x] = __fdiv_rn(a[x], P.qp1);
              }
            }
            const long long at = (long long)k * P.ld + e;
            if (whole) {
              ThetaTraits<TH>::stg(theta + at, a);
            } else {
              for (int x = 0; x < MV; ++x)
                if (e + x >= lo && e + x < hi) theta[at + x] = ThetaTraits<TH>::narrow(a[x]);
            }
          }
        }
        return (oor & 0xC0000000u) != 0;
      };
      if (P.inv_exact) {
        ma_pass(std::integral_constant<int, 0>{});
      } else if (ma_pass(std::integral_constant<int, 1>{})) {
        ma_pass(std::integral_constant<int, 2>{});
      }
      mbar_arrive(bars + kBarThetaEmpty + 8 * s);
      continue;
    }
    for (int k = 0; k < P.K; ++k) {
      const float* som = nullptr;
      const float* sde = nullptr;
      int slot = 0;
      if (bmuf) {
        slot = ring_taken % R;
        if (!mbar_wait_bounded(bars + kBarRingFull + 8 * slot, (ring_taken / R) & 1, P.status)) return;
        som = reinterpret_cast<const float*>(ring0 + (size_t)slot * P.slot_stride);
        sde = som + P.T;
      }
      for (int v = c; v < nv; v += P.ncons) {
        const int col = v * VEC;
        const long long e = e0 + col;
        if (e >= hi || e + VEC <= lo) continue;
        // staged layout of theta: box b = col / BW holds K rows of BW columns
        const int b = col >> P.bw_shift, cin = col & P.bw_mask;
        const int boxbase = b * box_elems + cin;
        // gossip average: own slice first, then the neighbours in draw order
        float a[VEC], t[VEC];
        ThetaTraits<TH>::lds_quad(sth + boxbase + k * BW, a);
        for (int j = 0; j < q; ++j) {
          ThetaTraits<TH>::lds_quad(sth + boxbase + snb[k * q + j] * BW, t);
#pragma unroll
          for (int x = 0; x < VEC; ++x) a[x] = __fadd_rn(a[x], t[x]);
        }
        average_divide(a, P.qp1, P.inv_qp1, P.inv_exact);
        const long long at = (long long)k * P.ld + e;
        const bool whole = e >= lo && e + VEC <= hi;
        if (!bmuf) {                                       // gossip-MA: theta <- average
          if (whole) {
            ThetaTraits<TH>::stg_quad(theta + at, a);
          } else {
            for (int x = 0; x < VEC; ++x)
              if (e + x >= lo && e + x < hi) theta[at + x] = ThetaTraits<TH>::narrow(a[x]);
          }
          continue;
        }
        const float4 W = *reinterpret_cast<const float4*>(som + col);
        const float4 D = *reinterpret_cast<const float4*>(sde + col);
        float wv[VEC] = {W.x, W.y, W.z, W.w}, dv[VEC] = {D.x, D.y, D.z, D.w};
#pragma unroll
        for (int x = 0; x < VEC; ++x) bmuf_filter<TH>(a[x], wv[x], dv[x], t[x], P.eta, P.zeta);
        if (whole) {
          __stcs(reinterpret_cast<float4*>(P.delta + at), make_float4(dv[0], dv[1], dv[2], dv[3]));
          __stcs(reinterpret_cast<float4*>(P.omega + at), make_float4(wv[0], wv[1], wv[2], wv[3]));
          ThetaTraits<TH>::stg_quad(theta + at, t);
        } else {
          // a vector that straddles the edge of the component: only the elements this tile owns
          for (int x = 0; x < VEC; ++x) {
            if (e + x >= lo && e + x < hi) {
              P.delta[at + x] = dv[x];
              P.omega[at + x] = wv[x];
              theta[at + x] = ThetaTraits<TH>::narrow(t[x]);
            }
          }
        }
      }
      if (bmuf) {
        mbar_arrive(bars + kBarRingEmpty + 8 * slot);    // this thread is done with the slot
        ++ring_taken;
      }
    }
    mbar_arrive(bars + kBarThetaEmpty + 8 * s);          // this thread is done with the theta stage
  }
}

// =================================================================================================
// Variant of the fused round that keeps the theta tile in tensor memory (TMEM) instead of shared
// memory.  A K x T fp32 tile of up to 256 KB does not fit shared memory next to anything else,
// but it is exactly what the 512 columns x 128 lanes of an SM's tensor memory hold.  Every row of
// theta, omega and Delta streams through one ring of shared-memory slots: first the K theta rows
// of a tile (several per slot), which each consumer thread moves from the slot into its own TMEM
// cells (tcgen05.st), then the output items, for which the thread reads its own and the drawn
// neighbours' theta back from those cells (tcgen05.ld).  A thread only ever reads cells it wrote
// itself, so TMEM needs no synchronisation between threads, and the run per row can be about
// twice as long as with a shared-memory tile.
//
// (gossip-BMUF mode only.  The same schedule was tried for gossip-MA, whose output items carry
// only averages: its consumers, 16 warps of serial TMEM round trips, could not keep up with 8
// bytes per element and it ran at 60 % of the shared-memory schedule's speed.)
//
// TMEM addressing: a warp reaches the 32 lanes 32 * (warp id % 4) ..; with the .32x32b.xN shape
// each thread moves the N consecutive 32-bit columns of its lane that start at the given column.
// Four consecutive elements of a row are one cell: 4 columns for fp32, 2 for bf16 (kept packed).
// Element group g (4 elements) of a tile lives in lane g % 128, columns ((g / 128) * K + row) *
// cell width.  The allocation is released by the warp that made it after every thread has
// reached the end of the kernel; no path returns early.
// =================================================================================================
struct TmemParams {
  const void* theta_in;    // same array as theta (read side)
  void* theta;
  float* omega;
  float* delta;
  const int64_t* off;
  const int32_t* tile_prefix;
  const int32_t* nbr;      // [m][K][q]
  int32_t* status;
  long long ld;
  int K, m, q;
  float eta, zeta, qp1, inv_qp1;
  int inv_exact;
  int T, ring, ncols;      // T multiple of 512; ring slots; TMEM columns (power of 2)
  uint32_t ring_off, meta_off, meta_stride;   // meta ring (4 entries): [TileDesc | nbr K*q ints]
  uint32_t slot_stride;    // bytes per ring slot
};

// Four consecutive theta elements of one row <-> this thread's TMEM cell.  Load and wait sit in
// ONE asm statement because the registers are only valid after the wait and nothing may be
// scheduled between the two.  (Several loads per wait were measured slower, not faster.)
template <typename TH> struct TmemCell;
template <> struct TmemCell<float> {
  static constexpr int COLS = 4;
  static __device__ __forceinline__ void deposit(uint32_t taddr, const float* src) {
    const float4 v = *reinterpret_cast<const float4*>(src);
    asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1, %2, %3, %4};" ::"r"(taddr),
                 "r"(__float_as_uint(v.x)), "r"(__float_as_uint(v.y)), "r"(__float_as_uint(v.z)),
                 "r"(__float_as_uint(v.w))
                 : "memory");
  }
  static __device__ __forceinline__ void fetch(uint32_t taddr, float (&x)[4]) {
    uint32_t a, b, c, d;
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(a), "=r"(b), "=r"(c), "=r"(d)
        : "r"(taddr)
        : "memory");
    x[0] = __uint_as_float(a); x[1] = __uint_as_float(b); x[2] = __uint_as_float(c); x[3] = __uint_as_float(d);
  }
  static __device__ __forceinline__ void sts_quad(float* dst, const float (&x)[4]) {
    *reinterpret_cast<float4*>(dst) = make_float4(x[0], x[1], x[2], x[3]);
  }
};
template <> struct TmemCell<__nv_bfloat16> {
  static constexpr int COLS = 2;
  static __device__ __forceinline__ void deposit(uint32_t taddr, const __nv_bfloat16* src) {
    const uint2 v = *reinterpret_cast<const uint2*>(src);
    asm volatile("tcgen05.st.sync.aligned.32x32b.x2.b32 [%0], {%1, %2};" ::"r"(taddr), "r"(v.x), "r"(v.y)
                 : "memory");
  }
  static __device__ __forceinline__ void fetch(uint32_t taddr, float (&x)[4]) {
    uint32_t a, b;
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0, %1}, [%2];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(a), "=r"(b)
        : "r"(taddr)
        : "memory");
    x[0] = __uint_as_float(a << 16); x[1] = __uint_as_float(a & 0xFFFF0000u);
    x[2] = __uint_as_float(b << 16); x[3] = __uint_as_float(b & 0xFFFF0000u);
  }
  static __device__ __forceinline__ void sts_quad(__nv_bfloat16* dst, const float (&x)[4]) {
    uint2 t;
    __nv_bfloat162 h;
    h = __floats2bfloat162_rn(x[0], x[1]); t.x = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2bfloat162_rn(x[2], x[3]); t.y = *reinterpret_cast<uint32_t*>(&h);
    *reinterpret_cast<uint2*>(dst) = t;
  }
};

// Sum of worker k's own cell and its q drawn neighbours' cells of element group `cell0` (the
// TMEM address of row 0's cell), own first, then draw order, each addition rounded.
template <typename TH>
__device__ __forceinline__ void tmem_gather(uint32_t cell0, int k, const int* nb, int q, float (&a)[4]) {
  constexpr int CW = TmemCell<TH>::COLS;
  TmemCell<TH>::fetch(cell0 + (uint32_t)(k * CW), a);
  for (int j = 0; j < q; ++j) {
    float t[4];
    TmemCell<TH>::fetch(cell0 + (uint32_t)(nb[j] * CW), t);
#pragma unroll
    for (int x = 0; x < 4; ++x) a[x] = __fadd_rn(a[x], t[x]);
  }
}

// What the producer must know to send a finished slot out: the staged range starts at e0, whole
// 16-byte pieces of the rows cover [sb, se); k < 0: a load item, nothing to send.
struct SlotInfo { long long e0, sb, se; int k; int pad; };

// Slot layout.  Load item: IN_ROWS rows of T theta elements.  Output item (one per worker):
// [omega T floats | Delta T floats | (BULK) new theta T elements].
// BULK: the outputs leave through bulk stores from the ring slot instead of st.global from
// registers.
template <typename TH, bool BULK>
__global__ void __launch_bounds__(544, 1) sync_fused_tmem_kernel(const TmemParams P) {
  constexpr int EB = (int)sizeof(TH);
  constexpr int CW = TmemCell<TH>::COLS;
  constexpr int IN_ROWS = 8 / EB;                    // theta rows per load item
  constexpr long long ALN = 16 / EB;                 // elements per 16 bytes of theta
  extern __shared__ __align__(128) unsigned char smem[];
  // [0,64) ring full, [64,128) ring empty (consumers done), [128,132) TMEM base address,
  // [192,448) per-slot retire information (BULK)
  const uint32_t bars = smem_u32(smem);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + 128);
  SlotInfo* sinfo = reinterpret_cast<SlotInfo*>(smem + 192);
  unsigned char* ring0 = smem + P.ring_off;
  unsigned char* meta0 = smem + P.meta_off;
  TH* const theta = reinterpret_cast<TH*>(P.theta);
  const TH* const theta_in = reinterpret_cast<const TH*>(P.theta_in);
  const int total = P.tile_prefix[P.m];
  const int R = P.ring, K = P.K, q = P.q, T = P.T;
  const int my_tiles = (int)blockIdx.x < total ? (total - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  const int ntheta = (K + IN_ROWS - 1) / IN_ROWS;                  // load items per tile
  const int nout = K;                                              // output items per tile
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int r = 0; r < R; ++r) {
      mbar_init(bars + 8 * r, 1);
      mbar_init(bars + 64 + 8 * r, 512);                 // every consumer thread arrives
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"((uint32_t)P.ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer warp
    int comp = 0, pfx_lo = 0, pfx_hi = 0;
    long long cb = 0, ce = 0;
    if (my_tiles > 0) {
      int lo_i = 0, hi_i = P.m;
      while (hi_i - lo_i > 1) {
        const int mid = (lo_i + hi_i) >> 1;
        if (__ldg(P.tile_prefix + mid) <= (int)blockIdx.x) lo_i = mid; else hi_i = mid;
      }
      comp = lo_i;
      pfx_lo = __ldg(P.tile_prefix + comp);
      pfx_hi = __ldg(P.tile_prefix + comp + 1);
      cb = __ldg(P.off + comp);
      ce = __ldg(P.off + comp + 1);
    }
    int gi = 0;              // ring items requested so far
    bool ok = true;
    // BULK: item j is finished by the consumers -> send its results out of the slot.  One bulk
    // group per item (an empty one for load items) so that "all but the newest group have been
    // read" means exactly "the slot about to be refilled is free".
    auto retire = [&](int j) -> bool {
      const int slot = j % R;
      bool fine = mbar_wait_bounded(bars + 64 + 8 * slot, (j / R) & 1, P.status);
      if (!__all_sync(0xffffffffu, fine)) return false;
      if (lane == 0) {
        const SlotInfo si = sinfo[slot];
        if (si.k >= 0 && si.se > si.sb) {
          const uint32_t base = smem_u32(ring0 + (size_t)slot * P.slot_stride);
          const uint32_t skip = (uint32_t)(si.sb - si.e0), n = (uint32_t)(si.se - si.sb);
          const long long at = (long long)si.k * P.ld + si.sb;
          asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(P.omega + at), "r"(base + skip * 4u), "r"(n * 4u) : "memory");
          asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(P.delta + at), "r"(base + (uint32_t)T * 4u + skip * 4u), "r"(n * 4u) : "memory");
          asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(theta + at), "r"(base + (uint32_t)T * 8u + skip * EB), "r"(n * EB) : "memory");
        }
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      }
      __syncwarp();
      return true;
    };
    for (int it = 0; it < my_tiles && ok; ++it) {
      const int w = (int)blockIdx.x + it * (int)gridDim.x;
      if (w >= pfx_hi) {
        while (w >= pfx_hi) {
          ++comp;
          pfx_lo = pfx_hi;
          pfx_hi = __ldg(P.tile_prefix + comp + 1);
        }
        cb = __ldg(P.off + comp);
        ce = __ldg(P.off + comp + 1);
      }
      const long long e0 = (cb & ~(long long)(kAlign - 1)) + (long long)(w - pfx_lo) * T;
      long long run = P.ld - e0;
      if (run > T) run = T;
      const long long lo = cb > e0 ? cb : e0, hi = ce < e0 + T ? ce : e0 + T;
      // tile descriptor + neighbour table into the meta ring (4 entries: the consumers are never
      // more than a ring of items, i.e. at most three tiles, behind)
      unsigned char* meta = meta0 + (size_t)(it & 3) * P.meta_stride;
      TileDesc* d = reinterpret_cast<TileDesc*>(meta);
      int* snb = reinterpret_cast<int*>(meta + sizeof(TileDesc));
      if (d->comp != comp || it < 4) {
        const int32_t* gnb = P.nbr + (size_t)comp * K * q;
        for (int x = lane; x < K * q; x += 32) snb[x] = __ldg(gnb + x);
      }
      __syncwarp();
      if (lane == 0) {
        d->e0 = e0;
        d->lo = lo;
        d->hi = hi;
        d->comp = comp;
      }
      __syncwarp();
      for (int item = 0; item < ntheta + nout && ok; ++item, ++gi) {
        const int slot = gi % R;
        if (BULK) {
          if (gi >= R - 1) ok = retire(gi - (R - 1));       // consumers done with it; its stores go out
          if (!ok) break;
          if (gi >= R && lane == 0)                          // the slot's own stores have read it
            asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
          __syncwarp();
        } else if (gi >= R) {
          bool fine = mbar_wait_bounded(bars + 64 + 8 * slot, ((gi / R) - 1) & 1, P.status);
          ok = __all_sync(0xffffffffu, fine);
          if (!ok) break;
        }
        if (lane == 0) {
          const uint32_t full = bars + 8 * slot;
          const uint32_t dst = smem_u32(ring0 + (size_t)slot * P.slot_stride);
          if (BULK) {
            SlotInfo si;
            si.e0 = e0;
            si.sb = (lo + ALN - 1) & ~(ALN - 1);
            si.se = hi & ~(ALN - 1);
            si.k = item < ntheta ? -1 : item - ntheta;
            si.pad = 0;
            sinfo[slot] = si;
          }
          if (item < ntheta) {
            const int r0 = IN_ROWS * item;
            const int rows = K - r0 < IN_ROWS ? K - r0 : IN_ROWS;
            const uint32_t bytes = (uint32_t)run * EB;
            mbar_arrive_expect_tx(full, (uint32_t)rows * bytes);
            for (int r = 0; r < rows; ++r)
              bulk_load_row(dst + (uint32_t)r * (uint32_t)T * EB, theta_in + (long long)(r0 + r) * P.ld + e0, bytes, full);
          } else {
            const long long at = (long long)(item - ntheta) * P.ld + e0;
            const uint32_t bytes = (uint32_t)run * 4u;
            mbar_arrive_expect_tx(full, 2u * bytes);
            bulk_load_row(dst, P.omega + at, bytes, full);
            bulk_load_row(dst + (uint32_t)T * 4u, P.delta + at, bytes, full);
          }
        }
      }
    }
    if (BULK) {
      for (int j = gi > R - 1 ? gi - (R - 1) : 0; j < gi && ok; ++j) ok = retire(j);
      if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
      __syncwarp();
    }
    if (!ok) {
      for (int j = gi > R ? gi - R : 0; j < gi; ++j)
        mbar_wait_bounded(bars + 8 * (j % R), (j / R) & 1, P.status);
    }
  } else {
    // -------------------------------------------------------------------- consumer warps (16)
    // lanes this warp reaches, and which of the four warps of that lane quarter it is
    // (24 consumer warps were measured slower than 16)
    const int quarter = warp & 3, sub = (warp - 1) >> 2;
    const uint32_t tlane = tmem_base + ((uint32_t)(quarter * 32) << 16);
    const int ngroups = T / 512;                  // element groups of 128 x 4 per row
    int gi = 0;
    bool ok = true;
    for (int it = 0; it < my_tiles && ok; ++it) {
      const unsigned char* meta = meta0 + (size_t)(it & 3) * P.meta_stride;
      const TileDesc* d = reinterpret_cast<const TileDesc*>(meta);
      const int* snb = reinterpret_cast<const int*>(meta + sizeof(TileDesc));
      long long e0 = 0, lo = 0, hi = 0, sb = 0, se = 0;
      for (int item = 0; item < ntheta + nout && ok; ++item, ++gi) {
        const int slot = gi % R;
        bool fine = mbar_wait_bounded(bars + 8 * slot, (gi / R) & 1, P.status);
        ok = __all_sync(0xffffffffu, fine);
        if (!ok) break;
        if (item == 0) {
          e0 = d->e0; lo = d->lo; hi = d->hi;
          sb = (lo + ALN - 1) & ~(ALN - 1);       // whole 16-byte pieces of theta inside the tile
          se = hi & ~(ALN - 1);
        }
        unsigned char* const sbase = ring0 + (size_t)slot * P.slot_stride;
        if (item < ntheta) {
          // deposit the theta rows of this item into this thread's TMEM cells
          const int r0 = IN_ROWS * item;
          const TH* rows_in = reinterpret_cast<const TH*>(sbase);
          for (int g = sub; g < ngroups; g += 4) {
            const int col = (g * 128 + quarter * 32 + lane) * 4;
#pragma unroll
            for (int r = 0; r < IN_ROWS; ++r)
              if (r0 + r < K)
                TmemCell<TH>::deposit(tlane + (uint32_t)((g * K + r0 + r) * CW), rows_in + (size_t)r * T + col);
          }
          asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        } else {
          const int k = item - ntheta;
          float* row0 = reinterpret_cast<float*>(sbase);
          float* row1 = row0 + T;
          TH* row2 = reinterpret_cast<TH*>(row1 + T);      // BULK: the new theta
          for (int g = sub; g < ngroups; g += 4) {
            const int col = (g * 128 + quarter * 32 + lane) * 4;
            const long long e = e0 + col;
            float a[4], t[4];
            __syncwarp();                          // lanes that left the last group early rejoin
            tmem_gather<TH>(tlane + (uint32_t)(g * K * CW), k, snb + k * q, q, a);
            if (e >= hi || e + 4 <= lo) continue;
            average_divide(a, P.qp1, P.inv_qp1, P.inv_exact);
            const float4 W = *reinterpret_cast<const float4*>(row0 + col);
            const float4 D = *reinterpret_cast<const float4*>(row1 + col);
            float wv[4] = {W.x, W.y, W.z, W.w}, dv[4] = {D.x, D.y, D.z, D.w};
#pragma unroll
            for (int x = 0; x < 4; ++x) bmuf_filter<TH>(a[x], wv[x], dv[x], t[x], P.eta, P.zeta);
            const long long at = (long long)k * P.ld + e;
            if (BULK && e >= sb && e + 4 <= se) {
              *reinterpret_cast<float4*>(row0 + col) = make_float4(wv[0], wv[1], wv[2], wv[3]);
              *reinterpret_cast<float4*>(row1 + col) = make_float4(dv[0], dv[1], dv[2], dv[3]);
              TmemCell<TH>::sts_quad(row2 + col, t);
            } else if (!BULK && e >= lo && e + 4 <= hi) {
              __stcs(reinterpret_cast<float4*>(P.delta + at), make_float4(dv[0], dv[1], dv[2], dv[3]));
              __stcs(reinterpret_cast<float4*>(P.omega + at), make_float4(wv[0], wv[1], wv[2], wv[3]));
              ThetaTraits<TH>::stg_quad(theta + at, t);
            } else {
              for (int x = 0; x < 4; ++x) {
                if (e + x >= lo && e + x < hi) {
                  P.delta[at + x] = dv[x];
                  P.omega[at + x] = wv[x];
                  theta[at + x] = ThetaTraits<TH>::narrow(t[x]);
                }
              }
            }
          }
        }
        if (BULK && item >= ntheta) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_arrive(bars + 64 + 8 * slot);
      }
    }
  }
  // every thread arrives here; only then is the tensor memory given back
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)P.ncols) : "memory");
  }
}

// Self-test of average_divide: runs its correction route (never the power-of-two shortcut) and
// the plain division over all 2^32 bit patterns of the dividend, four consecutive patterns per
// call as in the round kernels, and counts the patterns whose results differ in any bit.
__global__ void __launch_bounds__(256) divide_selftest_kernel(float b, float y, unsigned long long* mismatches,
                                                              unsigned int* first_bad) {
  const unsigned long long nquads = 1ull << 30;
  unsigned int bad = 0, first = 0xFFFFFFFFu;
  for (unsigned long long qd = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; qd < nquads;
       qd += (unsigned long long)gridDim.x * blockDim.x) {
    float a[4], ref[4];
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      a[x] = __uint_as_float((unsigned int)(qd * 4 + x));
      ref[x] = __fdiv_rn(a[x], b);
    }
    average_divide(a, b, y, 0);
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      if (__float_as_uint(a[x]) != __float_as_uint(ref[x])) {
        ++bad;
        const unsigned int pat = (unsigned int)(qd * 4 + x);
        if (pat < first) first = pat;
      }
    }
  }
  if (bad) {
    atomicAdd(mismatches, (unsigned long long)bad);
    atomicMin(first_bad, first);
  }
}

// Self-test of the bounded wait: one warp waits on a barrier that nothing will ever signal.  The
// wait must expire, set the status word and return; nothing here can hang or trap.
__global__ void wait_timeout_selftest_kernel(int32_t* status, int32_t* returned) {
  __shared__ __align__(8) unsigned long long bar_storage;
  const uint32_t bar = smem_u32(&bar_storage);
  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  const bool ok = mbar_wait_bounded(bar, 0, status);
  if (threadIdx.x == 0) *returned = ok ? 1 : 2;
}

// =================================================================================================
// Synthetic local step: theta <- store(theta - lr * (sigma * z)), z from the four 16-bit halves
// of two Philox words (Irwin-Hall, n = 4), keyed by (seed, step, worker, global element pair).
// =================================================================================================
__device__ __forceinline__ float noise_from_words(uint32_t a, uint32_t b) {
  const int sum = (int)((a & 0xFFFFu) + (a >> 16) + (b & 0xFFFFu) + (b >> 16));
  return __fmul_rn((float)(sum - 131070), 0x1.bb67aep-16f);   // 1 / sqrt((2^32 - 1) / 3)
}

template <typename TH>
__global__ void __launch_bounds__(256) perturb_kernel(TH* theta, int K, long long N, long long ld,
                                                      uint32_t key0, uint32_t key1, uint32_t step0,
                                                      int nsteps, float lr, float sigma,
                                                      long long elem_base) {
  constexpr int VEC = ThetaTraits<TH>::VEC;
  const long long nvec = (N + VEC - 1) / VEC;
  const int k = blockIdx.y;                 // one grid row per worker
  for (long long iv = (long long)blockIdx.x * blockDim.x + threadIdx.x; iv < nvec;
       iv += (long long)gridDim.x * blockDim.x) {
    const long long e = iv * VEC;
    TH* row = theta + (long long)k * ld + e;
    const int n = N - e < VEC ? (int)(N - e) : VEC;
    float v[VEC];
    if (n == VEC) {
      ThetaTraits<TH>::lds(row, v);   // a 16-byte load (rows and vectors are 16-byte aligned)
    } else {
      for (int x = 0; x < n; ++x) v[x] = ThetaTraits<TH>::widen(row[x]);
    }
    for (int s = 0; s < nsteps; ++s) {
      unsigned long long have = ~0ull;
      Philox4 r = {0, 0, 0, 0};
#pragma unroll
      for (int x = 0; x < VEC; ++x) {
        if (x < n) {
          const unsigned long long ge = (unsigned long long)(elem_base + e + x);
          const unsigned long long pair = ge >> 1;
          if (pair != have) {
            Philox4 ctr = {(uint32_t)pair, (uint32_t)(pair >> 32), (uint32_t)k, step0 + (uint32_t)s};
            r = philox4x32_10(ctr, key0, key1);
            have = pair;
          }
          const float z = (ge & 1) ? noise_from_words(r.z, r.w) : noise_from_words(r.x, r.y);
          const float upd = __fmul_rn(lr, __fmul_rn(sigma, z));
          v[x] = ThetaTraits<TH>::round_store(__fsub_rn(v[x], upd));
        }
      }
    }
    if (n == VEC) {
      ThetaTraits<TH>::stg(row, v);
    } else {
      for (int x = 0; x < n; ++x) row[x] = ThetaTraits<TH>::narrow(v[x]);
    }
  }
}

// =================================================================================================
// Local step with the optimiser of the paper's experiments (Section 3.2): Adagrad with the
// gradient norm of a group of components clipped.  Three kernels: per-(worker, block) partial sums
// of squares in double over the clip ranges, a fixed-order final sum that turns them into one
// scale factor per worker (deterministic: no atomics), and the element-wise update.
// =================================================================================================
constexpr int kMaxClipRanges = 16;
constexpr int kNormBlocks = 128;    // partial sums per worker

struct ClipRanges {
  int n;
  long long begin[kMaxClipRanges], end[kMaxClipRanges];
};

__global__ void __launch_bounds__(256) sumsq_partial_kernel(const float* grad, long long ld,
                                                            ClipRanges R, double* partial) {
  const int k = blockIdx.y;
  const float* row = grad + (long long)k * ld;
  // four independent partial sums per thread keep four loads in flight; the order of the
  // additions is fixed by the launch shape, so the result is reproducible
  double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (int r = 0; r < R.n; ++r) {
    long long e = R.begin[r] + (long long)blockIdx.x * blockDim.x + threadIdx.x;
    for (; e + 3 * stride < R.end[r]; e += 4 * stride) {
      const double g0 = (double)row[e], g1 = (double)row[e + stride];
      const double g2 = (double)row[e + 2 * stride], g3 = (double)row[e + 3 * stride];
      a0 += g0 * g0; a1 += g1 * g1; a2 += g2 * g2; a3 += g3 * g3;
    }
    for (; e < R.end[r]; e += stride) {
      const double g = (double)row[e];
      a0 += g * g;
    }
  }
  double acc = (a0 + a1) + (a2 + a3);
  __shared__ double warp_sum[8];
  for (int d = 16; d > 0; d >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, d);
  if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int w = 0; w < 8; ++w) s += warp_sum[w];
    partial[(size_t)k * gridDim.x + blockIdx.x] = s;
  }
}

__global__ void clip_scale_kernel(const double* partial, int K, int nblk, float clip_norm,
                                  float* scale) {
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= K) return;
  double s = 0.0;
  for (int b = 0; b < nblk; ++b) s += partial[(size_t)k * nblk + b];
  const float norm = (float)sqrt(s);
  scale[k] = __fdiv_rn(clip_norm, norm > clip_norm ? norm : clip_norm);
}

// The element-wise Adagrad update as a streaming kernel: 20 bytes per replica-parameter (fp32
// theta) and nothing else, so it is built like the fused round: persistent CTAs, a producer warp
// that has the copy engine fetch [gradient | accumulator | theta] chunks of one worker's row into a
// ring of shared-memory slots, 16 consumer warps that update accumulator and theta inside the slot,
// and bulk stores that send the two rows back.  Chunks are T consecutive elements of one row;
// consecutive CTAs take consecutive chunks.  Rows are read up to the padded stride (a multiple of
// 16 bytes); stores cover whole 16-byte pieces below N, the few elements after the last whole
// piece are stored by the thread that computed them, and the padding is never written.
struct AdagradParams {
  void* theta;
  const float* grad;
  float* accum;
  const float* scale;      // [K] clip factor per worker, or NULL
  int32_t* status;
  long long N, ld;
  int K, T, ring, chunks_per_row, groups;   // groups: consumer thread groups (1, 2 or 4)
  uint32_t ring_off, slot_stride;
  float lr, eps;
  ClipRanges R;
};

// What producer and consumers share about the chunk in a slot: it starts at element e0 of worker
// k's row and ends before hi (<= N); whole 16-byte pieces end at se; `where` places it relative
// to the clip ranges (0 outside all, 1 inside one, 2 mixed) and sc is the worker's clip factor.
struct AdagradSlot { long long e0, hi, se; int k; int where; float sc; int pad; };

template <typename TH>
__global__ void __launch_bounds__(544, 1) adagrad_stream_kernel(const AdagradParams P) {
  constexpr int EB = (int)sizeof(TH);
  constexpr long long ALN = 16 / EB;                 // elements per 16 bytes of theta
  extern __shared__ __align__(128) unsigned char smem[];
  // [0,64) slot full, [64,128) slot done (consumers), [128,512) per-slot chunk descriptors
  const uint32_t bars = smem_u32(smem);
  AdagradSlot* sinfo = reinterpret_cast<AdagradSlot*>(smem + 128);
  unsigned char* ring0 = smem + P.ring_off;
  TH* const theta = reinterpret_cast<TH*>(P.theta);
  const int R = P.ring, T = P.T;
  const long long total = (long long)P.chunks_per_row * P.K;
  const int my_chunks = (long long)blockIdx.x < total
                            ? (int)((total - (long long)blockIdx.x + (long long)gridDim.x - 1) / (long long)gridDim.x)
                            : 0;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int r = 0; r < R; ++r) {
      mbar_init(bars + 8 * r, 1);
      mbar_init(bars + 64 + 8 * r, 512 / P.groups);      // every thread of one consumer group arrives
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  if (warp == 0) {
    // ------------------------------------------------------------------ producer warp
    bool ok = true;
    // chunk j is finished by the consumers -> send accumulator and theta out of the slot.  One
    // bulk group per chunk, so that "all but the newest group have been read" means exactly
    // "the slot about to be refilled is free".
    auto retire = [&](int j) -> bool {
      const int slot = j % R;
      bool fine = mbar_wait_bounded(bars + 64 + 8 * slot, (j / R) & 1, P.status);
      if (!__all_sync(0xffffffffu, fine)) return false;
      if (lane == 0) {
        const AdagradSlot si = sinfo[slot];
        if (si.se > si.e0) {
          const uint32_t base = smem_u32(ring0 + (size_t)slot * P.slot_stride);
          const uint32_t n = (uint32_t)(si.se - si.e0);
          const long long at = (long long)si.k * P.ld + si.e0;
          asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(P.accum + at), "r"(base + (uint32_t)T * 4u), "r"(n * 4u) : "memory");
          asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(theta + at), "r"(base + (uint32_t)T * 8u), "r"(n * EB) : "memory");
        }
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      }
      __syncwarp();
      return true;
    };
    // this CTA's chunks are w = blockIdx.x + it * gridDim.x: keep (row, chunk in row) incrementally
    int k = (int)(blockIdx.x / (unsigned)P.chunks_per_row);
    int cin = (int)(blockIdx.x % (unsigned)P.chunks_per_row);
    const int dk = (int)(gridDim.x / (unsigned)P.chunks_per_row), dc = (int)(gridDim.x % (unsigned)P.chunks_per_row);
    float sc = (P.scale && lane == 0 && my_chunks > 0) ? __ldg(P.scale + k) : 1.0f;
    int it = 0;
    for (; it < my_chunks && ok; ++it) {
      const long long e0 = (long long)cin * T;
      long long run = P.ld - e0;                         // a row ends at ld: never read past it
      if (run > T) run = T;
      const long long hi = e0 + T < P.N ? e0 + T : P.N;
      const int slot = it % R;
      if (it >= R - 1) ok = retire(it - (R - 1));        // consumers done with it; its stores go out
      if (!ok) break;
      if (it >= R && lane == 0)                          // the slot's own stores have read it
        asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
      __syncwarp();
      if (lane == 0) {
        AdagradSlot si;
        si.e0 = e0; si.hi = hi; si.se = hi & ~(ALN - 1); si.k = k; si.where = 0; si.sc = sc; si.pad = 0;
        if (P.scale) {
          for (int r = 0; r < P.R.n; ++r) {
            if (e0 >= P.R.begin[r] && hi <= P.R.end[r]) si.where = 1;
            else if (e0 < P.R.end[r] && hi > P.R.begin[r] && si.where == 0) si.where = 2;
          }
        }
        sinfo[slot] = si;
        const uint32_t full = bars + 8 * slot;
        const uint32_t dst = smem_u32(ring0 + (size_t)slot * P.slot_stride);
        const long long at = (long long)k * P.ld + e0;
        mbar_arrive_expect_tx(full, (uint32_t)run * (8u + EB));
        bulk_load_row(dst, P.grad + at, (uint32_t)run * 4u, full);
        bulk_load_row(dst + (uint32_t)T * 4u, P.accum + at, (uint32_t)run * 4u, full);
        bulk_load_row(dst + (uint32_t)T * 8u, theta + at, (uint32_t)run * EB, full);
      }
      // next chunk of this CTA
      const int k_before = k;
      k += dk; cin += dc;
      if (cin >= P.chunks_per_row) { cin -= P.chunks_per_row; ++k; }
      if (P.scale && lane == 0 && k != k_before && it + 1 < my_chunks) sc = __ldg(P.scale + k);
    }
    for (int j = it > R - 1 ? it - (R - 1) : 0; j < it && ok; ++j) ok = retire(j);
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    __syncwarp();
    if (!ok) {
      // leave only after the copies already requested into this CTA's shared memory have landed
      for (int j = it > R ? it - R : 0; j < it; ++j)
        mbar_wait_bounded(bars + 8 * (j % R), (j / R) & 1, P.status);
    }
    return;
  }

  // -------------------------------------------------------------------- consumer warps (16)
  // The consumer threads form `groups` groups that take chunks in turn, so that several chunks
  // are being updated at once: one chunk's chain of loads, square root, divide and stores is
  // long, and a single group would make the ring wait for it.
  const int gsize = 512 / P.groups;
  const int grp = (threadIdx.x - 32) / gsize, c = (threadIdx.x - 32) - grp * gsize;
  for (int it = grp; it < my_chunks; it += P.groups) {
    const int slot = it % R;
    if (!mbar_wait_bounded(bars + 8 * slot, (it / R) & 1, P.status)) return;
    const AdagradSlot si = sinfo[slot];
    const long long e0 = si.e0, hi = si.hi, se = si.se;
    const int where = si.where;
    const float sc = si.sc;
    float* sg = reinterpret_cast<float*>(ring0 + (size_t)slot * P.slot_stride);
    float* sa = sg + T;
    TH* sth = reinterpret_cast<TH*>(sa + T);
#pragma unroll 2
    for (int col = c * 4; col < T; col += gsize * 4) {
      const long long e = e0 + col;
      if (e >= hi) break;
      const float4 gv = *reinterpret_cast<const float4*>(sg + col);
      const float4 av = *reinterpret_cast<const float4*>(sa + col);
      float g[4] = {gv.x, gv.y, gv.z, gv.w}, a[4] = {av.x, av.y, av.z, av.w}, th[4];
      ThetaTraits<TH>::lds_quad(sth + col, th);
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        bool inside = where == 1;
        if (where == 2)
          for (int r = 0; r < P.R.n; ++r) inside = inside || (e + x >= P.R.begin[r] && e + x < P.R.end[r]);
        float gx = g[x];
        if (inside) gx = __fmul_rn(gx, sc);
        a[x] = __fadd_rn(a[x], __fmul_rn(gx, gx));
        const float denom = __fadd_rn(__fsqrt_rn(a[x]), P.eps);
        th[x] = __fsub_rn(th[x], __fdiv_rn(__fmul_rn(P.lr, gx), denom));
      }
      if (e + 4 <= se) {
        *reinterpret_cast<float4*>(sa + col) = make_float4(a[0], a[1], a[2], a[3]);
        TmemCell<TH>::sts_quad(sth + col, th);
      } else {
        // after the last whole 16-byte piece of the row: only the elements below N
        const long long at = (long long)si.k * P.ld + e;
        for (int x = 0; x < 4; ++x) {
          if (e + x < hi) {
            P.accum[at + x] = a[x];
            theta[at + x] = ThetaTraits<TH>::narrow(th[x]);
          }
        }
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    mbar_arrive(bars + 64 + 8 * slot);
  }
}

// =================================================================================================
// Initialisation line of Algorithm 1 and its return line.
// =================================================================================================
template <typename TH>
__global__ void __launch_bounds__(256) init_kernel(const TH* theta0, TH* theta, float* omega,
                                                   float* delta, int K, long long N, long long ld) {
  constexpr int VEC = ThetaTraits<TH>::VEC;
  const long long nvec = (N + VEC - 1) / VEC;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < nvec;
       i += (long long)gridDim.x * blockDim.x) {
    const long long e = i * VEC;
    if (e + VEC <= N) {
      const uint4 raw = *reinterpret_cast<const uint4*>(theta0 + e);   // 16 bytes of theta_0
      float f[VEC];
      ThetaTraits<TH>::lds(theta0 + e, f);
      const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int k = 0; k < K; ++k) {
        const long long at = (long long)k * ld + e;
        __stcs(reinterpret_cast<uint4*>(theta + at), raw);
#pragma unroll
        for (int h = 0; h < VEC / 4; ++h) {
          __stcs(reinterpret_cast<float4*>(omega + at) + h,
                 make_float4(f[4 * h], f[4 * h + 1], f[4 * h + 2], f[4 * h + 3]));
          __stcs(reinterpret_cast<float4*>(delta + at) + h, zero);
        }
      }
    } else {
      for (long long x = e; x < N; ++x) {
        const TH v = theta0[x];
        for (int k = 0; k < K; ++k) {
          const long long at = (long long)k * ld + x;
          theta[at] = v;
          omega[at] = ThetaTraits<TH>::widen(v);
          delta[at] = 0.0f;
        }
      }
    }
  }
}

template <typename TH>
__global__ void __launch_bounds__(256) final_average_kernel(const TH* theta, TH* out, int K,
                                                            long long N, long long ld) {
  constexpr int VEC = ThetaTraits<TH>::VEC;
  const float fk = (float)K;
  const long long nvec = (N + VEC - 1) / VEC;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < nvec;
       i += (long long)gridDim.x * blockDim.x) {
    const long long e = i * VEC;
    if (e + VEC <= N) {
      float s[VEC], t[VEC];
      ThetaTraits<TH>::lds(theta + e, s);
      for (int k = 1; k < K; ++k) {                  // k = 0, 1, ..., K-1 in that order
        ThetaTraits<TH>::lds(theta + (long long)k * ld + e, t);
#pragma unroll
        for (int x = 0; x < VEC; ++x) s[x] = __fadd_rn(s[x], t[x]);
      }
#pragma unroll
      for (int x = 0; x < VEC; ++x) s[x] = __fdiv_rn(s[x], fk);
      ThetaTraits<TH>::stg(out + e, s);
    } else {
      for (long long x = e; x < N; ++x) {
        float s = ThetaTraits<TH>::widen(theta[x]);
        for (int k = 1; k < K; ++k)
          s = __fadd_rn(s, ThetaTraits<TH>::widen(theta[(long long)k * ld + x]));
        out[x] = ThetaTraits<TH>::narrow(__fdiv_rn(s, fk));
      }
    }
  }
}

// =================================================================================================
// One worker per GPU ("peer" form): this GPU holds worker `rank`'s theta (two buffers, read one /
// write the other), omega and Delta; the other workers' theta buffers are peer-mapped pointers.
// For every participating component the worker's q neighbours are drawn exactly as in the
// resident form, and the fused kernel pulls their slices straight from peer memory with
// non-multicast bulk copies into the same shared-memory stage as its own theta, omega and Delta
// slices, averages (own first, then draw order), filters, and writes omega and Delta in place and
// the new theta into the OTHER buffer: peers that are still reading this worker's current buffer
// never see a half-updated replica.  Components that do not take part are copied through to the
// other buffer.  Every row of a stage passes through once, so stages are simply pipelined.
// =================================================================================================
struct PeerPlanParams {
  int K, m, p, q, comp_base, rank, use_mask;
  uint64_t seed, round;
  const int32_t* periods;
  const uint8_t* mask;
  int32_t* nbr;    // [m][q] neighbours of worker `rank`
  uint8_t* due;    // [m]
};

__global__ void __launch_bounds__(256) peer_plan_kernel(PeerPlanParams P) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= P.m) return;
  P.due[i] = P.use_mask ? (P.mask[i] != 0) : (P.round % (uint64_t)P.periods[i] == 0);
  if (P.q == 0) return;
  int32_t a[kMaxCand];
  const int c = ring_candidates(P.rank, P.K, P.p, a);
  Philox4 r = {0, 0, 0, 0};
  for (int j = 0; j < P.q && j < c; ++j) {
    if ((j & 3) == 0) {
      Philox4 ctr = {(uint32_t)P.round, (uint32_t)(P.round >> 32), (uint32_t)(P.comp_base + i),
                     (uint32_t)P.rank | ((uint32_t)(j >> 2) << 16)};
      r = philox4x32_10(ctr, (uint32_t)P.seed, (uint32_t)(P.seed >> 32) ^ kTagSampler);
    }
    const uint32_t u = (j & 3) == 0 ? r.x : (j & 3) == 1 ? r.y : (j & 3) == 2 ? r.z : r.w;
    const int t = j + (int)__umulhi(u, (uint32_t)(c - j));
    const int32_t tmp = a[j];
    a[j] = a[t];
    a[t] = tmp;
    P.nbr[(size_t)i * P.q + j] = a[j];
  }
}

struct PeerParams {
  const void* const* theta_in;   // device array [K]: worker j's current theta buffer (peers included)
  void* theta_out;               // this worker's other buffer
  float* omega;                  // this worker's, [N]
  float* delta;
  const int64_t* off;            // [m+1]
  const int32_t* tile_prefix;    // [m+1], over ALL components
  const int32_t* nbr;            // [m][q]
  const uint8_t* due;            // [m]
  int32_t* status;
  long long N;                   // columns; rows are read up to N rounded up to 8 (<= ld)
  int rank, m, q, mode;
  float eta, zeta, qp1, inv_qp1;
  int inv_exact;
  int T, stages, ncons;
  uint32_t stage_stride, omega_off, delta_off, desc_off;   // stage: [q+1 theta rows | omega | Delta | desc]
};

template <typename TH>
__global__ void __launch_bounds__(1024, 1) peer_round_kernel(const PeerParams P) {
  constexpr int VEC = 4;
  extern __shared__ __align__(128) unsigned char smem[];
  const uint32_t bars = smem_u32(smem);            // [0,64) full, [64,128) empty
  unsigned char* stage0 = smem + 128;
  const int total = P.tile_prefix[P.m];
  const int S = P.stages;
  const bool bmuf = P.mode == GBMUF_MODE_BMUF;
  const int my_tiles = (int)blockIdx.x < total ? (total - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(bars + 8 * s, 1);
      mbar_init(bars + 64 + 8 * s, P.ncons);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  if (threadIdx.x < 32) {
    // ------------------------------------------------------------------ producer warp
    const int lane = threadIdx.x;
    int comp = 0, pfx_lo = 0, pfx_hi = 0;
    long long cb = 0, ce = 0;
    if (my_tiles > 0) {
      int lo_i = 0, hi_i = P.m;
      while (hi_i - lo_i > 1) {
        const int mid = (lo_i + hi_i) >> 1;
        if (__ldg(P.tile_prefix + mid) <= (int)blockIdx.x) lo_i = mid; else hi_i = mid;
      }
      comp = lo_i;
      pfx_lo = __ldg(P.tile_prefix + comp);
      pfx_hi = __ldg(P.tile_prefix + comp + 1);
      cb = __ldg(P.off + comp);
      ce = __ldg(P.off + comp + 1);
    }
    int issued = 0;
    bool ok = true;
    const long long row_end = (P.N + kAlign - 1) & ~(long long)(kAlign - 1);
    for (int it = 0; it < my_tiles; ++it) {
      const int w = (int)blockIdx.x + it * (int)gridDim.x;
      const int s = it % S;
      if (it >= S) {
        ok = mbar_wait_bounded(bars + 64 + 8 * s, ((it / S) - 1) & 1, P.status);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
      }
      if (w >= pfx_hi) {
        while (w >= pfx_hi) {
          ++comp;
          pfx_lo = pfx_hi;
          pfx_hi = __ldg(P.tile_prefix + comp + 1);
        }
        cb = __ldg(P.off + comp);
        ce = __ldg(P.off + comp + 1);
      }
      const long long e0 = (cb & ~(long long)(kAlign - 1)) + (long long)(w - pfx_lo) * P.T;
      long long load_end = (ce + kAlign - 1) & ~(long long)(kAlign - 1);
      if (load_end > e0 + P.T) load_end = e0 + P.T;
      if (load_end > row_end) load_end = row_end;
      const uint32_t nelem = (uint32_t)(load_end - e0);
      const uint32_t bytes_th = nelem * (uint32_t)sizeof(TH), bytes_f = nelem * 4u;
      const bool due = __ldg(P.due + comp) != 0;
      unsigned char* st = stage0 + (size_t)s * P.stage_stride;
      if (lane == 0) {
        TileDesc* d = reinterpret_cast<TileDesc*>(st + P.desc_off);
        d->e0 = e0;
        d->lo = cb > e0 ? cb : e0;
        d->hi = ce < e0 + P.T ? ce : e0 + P.T;
        d->comp = due ? comp : -1 - comp;            // negative: copy the component through
      }
      const uint32_t full = bars + 8 * s;
      const int nrows = due ? P.q + 1 : 1;
      if (lane == 0)
        mbar_arrive_expect_tx(full, (uint32_t)nrows * bytes_th + ((due && bmuf) ? 2u * bytes_f : 0u));
      __syncwarp();
      const uint32_t sbase = smem_u32(st);
      for (int r = lane; r < nrows; r += 32) {
        const int src_worker = r == 0 ? P.rank : __ldg(P.nbr + (size_t)comp * P.q + (r - 1));
        const TH* row = static_cast<const TH*>(P.theta_in[src_worker]);   // own or a peer's memory
        bulk_load_row(sbase + (uint32_t)r * (uint32_t)P.T * (uint32_t)sizeof(TH), row + e0, bytes_th, full);
      }
      if (due && bmuf && lane == 0) {
        bulk_load_row(sbase + P.omega_off, P.omega + e0, bytes_f, full);
        bulk_load_row(sbase + P.delta_off, P.delta + e0, bytes_f, full);
      }
      issued = it + 1;
    }
    if (!ok) {
      for (int it = issued > S ? issued - S : 0; it < issued; ++it)
        mbar_wait_bounded(bars + 8 * (it % S), (it / S) & 1, P.status);
    }
    return;
  }

  // -------------------------------------------------------------------- consumer warps
  const int c = threadIdx.x - 32;
  const int nv = P.T / VEC, q = P.q, T = P.T;
  TH* out = static_cast<TH*>(P.theta_out);
  for (int it = 0; it < my_tiles; ++it) {
    const int s = it % S;
    if (!mbar_wait_bounded(bars + 8 * s, (it / S) & 1, P.status)) return;
    unsigned char* st = stage0 + (size_t)s * P.stage_stride;
    const TH* sth = reinterpret_cast<const TH*>(st);
    const float* som = reinterpret_cast<const float*>(st + P.omega_off);
    const float* sde = reinterpret_cast<const float*>(st + P.delta_off);
    const TileDesc* d = reinterpret_cast<const TileDesc*>(st + P.desc_off);
    const long long e0 = d->e0, lo = d->lo, hi = d->hi;
    const bool due = d->comp >= 0;
    for (int v = c; v < nv; v += P.ncons) {
      const int col = v * VEC;
      const long long e = e0 + col;
      if (e >= hi || e + VEC <= lo) continue;
      const bool whole = e >= lo && e + VEC <= hi;
      float a[VEC], t[VEC];
      ThetaTraits<TH>::lds_quad(sth + col, a);
      if (!due) {                                         // not this round: carry theta over
        if (whole) {
          ThetaTraits<TH>::stg_quad(out + e, a);
        } else {
          for (int x = 0; x < VEC; ++x)
            if (e + x >= lo && e + x < hi) out[e + x] = ThetaTraits<TH>::narrow(a[x]);
        }
        continue;
      }
      for (int j = 1; j <= q; ++j) {                      // neighbours in draw order
        ThetaTraits<TH>::lds_quad(sth + (size_t)j * T + col, t);
#pragma unroll
        for (int x = 0; x < VEC; ++x) a[x] = __fadd_rn(a[x], t[x]);
      }
      average_divide(a, P.qp1, P.inv_qp1, P.inv_exact);
      if (!bmuf) {
        if (whole) {
          ThetaTraits<TH>::stg_quad(out + e, a);
        } else {
          for (int x = 0; x < VEC; ++x)
            if (e + x >= lo && e + x < hi) out[e + x] = ThetaTraits<TH>::narrow(a[x]);
        }
        continue;
      }
      const float4 W = *reinterpret_cast<const float4*>(som + col);
      const float4 D = *reinterpret_cast<const float4*>(sde + col);
      float wv[VEC] = {W.x, W.y, W.z, W.w}, dv[VEC] = {D.x, D.y, D.z, D.w};
#pragma unroll
      for (int x = 0; x < VEC; ++x) bmuf_filter<TH>(a[x], wv[x], dv[x], t[x], P.eta, P.zeta);
      if (whole) {
        __stcs(reinterpret_cast<float4*>(P.delta + e), make_float4(dv[0], dv[1], dv[2], dv[3]));
        __stcs(reinterpret_cast<float4*>(P.omega + e), make_float4(wv[0], wv[1], wv[2], wv[3]));
        ThetaTraits<TH>::stg_quad(out + e, t);
      } else {
        for (int x = 0; x < VEC; ++x) {
          if (e + x >= lo && e + x < hi) {
            P.delta[e + x] = dv[x];
            P.omega[e + x] = wv[x];
            out[e + x] = ThetaTraits<TH>::narrow(t[x]);
          }
        }
      }
    }
    mbar_arrive(bars + 64 + 8 * s);
  }
}

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
};

int host_candidates(int K, int p) {
  long long c = 2LL * p;
  if (c > K - 1) c = K - 1;
  return (int)c;
}

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

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Tensor map for boxes of K rows x BW columns over the [K][ld] theta array.
gbmuf_status build_tensor_maps(gbmuf_ctx* ctx, const Launch& L) {
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
  const long long cap = ctx->max_smem < ctx->smem_per_sm - 1024 ? ctx->max_smem : ctx->smem_per_sm - 1024;
  // Variant: flags bit 3 forces the shared-memory theta tile, bit 1 forces the tensor-memory tile
  // (bit 2: with bulk stores); with neither, the tensor-memory tile with bulk stores is used
  // wherever it applies (gossip-BMUF, 4 <= K <= 128) -- it is the faster one.
  const int cw = esz == 4 ? 4 : 2;                       // TMEM columns per group of 4 elements
  const bool tmem_ok = bmuf && K >= 4 && K <= 128;
  // (automatic choice only when the caller has not asked for anything specific to the
  // shared-memory tile: consumer threads, theta stages, or a tile width it cannot have)
  const bool auto_tmem = !(t.flags & 8) && tmem_ok && t.ncons == 0 && t.stages == 0 &&
                         (t.T == 0 || (t.T % 512 == 0 && (t.T / 512) * K * cw <= 512));
  const bool want_tmem = (t.flags & 2) || auto_tmem;
  if ((t.flags & 2) && !tmem_ok)
    return fail(ctx, GBMUF_ERR_UNSUPPORTED, "the tensor-memory variant needs gossip-BMUF mode and 4 <= K <= 128");
  if (want_tmem) {
    const bool bulk = (t.flags & 2) ? (t.flags & 4) != 0 : true;
    const bool forced = (t.flags & 2) != 0;
    // theta tile in tensor memory: K * (T/512) * cw <= 512 columns; T a multiple of 512
    // default width: measured best with 16 replicas (fp32: 3584 x 4 slots; bf16: 3072 x 6 slots)
    int T = t.T ? t.T : (esz == 4 ? 3584 : 3072);
    while (!t.T && T > 512 && (T / 512) * K * cw > 512) T -= 512;
    bool fits = T >= 512 && T % 512 == 0 && (T / 512) * K * cw <= 512;
    if (!fits && (forced || t.T))
      return fail(ctx, GBMUF_ERR_INVALID_ARG, "tensor-memory variant: tile_elems must be a multiple of 512 whose K rows fit 512 columns of tensor memory");
    if (fits) {
      L.T = T; L.BW = 256; L.stages = 1;
      L.ncons = 512;
      L.flags = (t.flags & 1) | 2 | (bulk ? 4 : 0);
      L.meta_off = 512;
      L.meta_stride = (uint32_t)(((long long)sizeof(TileDesc) + (long long)K * q * 4 + 127) / 128 * 128);
      L.ring_off = L.meta_off + 4 * L.meta_stride;
      L.slot_stride = (uint32_t)((bulk ? 8 + esz : 8) * T);
      // ring items per tile; the 4-entry descriptor ring needs the producer to stay within three
      // tiles of the consumers, i.e. a ring no deeper than three tiles' worth of items
      const int in_rows = 8 / esz;
      const int per_tile = (K + in_rows - 1) / in_rows + K;
      const int ring_cap = 3 * per_tile < kMaxRing ? 3 * per_tile : kMaxRing;
      // Ring depth: 4 slots of the default width measured best (3 starve the pipeline, 5 and more
      // put too much in flight; even counts did better than odd ones); narrower slots: more of them.
      int R = t.ring ? t.ring : (bulk ? 4 : 3);
      while (!t.ring && R > 2 && (long long)L.ring_off + (long long)R * L.slot_stride > cap) --R;
      while (!t.ring && bulk && R + 2 <= ring_cap && (long long)R * L.slot_stride < 160 * 1024 &&
             (long long)L.ring_off + (long long)(R + 2) * L.slot_stride <= cap) R += 2;
      if (!t.ring && R > ring_cap) R = ring_cap;
      const bool ring_fits = (long long)L.ring_off + (long long)R * L.slot_stride <= cap && R >= 2 && R <= ring_cap;
      if (!ring_fits && (forced || t.ring))
        return fail(ctx, GBMUF_ERR_UNSUPPORTED, "tensor-memory variant: the ring does not fit shared memory (or is deeper than three tiles)");
      if (ring_fits) {
        L.ring = R;
        L.smem = (uint32_t)(L.ring_off + (long long)R * L.slot_stride);
        int cols = 32;
        while (cols < (T / 512) * K * cw) cols <<= 1;
        L.tmem_cols = cols;
        L.stage_stride = 0; L.nbr_off = 0; L.desc_off = 0;
        *out = L;
        return GBMUF_OK;
      }
    }
  }
  L.flags = t.flags & 1;
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
// slot, the device limits and (shared-memory variant) the tensor map of theta.
gbmuf_status launch_round(gbmuf_ctx* ctx, const gbmuf_config& cfg, const Launch& L, void* theta,
                          float* omega, float* delta, long long ld, int m, const int64_t* off,
                          const int32_t* prefix, const int32_t* nbr, int32_t* status,
                          long long total, cudaStream_t st) {
  const int grid = (int)(total < ctx->num_sms ? total : ctx->num_sms);   // one persistent CTA per SM
  SyncParams P;
  fill_sync_params(cfg, L, theta, omega, delta, ld, m, off, prefix, nbr, status, &P);
  cudaError_t e;
  if (L.tmem_cols > 0) {
    TmemParams Q;
    Q.theta_in = theta; Q.theta = theta; Q.omega = omega; Q.delta = delta;
    Q.off = off; Q.tile_prefix = prefix; Q.nbr = nbr; Q.status = status;
    Q.ld = ld; Q.K = cfg.K; Q.m = m; Q.q = cfg.q;
    Q.eta = P.eta; Q.zeta = P.zeta; Q.qp1 = P.qp1; Q.inv_qp1 = P.inv_qp1; Q.inv_exact = P.inv_exact;
    Q.T = L.T; Q.ring = L.ring; Q.ncols = L.tmem_cols;
    Q.ring_off = L.ring_off; Q.meta_off = L.meta_off; Q.meta_stride = L.meta_stride; Q.slot_stride = L.slot_stride;
    const bool bulk = (L.flags & 4) != 0, bf = cfg.theta_dtype != GBMUF_F32;
    void (*kern)(const TmemParams);
    if (bf)
      kern = bulk ? sync_fused_tmem_kernel<__nv_bfloat16, true> : sync_fused_tmem_kernel<__nv_bfloat16, false>;
    else
      kern = bulk ? sync_fused_tmem_kernel<float, true> : sync_fused_tmem_kernel<float, false>;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem);
    if (e != cudaSuccess) return cuda_fail(ctx, "cudaFuncSetAttribute", e);
    kern<<<grid, 544, L.smem, st>>>(Q);
  } else if (cfg.theta_dtype == GBMUF_F32) {
    e = cudaFuncSetAttribute(sync_fused_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem);
    if (e != cudaSuccess) return cuda_fail(ctx, "cudaFuncSetAttribute", e);
    sync_fused_kernel<float><<<grid, 32 + L.ncons, L.smem, st>>>(P, ctx->map_theta);
  } else {
    e = cudaFuncSetAttribute(sync_fused_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem);
    if (e != cudaSuccess) return cuda_fail(ctx, "cudaFuncSetAttribute", e);
    sync_fused_kernel<__nv_bfloat16><<<grid, 32 + L.ncons, L.smem, st>>>(P, ctx->map_theta);
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, "launch of the fused round kernel", e);
  return GBMUF_OK;
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
    return fail(nullptr, GBMUF_ERR_UNSUPPORTED, "more than 256 workers (one staged box holds all K rows)");
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
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(ctx, "cudaDeviceSynchronize", e);
  free_tables(ctx);
  ctx->partitioned = false;
  ctx->m = m;
  ctx->off.assign(offsets, offsets + m + 1);
  if (periods) ctx->periods.assign(periods, periods + m); else ctx->periods.assign(m, 1);
  const size_t nb = (size_t)ctx->cfg.K * m * (ctx->cfg.q > 0 ? ctx->cfg.q : 1) * sizeof(int32_t);
  e = cudaMalloc(&ctx->d_off, (m + 1) * sizeof(int64_t));
  if (e == cudaSuccess) e = cudaMalloc(&ctx->d_periods, m * sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMalloc(&ctx->d_mask, m);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->d_prefix, (m + 1) * sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMalloc(&ctx->d_nbr, nb);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->d_nbr_export, nb);
  if (e == cudaSuccess) e = cudaMemcpy(ctx->d_off, ctx->off.data(), (m + 1) * sizeof(int64_t), cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(ctx->d_periods, ctx->periods.data(), m * sizeof(int32_t), cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemset(ctx->d_mask, 1, m);
  if (e != cudaSuccess) {
    free_tables(ctx);
    return e == cudaErrorMemoryAllocation ? fail(ctx, GBMUF_ERR_ALLOC, "partition tables") : cuda_fail(ctx, "partition upload", e);
  }
  ctx->partitioned = true;
  return GBMUF_OK;
}

gbmuf_status gbmuf_set_tuning(gbmuf_ctx* ctx, int32_t ncons, int32_t tile_elems, int32_t stages,
                              int32_t ring, int32_t flags) {
  if (!ctx) return GBMUF_ERR_INVALID_ARG;
  if (ncons < 0 || ncons > 992 || ncons % 32 != 0 || tile_elems < 0 || tile_elems > (1 << 16) ||
      stages < 0 || stages > kMaxThetaStages || ring < 0 || ring > kMaxRing || ring == 1 || flags < 0 || flags > 15 || ((flags & 4) && !(flags & 2)) || ((flags & 8) && (flags & 2)))
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
  if (stages) *stages = ctx->launch.tmem_cols > 0 ? 0 : ctx->launch.stages;
  return GBMUF_OK;
}

gbmuf_status gbmuf_init(gbmuf_ctx* ctx, const void* theta0, void* stream) {
  if (!ctx) return GBMUF_ERR_INVALID_ARG;
  if (!theta0 || (uintptr_t)theta0 % 16 != 0)
    return fail(ctx, GBMUF_ERR_INVALID_ARG, "theta0 must be a 16-byte aligned device pointer");
  DeviceGuard guard(ctx->cfg.device);
  if (!guard.ok) return fail(ctx, GBMUF_ERR_CUDA, "cudaSetDevice failed");
  const int grid = elementwise_grid(ctx, (ctx->cfg.N + 3) / 4);
  cudaStream_t st = (cudaStream_t)stream;
  if (ctx->cfg.theta_dtype == GBMUF_F32)
    init_kernel<float><<<grid, 256, 0, st>>>((const float*)theta0, (float*)ctx->theta, ctx->omega,
                                             ctx->delta, ctx->cfg.K, ctx->cfg.N, ctx->cfg.ld);
  else
    init_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)theta0,
                                                     (__nv_bfloat16*)ctx->theta, ctx->omega,
                                                     ctx->delta, ctx->cfg.K, ctx->cfg.N, ctx->cfg.ld);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, "launch of the init kernel", e);
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
    e = cudaFuncSetAttribute(adagrad_stream_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem);
    if (e != cudaSuccess) return cuda_fail(ctx, "cudaFuncSetAttribute", e);
    adagrad_stream_kernel<float><<<grid, 544, smem_bytes, st>>>(A);
  } else {
    e = cudaFuncSetAttribute(adagrad_stream_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem);
    if (e != cudaSuccess) return cuda_fail(ctx, "cudaFuncSetAttribute", e);
    adagrad_stream_kernel<__nv_bfloat16><<<grid, 544, smem_bytes, st>>>(A);
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, "launch of the Adagrad local-step kernels", e);
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
    e = cudaMemcpyAsync(ctx->d_mask, comp_mask, ctx->m, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_fail(ctx, "upload of the component mask", e);
  }
  SetupParams S;
  fill_setup(ctx, round, comp_mask != nullptr, true, ctx->d_nbr, &S);
  const long long items = (long long)ctx->cfg.K * ctx->m;
  round_setup_kernel<<<(int)((items + 255) / 256), 256, 0, st>>>(S);
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, "launch of the round set-up kernel", e);

  return launch_round(ctx, ctx->cfg, L, ctx->theta, ctx->omega, ctx->delta, ctx->cfg.ld, ctx->m, ctx->d_off,
                      ctx->d_prefix, ctx->d_nbr, ctx->d_status, total, st);
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
      if (cudaDeviceSynchronize() != cudaSuccess) rc = GBMUF_ERR_CUDA;
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
  cudaError_t e;
  if (!g_noalloc_ptr[cfg->device]) {
    // once per device, with that device current: ask the runtime where the array lives there
    unsigned char* ptr = nullptr;
    e = cudaGetSymbolAddress((void**)&ptr, g_noalloc_scratch);
    if (e != cudaSuccess || !ptr) return cuda_fail(nullptr, "cudaGetSymbolAddress of the fixed scratch array", e);
    g_noalloc_ptr[cfg->device] = ptr;
  }
  unsigned char* scratch = g_noalloc_ptr[cfg->device];

  // a context on the stack: it owns nothing, it only carries the description to the helpers
  gbmuf_ctx tmp;
  tmp.cfg = *cfg; tmp.theta = theta; tmp.omega = omega; tmp.delta = delta; tmp.m = m; tmp.cand = cand;
  int v = 0;
  cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, cfg->device); tmp.num_sms = v;
  cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, cfg->device); tmp.max_smem = v;
  cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerMultiprocessor, cfg->device); tmp.smem_per_sm = v;
  gbmuf_status st = plan_launch(&tmp, tmp.tuning, &tmp.launch);
  if (st == GBMUF_OK) st = build_tensor_maps(&tmp, tmp.launch);
  if (st != GBMUF_OK) { g_create_error = tmp.err; return st; }
  const Launch& L = tmp.launch;

  uint8_t flags[kNoAllocMaxM];
  long long total = 0;
  for (int i = 0; i < m; ++i) {
    flags[i] = comp_mask ? (comp_mask[i] != 0) : 1;
    if (!flags[i]) continue;
    const int64_t start = offsets[i] & ~(int64_t)(kAlign - 1);
    total += (offsets[i + 1] - start + L.T - 1) / L.T;
  }
  if (total > 0x3fffffffLL) return fail(nullptr, GBMUF_ERR_UNSUPPORTED, "more than 2^30 - 1 tiles");
  cudaStream_t cs = (cudaStream_t)stream;
  int32_t* d_status = reinterpret_cast<int32_t*>(scratch + kNaStatusOff);
  // the array keeps whatever the previous call left: the status word must start at zero, the
  // other tables are rewritten in full below for the sizes of this call
  e = cudaMemsetAsync(d_status, 0, sizeof(int32_t), cs);
  if (e == cudaSuccess && total > 0)
    e = cudaMemcpyAsync(scratch + kNaOffsetsOff, offsets, (size_t)(m + 1) * sizeof(int64_t), cudaMemcpyHostToDevice, cs);
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
    const long long items = (long long)cfg->K * m;
    round_setup_kernel<<<(int)((items + 255) / 256), 256, 0, cs>>>(S);
    e = cudaGetLastError();
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
// gbmuf_sync_round_host: one round over replicas that live in HOST memory.
// -------------------------------------------------------------------------------------------------
namespace {

struct HostSet {               // one of the buffer sets column chunks rotate through
  gbmuf_ctx ctx;               // describes the device chunk buffers to the launch helpers
  unsigned char* tables = nullptr;
  cudaStream_t stream = nullptr;
};

void free_host_sets(HostSet* sets, int n) {
  for (int i = 0; i < n; ++i) {
    cudaFree(sets[i].ctx.theta); cudaFree(sets[i].ctx.omega); cudaFree(sets[i].ctx.delta);
    cudaFree(sets[i].tables);
    if (sets[i].stream) cudaStreamDestroy(sets[i].stream);
  }
}

}  // namespace

gbmuf_status gbmuf_sync_round_host(const gbmuf_config* cfg, void* theta, float* omega, float* delta,
                                   int32_t m, const int64_t* offsets, const uint8_t* comp_mask,
                                   uint64_t round, int64_t chunk_cols) {
  if (!cfg) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "cfg must not be NULL");
  if (cfg->K < 1 || cfg->K > 256 || cfg->N < 1 || cfg->ld < cfg->N || cfg->p < 0 || cfg->q < 0 ||
      cfg->comp_base < 0 || (cfg->mode != GBMUF_MODE_BMUF && cfg->mode != GBMUF_MODE_MA) ||
      (cfg->theta_dtype != GBMUF_F32 && cfg->theta_dtype != GBMUF_BF16) ||
      !(cfg->eta == cfg->eta) || !(cfg->zeta == cfg->zeta) || cfg->device < 0)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "configuration out of range (see gbmuf_create)");
  const int cand = host_candidates(cfg->K, cfg->p);
  if (cfg->q > cand || cand > kMaxCand)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "q exceeds the ring neighbours min(2p, K-1), or more than 64 of them");
  if (!theta || !omega || !delta) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "theta, omega and delta must not be NULL");
  if (m < 1 || m > 65536 || !offsets) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "m must be in 1..65536 and offsets not NULL");
  if (offsets[0] != 0 || offsets[m] != cfg->N)
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "offsets[0] must be 0 and offsets[m] must be N");
  for (int i = 0; i < m; ++i)
    if (offsets[i + 1] <= offsets[i]) return fail(nullptr, GBMUF_ERR_INVALID_ARG, "offsets must be strictly increasing");
  if (chunk_cols < 0 || (chunk_cols > 0 && chunk_cols % 32 != 0) || chunk_cols > (1LL << 30))
    return fail(nullptr, GBMUF_ERR_INVALID_ARG, "chunk_cols must be 0 or a multiple of 32 up to 2^30");
  if (chunk_cols == 0) chunk_cols = 1 << 22;
  const long long N = cfg->N;
  if (chunk_cols > (N + 31) / 32 * 32) chunk_cols = (N + 31) / 32 * 32;
  const long long nchunks = (N + chunk_cols - 1) / chunk_cols;
  const int esz = cfg->theta_dtype == GBMUF_F32 ? 4 : 2;
  const int K = cfg->K, q = cfg->q;

  DeviceGuard guard(cfg->device);
  if (!guard.ok) return fail(nullptr, GBMUF_ERR_CUDA, "cudaSetDevice failed");

  constexpr int kSets = 3;
  const int nsets = nchunks < kSets ? (int)nchunks : kSets;
  HostSet sets[kSets];
  for (int i = 0; i < kSets; ++i) { sets[i].ctx.theta = nullptr; sets[i].ctx.omega = nullptr; sets[i].ctx.delta = nullptr; }
  // table block of one set: offsets int64 [m+2] | prefix int32 [m+2] | nbr int32 [K*(m+1)*q] | mask
  const size_t t_off = 0, t_prefix = ((size_t)(m + 2) * 8 + 255) / 256 * 256;
  const size_t t_nbr = t_prefix + ((size_t)(m + 2) * 4 + 255) / 256 * 256;
  const size_t t_mask = t_nbr + ((size_t)K * (m + 1) * (q > 0 ? q : 1) * 4 + 255) / 256 * 256;
  const size_t t_status = t_mask + ((size_t)(m + 1) + 255) / 256 * 256;
  const size_t t_bytes = t_status + 256;
  gbmuf_status st = GBMUF_OK;
  cudaError_t e = cudaSuccess;
  for (int i = 0; i < nsets && st == GBMUF_OK; ++i) {
    gbmuf_ctx& c = sets[i].ctx;
    c.cfg = *cfg; c.cfg.N = chunk_cols; c.cfg.ld = chunk_cols; c.m = m; c.cand = cand;
    c.theta = nullptr; c.omega = nullptr; c.delta = nullptr;
    int v = 0;
    cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, cfg->device); c.num_sms = v;
    cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, cfg->device); c.max_smem = v;
    cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerMultiprocessor, cfg->device); c.smem_per_sm = v;
    e = cudaMalloc(&c.theta, (size_t)K * chunk_cols * esz);
    if (e == cudaSuccess) e = cudaMalloc(&c.omega, (size_t)K * chunk_cols * 4);
    if (e == cudaSuccess) e = cudaMalloc(&c.delta, (size_t)K * chunk_cols * 4);
    if (e == cudaSuccess) e = cudaMalloc(&sets[i].tables, t_bytes);
    if (e == cudaSuccess) e = cudaMemset(sets[i].tables + t_status, 0, 256);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&sets[i].stream, cudaStreamNonBlocking);
    if (e != cudaSuccess) {
      st = e == cudaErrorMemoryAllocation ? fail(nullptr, GBMUF_ERR_ALLOC, "device chunk buffers")
                                          : cuda_fail(nullptr, "set-up of the chunk buffers", e);
      break;
    }
    st = plan_launch(&c, c.tuning, &c.launch);
    if (st == GBMUF_OK) st = build_tensor_maps(&c, c.launch);
    if (st != GBMUF_OK) g_create_error = c.err;
  }
  if (st != GBMUF_OK) { free_host_sets(sets, nsets); return st; }

  // per-chunk host tables must outlive the asynchronous uploads
  std::vector<std::vector<int64_t>> chunk_off((size_t)nchunks);
  std::vector<std::vector<uint8_t>> chunk_mask((size_t)nchunks);
  int first = 0;   // first component that reaches into the current chunk
  for (long long ci = 0; ci < nchunks && st == GBMUF_OK; ++ci) {
    const long long c0 = ci * chunk_cols, c1 = c0 + chunk_cols < N ? c0 + chunk_cols : N;
    while (offsets[first + 1] <= c0) ++first;
    std::vector<int64_t>& lo = chunk_off[(size_t)ci];
    std::vector<uint8_t>& mk = chunk_mask[(size_t)ci];
    lo.push_back(0);
    int i = first;
    long long total = 0;
    HostSet& hs = sets[ci % nsets];
    const int T = hs.ctx.launch.T;
    while (true) {
      const long long b = offsets[i] > c0 ? offsets[i] - c0 : 0;
      const long long en = offsets[i + 1] < c1 ? offsets[i + 1] - c0 : c1 - c0;
      const uint8_t due = comp_mask ? (comp_mask[i] != 0) : 1;
      mk.push_back(due);
      lo.push_back(en);
      if (due) total += (en - (b & ~(long long)(kAlign - 1)) + T - 1) / T;
      if (offsets[i + 1] >= c1) break;
      ++i;
    }
    if (total == 0) continue;                    // nothing in this chunk takes part: leave it alone
    const int mc = (int)mk.size();
    cudaStream_t cs = hs.stream;
    const size_t w_th = (size_t)(c1 - c0) * esz, w_f = (size_t)(c1 - c0) * 4;
    e = cudaMemcpy2DAsync(hs.ctx.theta, (size_t)chunk_cols * esz, (const char*)theta + (size_t)c0 * esz,
                          (size_t)cfg->ld * esz, w_th, K, cudaMemcpyHostToDevice, cs);
    if (e == cudaSuccess && cfg->mode == GBMUF_MODE_BMUF) {
      e = cudaMemcpy2DAsync(hs.ctx.omega, (size_t)chunk_cols * 4, omega + c0, (size_t)cfg->ld * 4, w_f, K,
                            cudaMemcpyHostToDevice, cs);
      if (e == cudaSuccess)
        e = cudaMemcpy2DAsync(hs.ctx.delta, (size_t)chunk_cols * 4, delta + c0, (size_t)cfg->ld * 4, w_f, K,
                              cudaMemcpyHostToDevice, cs);
    }
    if (e == cudaSuccess)
      e = cudaMemcpyAsync(hs.tables + t_off, lo.data(), (size_t)(mc + 1) * 8, cudaMemcpyHostToDevice, cs);
    if (e == cudaSuccess)
      e = cudaMemcpyAsync(hs.tables + t_mask, mk.data(), (size_t)mc, cudaMemcpyHostToDevice, cs);
    if (e != cudaSuccess) { st = cuda_fail(nullptr, "host-to-device copy of a column chunk", e); break; }

    SetupParams S;
    S.K = K; S.m = mc; S.p = cfg->p; S.q = q; S.comp_base = cfg->comp_base + first; S.T = T;
    S.use_mask = 1; S.plan = 1; S.seed = cfg->seed; S.round = round;
    S.off = reinterpret_cast<const int64_t*>(hs.tables + t_off);
    S.periods = nullptr;
    S.mask = hs.tables + t_mask;
    S.nbr = reinterpret_cast<int32_t*>(hs.tables + t_nbr);
    S.tile_prefix = reinterpret_cast<int32_t*>(hs.tables + t_prefix);
    round_setup_kernel<<<(int)(((long long)K * mc + 255) / 256), 256, 0, cs>>>(S);
    e = cudaGetLastError();
    if (e != cudaSuccess) { st = cuda_fail(nullptr, "launch of the round set-up kernel", e); break; }
    const Launch& L = hs.ctx.launch;
    st = launch_round(&hs.ctx, *cfg, L, hs.ctx.theta, hs.ctx.omega, hs.ctx.delta, chunk_cols, mc, S.off,
                      S.tile_prefix, S.nbr, reinterpret_cast<int32_t*>(hs.tables + t_status), total, cs);
    if (st != GBMUF_OK) { g_create_error = hs.ctx.err; break; }
    e = cudaMemcpy2DAsync((char*)theta + (size_t)c0 * esz, (size_t)cfg->ld * esz, hs.ctx.theta,
                          (size_t)chunk_cols * esz, w_th, K, cudaMemcpyDeviceToHost, cs);
    if (e == cudaSuccess && cfg->mode == GBMUF_MODE_BMUF) {
      e = cudaMemcpy2DAsync(omega + c0, (size_t)cfg->ld * 4, hs.ctx.omega, (size_t)chunk_cols * 4, w_f, K,
                            cudaMemcpyDeviceToHost, cs);
      if (e == cudaSuccess)
        e = cudaMemcpy2DAsync(delta + c0, (size_t)cfg->ld * 4, hs.ctx.delta, (size_t)chunk_cols * 4, w_f, K,
                              cudaMemcpyDeviceToHost, cs);
    }
    if (e != cudaSuccess) { st = cuda_fail(nullptr, "device-to-host copy of a column chunk", e); break; }
  }
  int32_t worst = 0;
  for (int i = 0; i < nsets; ++i) {
    e = cudaStreamSynchronize(sets[i].stream);
    int32_t word = 0;
    if (e == cudaSuccess) e = cudaMemcpy(&word, sets[i].tables + t_status, 4, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess && st == GBMUF_OK) st = cuda_fail(nullptr, "waiting for the column chunks", e);
    if (word != 0) worst = word;
  }
  free_host_sets(sets, nsets);
  if (st == GBMUF_OK && worst != 0)
    st = fail(nullptr, GBMUF_ERR_TIMEOUT, "a bounded device-side wait expired; the host arrays are unspecified");
  return st;
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
  e = cudaMalloc(&h->d_status, sizeof(int32_t));
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
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(nullptr, "cudaDeviceSynchronize", e);
  cudaFree(h->tables);
  h->tables = nullptr;
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
  e = cudaMalloc(&h->tables, bytes);
  if (e == cudaSuccess) e = cudaMemcpy(h->tables, h->off.data(), (size_t)(m + 1) * 8, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(h->tables + h->t_prefix, prefix.data(), (size_t)(m + 1) * 4, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(h->tables + h->t_periods, h->periods.data(), (size_t)m * 4, cudaMemcpyHostToDevice);
  if (e != cudaSuccess) {
    cudaFree(h->tables);
    h->tables = nullptr;
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
    e = cudaMemcpyAsync(h->tables + h->t_mask, comp_mask, (size_t)h->m, cudaMemcpyHostToDevice, st);
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
  if (h->cfg.theta_dtype == GBMUF_F32) {
    e = cudaFuncSetAttribute(peer_round_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, h->max_smem);
    if (e == cudaSuccess) peer_round_kernel<float><<<grid, 32 + h->ncons, h->smem, st>>>(P);
  } else {
    e = cudaFuncSetAttribute(peer_round_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, h->max_smem);
    if (e == cudaSuccess) peer_round_kernel<__nv_bfloat16><<<grid, 32 + h->ncons, h->smem, st>>>(P);
  }
  if (e == cudaSuccess) e = cudaGetLastError();
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
      if (cudaDeviceSynchronize() != cudaSuccess) rc = GBMUF_ERR_CUDA;
      cudaFree(h->tables); cudaFree(h->d_status); cudaFree(h->d_theta_in[0]); cudaFree(h->d_theta_in[1]);
    } else {
      rc = GBMUF_ERR_CUDA;
    }
  }
  delete h;
  return rc;
}

}  // extern "C"
