// The fused round with the theta tile in shared memory; averaging division and filter.
// Part of libgbmuf (CUDA, sm_100a); included by gbmuf.cu, which is the only translation unit.
#ifndef GBMUF_CSRC_SYNC_FUSED_CUH
#define GBMUF_CSRC_SYNC_FUSED_CUH

namespace {

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
// Exponent test: bit 30 of the result is set iff the biased exponent of s is in [64, 191], i.e.
// iff 2^-63 <= |s| < 2^65 (exponent bits 7 and 6 differ); results of several values may be AND-ed.
__device__ __forceinline__ uint32_t mid_range_bit(float s) {
  const uint32_t u = __float_as_uint(s);
  return u ^ (u + u);
}
constexpr uint32_t kMidRange = 0x40000000u;
__device__ __forceinline__ float divide_corrected(float s, float b, float y) {
  const float q0 = __fmul_rn(s, y);
  const float r = __fmaf_rn(-b, q0, s);
  return __fmaf_rn(r, y, q0);
}
__device__ __forceinline__ void average_divide(float (&a)[4], float b, float y, int y_exact) {
  if (y_exact) {
#pragma unroll
    for (int x = 0; x < 4; ++x) a[x] = __fmul_rn(a[x], y);
  } else if (mid_range_bit(a[0]) & mid_range_bit(a[1]) & mid_range_bit(a[2]) & mid_range_bit(a[3]) & kMidRange) {
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
  grid_launch_dependents();
  constexpr int VEC = 4;   // elements per thread and row: 16 bytes of omega / Delta, 16 or 8 of theta
  extern __shared__ __align__(128) unsigned char smem[];
  const uint32_t bars = smem_u32(smem);
  unsigned char* stage0 = smem + kBarBytes;
  unsigned char* ring0 = smem + P.ring_off;
  const int S = P.stages, R = P.ring;
  const bool bmuf = P.mode == GBMUF_MODE_BMUF;

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
  // everything above overlapped the round set-up kernel; its tables are read from here on
  grid_dependency_wait();
  const int total = P.tile_prefix[P.m];
  const int my_tiles = (int)blockIdx.x < total ? (total - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;

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
      // The neighbour count is a compile-time constant for q = 1 .. 4 (QC; 0 = any q at run
      // time): the gather loop then unrolls completely, which halves the instructions per element.
      auto ma_pass = [&](auto div_tag, auto q_tag) -> bool {
        constexpr int DIV = decltype(div_tag)::value;
        constexpr int QC = decltype(q_tag)::value;
        const int qn = QC ? QC : q;
        uint32_t mid = 0xFFFFFFFFu;                 // bit 30 stays set while every sum is in the middle range
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
#pragma unroll
            for (int j = 0; j < qn; ++j) {
              ThetaTraits<TH>::lds(sth + boxbase + snb[k * qn + j] * BW, t);
#pragma unroll
              for (int x = 0; x < MV; ++x) a[x] = __fadd_rn(a[x], t[x]);
            }
#pragma unroll
            for (int x = 0; x < MV; ++x) {
              if (DIV == 0) {
                a[x] = __fmul_rn(a[x], P.inv_qp1);
              } else if (DIV == 1) {
                mid &= mid_range_bit(a[x]);
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
        return (mid & kMidRange) == 0;
      };
      auto ma_tile = [&](auto q_tag) {
        constexpr int QC = decltype(q_tag)::value;
        constexpr bool pow2 = QC == 1 || QC == 3;          // q + 1 a power of two: exact reciprocal
        if (QC ? pow2 : P.inv_exact != 0) {
          if constexpr (QC == 0 || pow2) ma_pass(std::integral_constant<int, 0>{}, q_tag);
        } else {
          if constexpr (!pow2)
            if (ma_pass(std::integral_constant<int, 1>{}, q_tag)) ma_pass(std::integral_constant<int, 2>{}, q_tag);
        }
      };
      // (bf16 theta only: its consumers are bound by instruction issue and gain 10 %; the fp32
      // round is bound by memory and measured 2-3 % slower with the unrolled gather at q = 2)
      if constexpr (sizeof(TH) == 2) {
        switch (q) {
          case 1: ma_tile(std::integral_constant<int, 1>{}); break;
          case 2: ma_tile(std::integral_constant<int, 2>{}); break;
          case 3: ma_tile(std::integral_constant<int, 3>{}); break;
          case 4: ma_tile(std::integral_constant<int, 4>{}); break;
          default: ma_tile(std::integral_constant<int, 0>{}); break;
        }
      } else {
        ma_tile(std::integral_constant<int, 0>{});
      }
      mbar_arrive(bars + kBarThetaEmpty + 8 * s);
      continue;
    }
    // gossip-BMUF: worker by worker, as the omega / Delta rows arrive in the ring
    for (int k = 0; k < P.K; ++k) {
      const int slot = ring_taken % R;
      if (!mbar_wait_bounded(bars + kBarRingFull + 8 * slot, (ring_taken / R) & 1, P.status)) return;
      const float* som = reinterpret_cast<const float*>(ring0 + (size_t)slot * P.slot_stride);
      const float* sde = som + P.T;
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
        const float4 W = *reinterpret_cast<const float4*>(som + col);
        const float4 D = *reinterpret_cast<const float4*>(sde + col);
        float wv[VEC] = {W.x, W.y, W.z, W.w}, dv[VEC] = {D.x, D.y, D.z, D.w};
#pragma unroll
        for (int x = 0; x < VEC; ++x) bmuf_filter<TH>(a[x], wv[x], dv[x], t[x], P.eta, P.zeta);
        if (e >= lo && e + VEC <= hi) {
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
      mbar_arrive(bars + kBarRingEmpty + 8 * slot);      // this thread is done with the slot
      ++ring_taken;
    }
    mbar_arrive(bars + kBarThetaEmpty + 8 * s);          // this thread is done with the theta stage
  }
}

}  // namespace

#endif  // GBMUF_CSRC_SYNC_FUSED_CUH
