// One worker per GPU: plan and round kernels over peer-mapped buffers.
// Part of libgbmuf (CUDA, sm_100a); included by gbmuf.cu, which is the only translation unit.
#ifndef GBMUF_CSRC_PEER_CUH
#define GBMUF_CSRC_PEER_CUH

namespace {

// =================================================================================================
// One worker per GPU ("peer" form): this GPU holds worker `rank`'s theta (two buffers, read one /
// write the other), omega and Delta; the other workers' theta buffers are peer-mapped pointers.
// For every participating component the worker's q neighbours are drawn exactly as in the
// resident form, and the fused kernel pulls their slices straight from peer memory with
// plain (single-destination) bulk copies into the same shared-memory stage as its own theta, omega and Delta
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

}  // namespace

#endif  // GBMUF_CSRC_PEER_CUH
