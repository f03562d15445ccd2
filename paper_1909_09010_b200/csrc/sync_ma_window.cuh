// The gossip-MA round for many workers: a window of rows along the ring in shared memory.
// Part of libgbmuf (CUDA, sm_100a); included by gbmuf.cu, which is the only translation unit.
#ifndef GBMUF_CSRC_SYNC_MA_WINDOW_CUH
#define GBMUF_CSRC_SYNC_MA_WINDOW_CUH

namespace {

// =================================================================================================
// gossip-MA (Algorithm 1, the branch theta <- average) with many workers.
//
// The gossip-MA schedule of sync_fused_kernel keeps all K rows of a tile in shared memory, so its
// tiles get narrow as K grows (128 columns at K = 256) and DRAM efficiency with them.  But
// Definition 1's ring means worker k only ever averages with workers within ring distance p, so
// only 2p + 1 rows have to be resident while worker k is computed.  This kernel walks the workers
// k = 0 .. K-1 of a tile and streams the rows through a RING of row slots, each a whole row of T
// elements (6 to 8 KB runs):
//
//   ring index i = 0 .. K-1:  i < p is row K - p + i (the last p rows, which the first workers need
//                             before everything else), i >= p is row i (so the last p rows are
//                             requested twice per tile: p extra row reads out of K);
//   kept rows:                rows 0 .. p-1 live in p slots of their own for the whole tile: the
//                             round is in place, the last workers need them again, and by then
//                             the first workers have overwritten them in global memory.  There
//                             are two such sets, used by alternate tiles, so that the next
//                             tile's kept rows can be fetched while this tile's last workers run.
//
// Worker k needs "virtual indices" v = k + d for its own row (d = 0) and its drawn neighbours
// (signed ring distance |d| <= p): v < 0 is ring index v + p, 0 <= v < p kept row v,
// p <= v < K ring index v, v >= K kept row v - K.  Ring index i is needed last by worker i + p
// (or earlier), so after worker k the consumers release ring index k - p and, after the last
// worker, the rest.  Ring indices run on over the tiles of a CTA (slot = running index mod R), so
// the producer can prefetch the next tile's first rows while the last workers of this one run.
//
// Warp 0 produces (tile lookup, neighbour table of the component as slot codes, one bulk copy
// per row, completion counted on the row's barrier), the other warps consume: each thread owns
// 16 bytes of the row (4 fp32 / 8 bf16 elements), sums own + neighbours out of shared memory in
// draw order, divides, and stores its 16 bytes of the new theta to global memory.  Every wait is
// bounded.
// =================================================================================================
struct MaWinParams {
  void* theta;
  const int64_t* off;
  const int32_t* tile_prefix;
  const int32_t* nbr;      // [m][K][q]
  int32_t* status;
  long long ld;
  int K, m, q, p;
  float qp1, inv_qp1;
  int inv_exact;
  int T, R, ncons;         // elements per row slot, ring slots, consumer threads (T / elements per 16 B)
  uint32_t row_bytes;      // T * element size
  uint32_t meta_off, meta_stride;   // two entries: [TileDesc | codes K*q ints]
  uint32_t kept_off;       // 2 sets of p row slots
  uint32_t ring_off;       // R row slots
};

constexpr int kMaWinMaxRing = 32;
// barrier block: ring full [0, 256), ring empty [256, 512), kept full [512, 528), kept empty [528, 544)
constexpr uint32_t kMwRingFull = 0, kMwRingEmpty = 256, kMwKeptFull = 512, kMwKeptEmpty = 528;
constexpr uint32_t kMwBarBytes = 640;
constexpr int kMwKeptFlag = 0x40000000;   // slot code: a kept row (low bits: which); else a signed ring offset + bias
constexpr int kMwBias = 1 << 20;

template <typename TH>
__global__ void __launch_bounds__(1024, 1) sync_ma_window_kernel(const MaWinParams P) {
  constexpr int MV = ThetaTraits<TH>::VEC;      // elements per 16 bytes
  extern __shared__ __align__(128) unsigned char smem[];
  const uint32_t bars = smem_u32(smem);
  unsigned char* meta0 = smem + P.meta_off;
  unsigned char* kept0 = smem + P.kept_off;
  unsigned char* ring0 = smem + P.ring_off;
  const int K = P.K, q = P.q, p = P.p, R = P.R;
  TH* const theta = reinterpret_cast<TH*>(P.theta);

  if (threadIdx.x == 0) {
    for (int r = 0; r < R; ++r) {
      mbar_init(bars + kMwRingFull + 8 * r, 1);
      mbar_init(bars + kMwRingEmpty + 8 * r, P.ncons);
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(bars + kMwKeptFull + 8 * s, 1);
      mbar_init(bars + kMwKeptEmpty + 8 * s, P.ncons);
    }
    for (int s = 0; s < 2; ++s) reinterpret_cast<TileDesc*>(meta0 + (size_t)s * P.meta_stride)->comp = -1;
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
    long long gi = 0;          // ring rows requested so far, over all tiles of this CTA
    int meta_comp[2] = {-1, -1};
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
      const long long e0 = (cb & ~(long long)(kAlign - 1)) + (long long)(w - pfx_lo) * P.T;
      long long run = P.ld - e0;                         // a row ends at ld: never read past it
      if (run > P.T) run = P.T;
      const uint32_t bytes = (uint32_t)run * (uint32_t)sizeof(TH);
      const int set = it & 1;
      // The meta entry and the kept rows of this tile re-use what tile it - 2 used: wait until
      // the consumers have finished that tile.
      if (it >= 2) {
        bool fine = mbar_wait_bounded(bars + kMwKeptEmpty + 8 * set, ((it >> 1) - 1) & 1, P.status);
        ok = __all_sync(0xffffffffu, fine);
        if (!ok) break;
      }
      unsigned char* meta = meta0 + (size_t)set * P.meta_stride;
      TileDesc* d = reinterpret_cast<TileDesc*>(meta);
      int* codes = reinterpret_cast<int*>(meta + sizeof(TileDesc));
      if (meta_comp[set] != comp) {
        // the drawn neighbours as slot codes: kept row v (or v - K), else the signed ring offset
        // from the worker's own ring index (v - k, or v + p - k for the first read of a last row)
        const int32_t* gnb = P.nbr + (size_t)comp * K * q;
        for (int x = lane; x < K * q; x += 32) {
          const int n = __ldg(gnb + x);
          const int k = x / q;
          int dist = n - k;
          if (dist > p) dist -= K;
          if (dist < -p) dist += K;
          const int v = k + dist;
          int code;
          if (v < 0) code = kMwBias + dist + p;
          else if (v < p) code = kMwKeptFlag | v;
          else if (v < K) code = kMwBias + dist;
          else code = kMwKeptFlag | (v - K);
          codes[x] = code;
        }
        meta_comp[set] = comp;
      }
      __syncwarp();
      if (lane == 0) {
        d->e0 = e0;
        d->lo = cb > e0 ? cb : e0;
        d->hi = ce < e0 + P.T ? ce : e0 + P.T;
        d->comp = comp;
      }
      __syncwarp();
      // kept rows 0 .. p-1 (the barrier's completion also publishes the meta entry above)
      if (lane == 0) {
        const uint32_t full = bars + kMwKeptFull + 8 * set;
        const uint32_t dst = smem_u32(kept0 + (size_t)set * p * P.row_bytes);
        mbar_arrive_expect_tx(full, (uint32_t)p * bytes);       // p = 0: a plain arrival
        for (int r = 0; r < p; ++r)
          bulk_load_row(dst + (uint32_t)r * P.row_bytes, theta + (long long)r * P.ld + e0, bytes, full);
      }
      // ring rows
      for (int i = 0; i < K && ok; ++i, ++gi) {
        const int slot = (int)(gi % R);
        if (gi >= R) {
          bool fine = mbar_wait_bounded(bars + kMwRingEmpty + 8 * slot, (uint32_t)((gi / R) - 1) & 1, P.status);
          ok = __all_sync(0xffffffffu, fine);
          if (!ok) break;
        }
        if (lane == 0) {
          const int row = i < p ? K - p + i : i;
          const uint32_t full = bars + kMwRingFull + 8 * slot;
          mbar_arrive_expect_tx(full, bytes);
          bulk_load_row(smem_u32(ring0 + (size_t)slot * P.row_bytes), theta + (long long)row * P.ld + e0, bytes, full);
        }
      }
    }
    if (!ok) {
      // leave only after the copies already requested into this CTA's shared memory have landed
      for (long long j = gi > R ? gi - R : 0; j < gi; ++j)
        mbar_wait_bounded(bars + kMwRingFull + 8 * (int)(j % R), (uint32_t)(j / R) & 1, P.status);
    }
    return;
  }

  // -------------------------------------------------------------------- consumer warps
  const int c = threadIdx.x - 32;
  const int col = c * MV;                 // this thread's 16 bytes of every row
  long long gi = 0;                       // ring index of worker 0 of the current tile, running
  for (int it = 0; it < my_tiles; ++it) {
    const int set = it & 1;
    if (!mbar_wait_bounded(bars + kMwKeptFull + 8 * set, (uint32_t)(it >> 1) & 1, P.status)) return;
    const unsigned char* meta = meta0 + (size_t)set * P.meta_stride;
    const TileDesc* d = reinterpret_cast<const TileDesc*>(meta);
    const int* codes = reinterpret_cast<const int*>(meta + sizeof(TileDesc));
    const long long e0 = d->e0, lo = d->lo, hi = d->hi;
    const TH* kept = reinterpret_cast<const TH*>(kept0 + (size_t)set * p * P.row_bytes);
    const long long e = e0 + col;
    const bool mine = col < P.T && e < hi && e + MV > lo;
    const bool whole = e >= lo && e + MV <= hi;
    int cur = (int)(gi % R);              // slot of ring index k
    // the newest ring index the next worker needs, min(k + p, K - 1): slot and barrier phase
    int ahead = cur;
    uint32_t ahead_par = (uint32_t)(gi / R) & 1;
    if (!mbar_wait_bounded(bars + kMwRingFull + 8 * ahead, ahead_par, P.status)) return;
    for (int i = 1; i <= p && i < K; ++i) {          // before worker 0: ring indices 0 .. min(p, K-1)
      if (++ahead == R) { ahead = 0; ahead_par ^= 1; }
      if (!mbar_wait_bounded(bars + kMwRingFull + 8 * ahead, ahead_par, P.status)) return;
    }
    for (int k = 0; k < K; ++k) {
      if (k > 0 && k + p < K) {
        // one more ring index becomes needed with every worker
        if (++ahead == R) { ahead = 0; ahead_par ^= 1; }
        if (!mbar_wait_bounded(bars + kMwRingFull + 8 * ahead, ahead_par, P.status)) return;
      }
      if (mine) {
        float a[MV], t[MV];
        const TH* own = k < p ? kept + (size_t)k * P.T : reinterpret_cast<const TH*>(ring0 + (size_t)cur * P.row_bytes);
        ThetaTraits<TH>::lds(own + col, a);
        for (int j = 0; j < q; ++j) {
          const int code = codes[k * q + j];
          const TH* src;
          if (code & kMwKeptFlag) {
            src = kept + (size_t)(code & 0xFFFF) * P.T;
          } else {
            int s = cur + (code - kMwBias);
            if (s < 0) s += R;
            if (s >= R) s -= R;
            src = reinterpret_cast<const TH*>(ring0 + (size_t)s * P.row_bytes);
          }
          ThetaTraits<TH>::lds(src + col, t);
#pragma unroll
          for (int x = 0; x < MV; ++x) a[x] = __fadd_rn(a[x], t[x]);
        }
        if (P.inv_exact) {
#pragma unroll
          for (int x = 0; x < MV; ++x) a[x] = __fmul_rn(a[x], P.inv_qp1);
        } else {
          uint32_t mid = 0xFFFFFFFFu;
#pragma unroll
          for (int x = 0; x < MV; ++x) mid &= mid_range_bit(a[x]);
          if (mid & kMidRange) {
#pragma unroll
            for (int x = 0; x < MV; ++x) a[x] = divide_corrected(a[x], P.qp1, P.inv_qp1);
          } else {
#pragma unroll
            for (int x = 0; x < MV; ++x) a[x] = __fdiv_rn(a[x], P.qp1);
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
      // ring index k - p is not needed by any later worker
      if (k >= p) {
        int s = cur - p;
        if (s < 0) s += R;
        mbar_arrive(bars + kMwRingEmpty + 8 * s);
      }
      if (++cur == R) cur = 0;
    }
    // after the last worker: the ring indices nobody released yet, and the kept rows / meta entry
    for (int i = (K - p > 0 ? K - p : 0); i < K; ++i) mbar_arrive(bars + kMwRingEmpty + 8 * (int)((gi + i) % R));
    mbar_arrive(bars + kMwKeptEmpty + 8 * set);
    gi += K;
  }
}

}  // namespace

#endif  // GBMUF_CSRC_SYNC_MA_WINDOW_CUH
