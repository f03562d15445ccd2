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
  int T, R, ncons;         // elements per row slot, ring slots, consumer threads: T / (V * elements per 16 B)
  uint32_t row_bytes;      // T * element size
  uint32_t meta_off, meta_stride;   // two entries: [TileDesc | codes K*q ints]
  uint32_t kept_off;       // 2 sets of p row slots
  uint32_t ring_off;       // R row slots
};

constexpr int kMaWinMaxRing = 64;
constexpr int kMwUnroll = 4;     // workers per consumer iteration
// barrier block: ring full [0, 512), ring empty [512, 1024), kept full [1024, 1040), kept empty [1040, 1056)
constexpr uint32_t kMwRingFull = 0, kMwRingEmpty = 512, kMwKeptFull = 1024, kMwKeptEmpty = 1040;
constexpr uint32_t kMwBarBytes = 1152;

// 16 bytes from shared memory by 32-bit shared address (the consumers' inner loop works on plain
// 32-bit offsets: 64-bit generic pointers cost several instructions per access)
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
template <typename TH> struct Row16;          // the elements in 16 bytes of a row, widened to fp32
template <> struct Row16<float> {
  static __device__ __forceinline__ void widen(const uint4& v, float (&x)[4]) {
    x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y); x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
  }
};
template <> struct Row16<__nv_bfloat16> {
  static __device__ __forceinline__ void widen(const uint4& v, float (&x)[8]) {
    x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xFFFF0000u);
    x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xFFFF0000u);
    x[4] = __uint_as_float(v.z << 16); x[5] = __uint_as_float(v.z & 0xFFFF0000u);
    x[6] = __uint_as_float(v.w << 16); x[7] = __uint_as_float(v.w & 0xFFFF0000u);
  }
};

template <typename TH, int V>
__global__ void __launch_bounds__(544, 1) sync_ma_window_kernel(const MaWinParams P) {
  grid_launch_dependents();
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
      mbar_init(bars + kMwRingEmpty + 8 * r, P.ncons / 32);   // one arrival per consumer warp
    }
    for (int s = 0; s < 2; ++s) {
      mbar_init(bars + kMwKeptFull + 8 * s, 1);
      mbar_init(bars + kMwKeptEmpty + 8 * s, P.ncons / 32);
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
    // ring rows are requested in one running sequence over all tiles of this CTA; the next one
    // goes to `slot`, whose barriers are in phase `slot_par`.  (Kept incremental: this loop runs
    // once per row and a division in it would cost more than the copy it issues.)
    int slot = 0;
    uint32_t slot_par = 0;
    bool wrapped = false;      // the ring has been filled once: a slot must be released before re-use
    int meta_comp0 = -1, meta_comp1 = -1;   // which component's codes each meta entry holds
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
      if ((set ? meta_comp1 : meta_comp0) != comp) {
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
          // (kept row: its byte offset in the kept set, flagged by bit 0; else the signed byte
          // offset from the worker's own ring slot)
          int code;
          const int rb = (int)P.row_bytes;
          if (v < 0) code = ((dist + p) * rb) * 2;
          else if (v < p) code = (v * rb) * 2 + 1;
          else if (v < K) code = (dist * rb) * 2;
          else code = ((v - K) * rb) * 2 + 1;
          codes[x] = code;
        }
        if (set) meta_comp1 = comp; else meta_comp0 = comp;
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
      const TH* src = theta + (long long)(K - p) * P.ld + e0;      // ring index 0 is row K - p
      for (int i = 0; i < K && ok; ++i) {
        if (i == p) src = theta + (long long)p * P.ld + e0;        // ring index i >= p is row i
        if (wrapped) {
          // the slot's previous occupant was released in the phase before the current one
          bool fine = mbar_wait_bounded(bars + kMwRingEmpty + 8 * slot, slot_par ^ 1, P.status);
          ok = __all_sync(0xffffffffu, fine);
          if (!ok) break;
        }
        if (lane == 0) {
          const uint32_t full = bars + kMwRingFull + 8 * slot;
          mbar_arrive_expect_tx(full, bytes);
          bulk_load_row(smem_u32(ring0 + (size_t)slot * P.row_bytes), src, bytes, full);
        }
        src += P.ld;
        if (++slot == R) { slot = 0; slot_par ^= 1; wrapped = true; }
      }
    }
    if (!ok) {
      // leave only after the copies already requested into this CTA's shared memory have landed:
      // every slot's newest request is in phase slot_par (slots before `slot`) or the one before
      for (int j = 0; j < R; ++j) {
        const bool cur_phase = j < slot;
        if (!cur_phase && !wrapped) continue;                      // never requested
        mbar_wait_bounded(bars + kMwRingFull + 8 * j, cur_phase ? slot_par : slot_par ^ 1, P.status);
      }
    }
    return;
  }

  // -------------------------------------------------------------------- consumer warps
  // A row is 8 KB at most, so a worker takes well under a microsecond: the loop over the workers
  // has to be lean.  A thread owns V pieces of 16 bytes of every row (columns (c + v * ncons) *
  // MV; V = 1 is what is launched: with 2 and 4 pieces and a half or a quarter of the warps the
  // round ran slower, the warps' instruction streams being latency-bound); workers are taken
  // four at a time, stage by stage, so that the shared-memory round trips of one overlap the
  // arithmetic of the others; addresses are 32-bit shared addresses, slot and phase are carried
  // along instead of recomputed, and a warp arrives on a barrier once, through lane 0, after
  // all its lanes have finished reading.
  const int c = threadIdx.x - 32;
  const bool lane0 = (threadIdx.x & 31) == 0;
  const uint32_t rb = P.row_bytes;
  const int ring_bytes = R * (int)rb;
  const uint32_t ring_b = smem_u32(ring0) + (uint32_t)c * 16u;
  const uint32_t vstep = (uint32_t)P.ncons * 16u;          // bytes between a thread's pieces
  int cur = 0;                            // slot of the current worker's ring index, running over tiles
  int cur_off = 0;                        // cur * row bytes
  uint32_t cur_par = 0;                   // and the phase of that slot's barriers
  for (int it = 0; it < my_tiles; ++it) {
    const int set = it & 1;
    if (!mbar_wait_bounded(bars + kMwKeptFull + 8 * set, (uint32_t)(it >> 1) & 1, P.status)) return;
    const unsigned char* meta = meta0 + (size_t)set * P.meta_stride;
    const TileDesc* d = reinterpret_cast<const TileDesc*>(meta);
    const int* codes = reinterpret_cast<const int*>(meta + sizeof(TileDesc));
    const long long e0 = d->e0, lo = d->lo, hi = d->hi;
    const uint32_t kept_b = smem_u32(kept0 + (size_t)set * p * rb) + (uint32_t)c * 16u;
    bool mine[V], whole[V];
    bool any = false;
#pragma unroll
    for (int v = 0; v < V; ++v) {
      const long long e = e0 + (long long)(c + v * P.ncons) * MV;
      mine[v] = e < hi && e + MV > lo;
      whole[v] = e >= lo && e + MV <= hi;
      any |= mine[v];
    }
    TH* gp = theta + e0 + (long long)c * MV;   // this thread's first piece of worker k's row
    // the newest ring index the next worker needs, min(k + p, K - 1): slot and barrier phase
    int ahead = cur;
    uint32_t ahead_par = cur_par;
    if (!mbar_wait_bounded(bars + kMwRingFull + 8 * ahead, ahead_par, P.status)) return;
    for (int i = 1; i <= p && i < K; ++i) {          // before worker 0: ring indices 0 .. min(p, K-1)
      if (++ahead == R) { ahead = 0; ahead_par ^= 1; }
      if (!mbar_wait_bounded(bars + kMwRingFull + 8 * ahead, ahead_par, P.status)) return;
    }
    int ahead_idx = p < K ? p : K - 1;     // the ring index `ahead` stands for
    for (int k = 0; k < K; k += kMwUnroll) {
      const int nu = K - k < kMwUnroll ? K - k : kMwUnroll;
      const int need = k + nu - 1 + p < K - 1 ? k + nu - 1 + p : K - 1;
      while (ahead_idx < need) {            // ring indices that become needed with these workers
        ++ahead_idx;
        if (++ahead == R) { ahead = 0; ahead_par ^= 1; }
        const uint32_t bar = bars + kMwRingFull + 8 * ahead;
        if (!mbar_try_wait(bar, ahead_par) && !mbar_wait_bounded(bar, ahead_par, P.status)) return;
      }
      if (any) {
        float a[kMwUnroll][V][MV];
        int off[kMwUnroll];                 // byte offset of worker k + u's own ring slot
#pragma unroll
        for (int u = 0; u < kMwUnroll; ++u) {
          int o = cur_off + u * (int)rb;
          o -= o >= ring_bytes ? ring_bytes : 0;
          off[u] = o;
          if (u < nu) {
            const uint32_t src = k + u < p ? kept_b + (uint32_t)(k + u) * rb : ring_b + (uint32_t)o;
#pragma unroll
            for (int v = 0; v < V; ++v) Row16<TH>::widen(lds128(src + (uint32_t)v * vstep), a[u][v]);
          }
        }
        for (int j = 0; j < q; ++j) {
#pragma unroll
          for (int u = 0; u < kMwUnroll; ++u) {
            if (u < nu) {
              const int code = codes[(k + u) * q + j];
              const int off_n = code >> 1;               // byte offset (signed for ring rows)
              int o = off[u] + off_n;
              o += o < 0 ? ring_bytes : 0;
              o -= o >= ring_bytes ? ring_bytes : 0;
              const uint32_t src = (code & 1) ? kept_b + (uint32_t)off_n : ring_b + (uint32_t)o;
              uint4 raw[V];
#pragma unroll
              for (int v = 0; v < V; ++v) raw[v] = lds128(src + (uint32_t)v * vstep);
#pragma unroll
              for (int v = 0; v < V; ++v) {
                float t[MV];
                Row16<TH>::widen(raw[v], t);
#pragma unroll
                for (int x = 0; x < MV; ++x) a[u][v][x] = __fadd_rn(a[u][v][x], t[x]);
              }
            }
          }
        }
#pragma unroll
        for (int u = 0; u < kMwUnroll; ++u) {
          if (u < nu) {
            TH* out = gp + (long long)u * P.ld;
#pragma unroll
            for (int v = 0; v < V; ++v) {
              if (P.inv_exact) {
#pragma unroll
                for (int x = 0; x < MV; ++x) a[u][v][x] = __fmul_rn(a[u][v][x], P.inv_qp1);
              } else {
                uint32_t mid = 0xFFFFFFFFu;
#pragma unroll
                for (int x = 0; x < MV; ++x) mid &= mid_range_bit(a[u][v][x]);
                if (mid & kMidRange) {
#pragma unroll
                  for (int x = 0; x < MV; ++x) a[u][v][x] = divide_corrected(a[u][v][x], P.qp1, P.inv_qp1);
                } else {
#pragma unroll
                  for (int x = 0; x < MV; ++x) a[u][v][x] = __fdiv_rn(a[u][v][x], P.qp1);
                }
              }
              TH* ov = out + (long long)v * P.ncons * MV;
              if (whole[v]) {
                ThetaTraits<TH>::stg(ov, a[u][v]);
              } else if (mine[v]) {
                const long long e = e0 + (long long)(c + v * P.ncons) * MV;
                for (int x = 0; x < MV; ++x)
                  if (e + x >= lo && e + x < hi) ov[x] = ThetaTraits<TH>::narrow(a[u][v][x]);
              }
            }
          }
        }
      }
      gp += (long long)nu * P.ld;
      // ring indices up to k + nu - 1 - p are not needed by any later worker
      __syncwarp();
      if (lane0) {
        for (int u = 0; u < nu; ++u) {
          if (k + u >= p) {
            int s2 = cur + u - p;
            s2 += s2 < 0 ? R : 0;
            s2 -= s2 >= R ? R : 0;
            mbar_arrive(bars + kMwRingEmpty + 8 * s2);
          }
        }
      }
      cur += nu;
      cur_off += nu * (int)rb;
      if (cur >= R) { cur -= R; cur_off -= ring_bytes; cur_par ^= 1; }
    }
    // after the last worker (cur is now the slot of the next tile's ring index 0): the last
    // min(p, K) ring indices, which nobody released yet, and the kept rows / meta entry
    __syncwarp();
    if (lane0) {
      int s = cur;
      for (int i = 0; i < p && i < K; ++i) {
        if (--s < 0) s = R - 1;
        mbar_arrive(bars + kMwRingEmpty + 8 * s);
      }
      mbar_arrive(bars + kMwKeptEmpty + 8 * set);
    }
  }
}

}  // namespace

#endif  // GBMUF_CSRC_SYNC_MA_WINDOW_CUH
