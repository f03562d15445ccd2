// The fused round with the theta tile in tensor memory; device self-tests.
// Part of libgbmuf (CUDA, sm_100a); included by gbmuf.cu, which is the only translation unit.
#ifndef GBMUF_CSRC_SYNC_FUSED_TMEM_CUH
#define GBMUF_CSRC_SYNC_FUSED_TMEM_CUH

namespace {

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
// Element group g (4 elements) of a tile lives in lane g % 128, columns ((g / 128) * W + cell row)
// * cell width, W the number of rows held at once.  The allocation is released by the warp that
// made it after every thread has reached the end of the kernel; no path returns early.
//
// Which rows are held.  Definition 1's ring means worker k only ever averages with workers within
// ring distance p, so with many workers the K rows of a tile need not all be resident.  The rows
// of a tile are requested in a sequence of `npos` positions and worker k's output item is issued
// once position k + lead has been requested (or all have).
//   all rows (W = K):     npos = K, position s is row s and lives in cell row s; every row is
//                         requested before the first output item (lead >= K).
//   ring window (W < K):  position s is row (s - p) mod K, lead = 2p: worker k needs exactly
//                         positions k .. k + 2p (its own row is position k + p).  Position s
//                         lives in cell row s mod W, W = 2p + rows per load item: a load item
//                         requested while worker k is next overwrites positions below k only.
//                         The ring closes on itself, so the last workers need the first rows
//                         again (positions K + p .. K + 2p - 1 = rows 0 .. p - 1), which the
//                         first workers have overwritten in global memory by then (the round
//                         is in place): those rows are put into p extra cell rows when they
//                         first arrive and stay there.  The last p rows, which the first
//                         workers need before everything else and the last workers own, are
//                         either requested twice (npos = K + p, keep_lo = p, 3p + rows-per-item
//                         cell rows, p extra row reads per tile out of K) or kept as well
//                         (npos = K, keep_lo = 0, 4p + rows-per-item cell rows, every row read
//                         once).  A position at or beyond npos is a kept row and lives in cell
//                         row W + (position - npos).
// Consumers take the items in the same order as the producer requests them, so "overwrites only
// what no later worker needs" holds by program order; no extra synchronisation is involved.
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
  int W, wtot, npos, lead, pshift;   // window cell rows, all cell rows (W + kept rows),
                                     // positions per tile, output lead, p (window) or 0
  int keep_lo;                       // window: positions keep_lo .. 2p - 1 are also kept
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
  // the same cell row of two element groups with one wait
  static __device__ __forceinline__ void fetch2(uint32_t t0, uint32_t t1, float (&x)[4], float (&y)[4]) {
    uint32_t r[8];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%8];\n\t"
        "tcgen05.ld.sync.aligned.32x32b.x4.b32 {%4, %5, %6, %7}, [%9];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
        : "r"(t0), "r"(t1)
        : "memory");
#pragma unroll
    for (int c = 0; c < 4; ++c) { x[c] = __uint_as_float(r[c]); y[c] = __uint_as_float(r[4 + c]); }
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
  static __device__ __forceinline__ void fetch2(uint32_t t0, uint32_t t1, float (&x)[4], float (&y)[4]) {
    uint32_t a, b, c, d;
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0, %1}, [%4];\n\t"
        "tcgen05.ld.sync.aligned.32x32b.x2.b32 {%2, %3}, [%5];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(a), "=r"(b), "=r"(c), "=r"(d)
        : "r"(t0), "r"(t1)
        : "memory");
    x[0] = __uint_as_float(a << 16); x[1] = __uint_as_float(a & 0xFFFF0000u);
    x[2] = __uint_as_float(b << 16); x[3] = __uint_as_float(b & 0xFFFF0000u);
    y[0] = __uint_as_float(c << 16); y[1] = __uint_as_float(c & 0xFFFF0000u);
    y[2] = __uint_as_float(d << 16); y[3] = __uint_as_float(d & 0xFFFF0000u);
  }
};

// Sum of a worker's own cell (cell row `own`) and its q drawn neighbours' cells (cell rows nb[])
// of element group `cell0` (the TMEM address of cell row 0), own first, then draw order, each
// addition rounded.
template <typename TH>
__device__ __forceinline__ void tmem_gather(uint32_t cell0, int own, const int* nb, int q, float (&a)[4]) {
  constexpr int CW = TmemCell<TH>::COLS;
  TmemCell<TH>::fetch(cell0 + (uint32_t)(own * CW), a);
  for (int j = 0; j < q; ++j) {
    float t[4];
    TmemCell<TH>::fetch(cell0 + (uint32_t)(nb[j] * CW), t);
#pragma unroll
    for (int x = 0; x < 4; ++x) a[x] = __fadd_rn(a[x], t[x]);
  }
}

// The same sums for two element groups of the thread at once (cell row 0 at cellA and cellB): one
// wait per pair of loads, so the two groups' tensor-memory round trips overlap.
template <typename TH>
__device__ __forceinline__ void tmem_gather2(uint32_t cellA, uint32_t cellB, int own, const int* nb, int q,
                                             float (&a)[4], float (&b)[4]) {
  constexpr int CW = TmemCell<TH>::COLS;
  TmemCell<TH>::fetch2(cellA + (uint32_t)(own * CW), cellB + (uint32_t)(own * CW), a, b);
  for (int j = 0; j < q; ++j) {
    float t[4], u[4];
    const uint32_t o = (uint32_t)(nb[j] * CW);
    TmemCell<TH>::fetch2(cellA + o, cellB + o, t, u);
#pragma unroll
    for (int x = 0; x < 4; ++x) { a[x] = __fadd_rn(a[x], t[x]); b[x] = __fadd_rn(b[x], u[x]); }
  }
}
// A thread's element groups are taken two at a time.  (Several cell rows of ONE group per wait --
// two, or four from many neighbours on -- measured slower or no faster; with 15 neighbours the
// pairs run the round in 16.97 ms against 19.4 ms with four cells of one group per wait.)
constexpr bool kPairGroups = true;

// What the producer must know to send a finished slot out: the staged range starts at e0, whole
// 16-byte pieces of the rows cover [sb, se); k < 0: a load item, nothing to send.
struct SlotInfo { long long e0, sb, se; int k; int pad; };

// Slot layout.  Load item: IN_ROWS rows of T theta elements.  Output item (one per worker):
// [omega T floats | Delta T floats | (BULK) new theta T elements].
// BULK: the outputs leave through bulk stores from the ring slot instead of st.global from
// registers.
// WIN: ring window (else all K rows resident; the window's arithmetic then folds away).
template <typename TH, bool BULK, bool WIN>
__global__ void __launch_bounds__(544, 1) sync_fused_tmem_kernel(const TmemParams P) {
  grid_launch_dependents();
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
  const int R = P.ring, K = P.K, q = P.q, T = P.T;
  const int W = WIN ? P.W : K, wtot = WIN ? P.wtot : K, npos = WIN ? P.npos : K, pshift = WIN ? P.pshift : 0;
  // Items of a tile, in the order both sides generate them: with `s` positions requested and `k`
  // workers put out, the next item is a load item (positions s .. s + IN_ROWS - 1) while
  // s < npos and s <= k + lead, else worker k's output item.
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int r = 0; r < R; ++r) {
      mbar_init(bars + 8 * r, 1);
      mbar_init(bars + 64 + 8 * r, 16);                  // every consumer warp arrives (through lane 0)
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
  // everything above overlapped the round set-up kernel; its tables are read from here on
  grid_dependency_wait();
  const int total = P.tile_prefix[P.m];
  const int my_tiles = (int)blockIdx.x < total ? (total - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;

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
        // the drawn neighbours as cell rows: the worker id itself when all rows are held, else
        // the neighbour's position k + p + (signed ring distance), folded into the window or, past
        // the last requested position, one of the kept first rows
        const int32_t* gnb = P.nbr + (size_t)comp * K * q;
        for (int x = lane; x < K * q; x += 32) {
          int n = __ldg(gnb + x);
          if (WIN) {
            const int k = x / q;
            int dist = n - k;
            if (dist > pshift) dist -= K;
            if (dist < -pshift) dist += K;
            const int pos = k + pshift + dist;
            n = pos < npos ? pos % W : W + (pos - npos);
          }
          snb[x] = n;
        }
      }
      __syncwarp();
      if (lane == 0) {
        d->e0 = e0;
        d->lo = lo;
        d->hi = hi;
        d->comp = comp;
      }
      __syncwarp();
      for (int s = 0, k = 0; k < K && ok; ++gi) {
        const bool is_load = s < npos && (!WIN || s <= k + P.lead);
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
            si.k = is_load ? -1 : k;
            si.pad = 0;
            sinfo[slot] = si;
          }
          if (is_load) {
            const int rows = npos - s < IN_ROWS ? npos - s : IN_ROWS;
            const uint32_t bytes = (uint32_t)run * EB;
            mbar_arrive_expect_tx(full, (uint32_t)rows * bytes);
            for (int r = 0; r < rows; ++r) {
              const int row = WIN ? (s + r + K - pshift) % K : s + r;
              bulk_load_row(dst + (uint32_t)r * (uint32_t)T * EB, theta_in + (long long)row * P.ld + e0, bytes, full);
            }
          } else {
            const long long at = (long long)k * P.ld + e0;
            const uint32_t bytes = (uint32_t)run * 4u;
            mbar_arrive_expect_tx(full, 2u * bytes);
            bulk_load_row(dst, P.omega + at, bytes, full);
            bulk_load_row(dst + (uint32_t)T * 4u, P.delta + at, bytes, full);
          }
        }
        if (is_load) s += IN_ROWS; else ++k;
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
      bool first = true;
      for (int s = 0, k = 0; k < K && ok; ++gi) {
        const bool is_load = s < npos && (!WIN || s <= k + P.lead);
        const int slot = gi % R;
        bool fine = mbar_wait_bounded(bars + 8 * slot, (gi / R) & 1, P.status);
        ok = __all_sync(0xffffffffu, fine);
        if (!ok) break;
        if (first) {
          first = false;
          e0 = d->e0; lo = d->lo; hi = d->hi;
          sb = (lo + ALN - 1) & ~(ALN - 1);       // whole 16-byte pieces of theta inside the tile
          se = hi & ~(ALN - 1);
        }
        unsigned char* const sbase = ring0 + (size_t)slot * P.slot_stride;
        if (is_load) {
          // deposit the theta rows of this item into this thread's TMEM cells
          const TH* rows_in = reinterpret_cast<const TH*>(sbase);
          int cell[IN_ROWS], keep[IN_ROWS];         // keep: cell row of a kept first row, or -1
#pragma unroll
          for (int r = 0; r < IN_ROWS; ++r) {
            cell[r] = WIN ? (s + r) % W : s + r;
            keep[r] = (WIN && s + r >= P.keep_lo && s + r < 2 * pshift) ? W + s + r - P.keep_lo : -1;
          }
          for (int g = sub; g < ngroups; g += 4) {
            const int col = (g * 128 + quarter * 32 + lane) * 4;
#pragma unroll
            for (int r = 0; r < IN_ROWS; ++r)
              if (s + r < npos) {
                TmemCell<TH>::deposit(tlane + (uint32_t)((g * wtot + cell[r]) * CW), rows_in + (size_t)r * T + col);
                if (WIN && keep[r] >= 0)
                  TmemCell<TH>::deposit(tlane + (uint32_t)((g * wtot + keep[r]) * CW), rows_in + (size_t)r * T + col);
              }
          }
          asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        } else {
          const int own = !WIN ? k : k + pshift < npos ? (k + pshift) % W : W + k + pshift - npos;
          float* row0 = reinterpret_cast<float*>(sbase);
          float* row1 = row0 + T;
          TH* row2 = reinterpret_cast<TH*>(row1 + T);      // BULK: the new theta
          // one element group of this worker: average, filter, outputs (into the slot or to memory)
          auto finish_group = [&](int g, float (&a)[4]) {
            const int col = (g * 128 + quarter * 32 + lane) * 4;
            const long long e = e0 + col;
            if (e >= hi || e + 4 <= lo) return;
            float t[4];
            average_divide(a, P.qp1, P.inv_qp1, P.inv_exact);
            const float4 Wv = *reinterpret_cast<const float4*>(row0 + col);
            const float4 Dv = *reinterpret_cast<const float4*>(row1 + col);
            float wv[4] = {Wv.x, Wv.y, Wv.z, Wv.w}, dv[4] = {Dv.x, Dv.y, Dv.z, Dv.w};
#pragma unroll
            for (int x = 0; x < 4; ++x) bmuf_filter<TH>(a[x], wv[x], dv[x], t[x], P.eta, P.zeta);
            const long long at = (long long)k * P.ld + e;
            if (BULK && e >= sb && e + 4 <= se) {
              *reinterpret_cast<float4*>(row0 + col) = make_float4(wv[0], wv[1], wv[2], wv[3]);
              *reinterpret_cast<float4*>(row1 + col) = make_float4(dv[0], dv[1], dv[2], dv[3]);
              ThetaTraits<TH>::sts_quad(row2 + col, t);
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
          };
          const bool pairs = kPairGroups;
          for (int g = sub; g < ngroups; g += pairs ? 8 : 4) {
            float a[4], b[4];
            __syncwarp();                          // lanes that left the last group early rejoin
            if (pairs && g + 4 < ngroups) {
              tmem_gather2<TH>(tlane + (uint32_t)(g * wtot * CW), tlane + (uint32_t)((g + 4) * wtot * CW), own,
                               snb + k * q, q, a, b);
              finish_group(g, a);
              finish_group(g + 4, b);
            } else {
              tmem_gather<TH>(tlane + (uint32_t)(g * wtot * CW), own, snb + k * q, q, a);
              finish_group(g, a);
            }
          }
        }
        // every thread makes its own writes to the slot visible to the copy engine; then the warp
        // arrives once (16 arrivals per item instead of 512 on one barrier)
        if (BULK && !is_load) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + 64 + 8 * slot);
        if (is_load) s += IN_ROWS; else ++k;
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

}  // namespace

#endif  // GBMUF_CSRC_SYNC_FUSED_TMEM_CUH
