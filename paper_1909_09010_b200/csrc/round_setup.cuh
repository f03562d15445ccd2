// Neighbour draws and the tile work-list of a round.
// Part of libgbmuf (CUDA, sm_100a); included by gbmuf.cu, which is the only translation unit.
#ifndef GBMUF_CSRC_ROUND_SETUP_CUH
#define GBMUF_CSRC_ROUND_SETUP_CUH

namespace {

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
  // This kernel is itself launched as a programmatic dependent: it may become resident while the
  // kernel before it in the stream (a local step, the previous round) still runs, which hides
  // its launch latency.  It must not touch the tables before that kernel has finished -- the
  // previous round reads them -- so it waits first.  Then the round kernel that follows may begin
  // its prologue; it in turn waits for this grid to finish before it reads the tables written
  // below (and thereby, transitively, for everything before this grid).
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
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

}  // namespace

#endif  // GBMUF_CSRC_ROUND_SETUP_CUH
