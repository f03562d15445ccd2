// Local steps (synthetic noise, Adagrad), initialisation and final average.
// Part of libgbmuf (CUDA, sm_100a); included by gbmuf.cu, which is the only translation unit.
#ifndef GBMUF_CSRC_LOCAL_STEP_CUH
#define GBMUF_CSRC_LOCAL_STEP_CUH

namespace {

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
  grid_launch_dependents();
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
  grid_launch_dependents();
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
        ThetaTraits<TH>::sts_quad(sth + col, th);
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
// Initialisation as a copy-engine job: a chunk of theta_0 is fetched into shared memory once and
// sent out 3K times -- to theta^k and omega^k of every worker, plus a block of zeros to Delta^k
// -- by bulk stores; the threads only widen bf16 to fp32 for omega and handle the few elements
// after the last whole 16-byte piece of theta_0.  4 + 12K bytes per parameter, all but 4 written.
constexpr int kInitChunk = 4096;     // elements per chunk
constexpr int kInitSlots = 3;        // chunks whose stores may be in flight

template <typename TH>
__global__ void __launch_bounds__(128) init_stream_kernel(const TH* theta0, TH* theta, float* omega,
                                                          float* delta, int K, long long N,
                                                          long long ld, int32_t* status) {
  constexpr int EB = (int)sizeof(TH);
  constexpr int T = kInitChunk, R = kInitSlots;
  constexpr bool WIDEN = EB != 4;                       // omega needs its own fp32 copy
  constexpr uint32_t SLOT = (uint32_t)T * EB + (WIDEN ? (uint32_t)T * 4u : 0u);
  extern __shared__ __align__(128) unsigned char smem[];
  // [0, 64) barriers | [128, 128 + 4T) zeros | slots: [theta_0 chunk | (bf16) the chunk as fp32]
  const uint32_t bars = smem_u32(smem);
  float* zeros = reinterpret_cast<float*>(smem + 128);
  unsigned char* slot0 = smem + 128 + (size_t)T * 4;
  const long long nchunks = (N + T - 1) / T;
  if (threadIdx.x == 0) {
    for (int r = 0; r < R; ++r) mbar_init(bars + 8 * r, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = threadIdx.x; i < T; i += blockDim.x) zeros[i] = 0.0f;
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();

  int it = 0;
  for (long long ch = blockIdx.x; ch < nchunks; ch += gridDim.x, ++it) {
    const int slot = it % R;
    const long long e0 = ch * T;
    const int n = (int)(N - e0 < T ? N - e0 : T);        // elements of this chunk
    const int nw = n & ~(16 / EB - 1);                   // ... in whole 16-byte pieces of theta_0
    unsigned char* sb = slot0 + (size_t)slot * SLOT;
    if (threadIdx.x == 0) {
      // the stores issued from this slot R chunks ago must have read it
      if (it >= R) asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(R - 1) : "memory");
      if (nw > 0) {
        mbar_arrive_expect_tx(bars + 8 * slot, (uint32_t)nw * EB);
        bulk_load_row(smem_u32(sb), theta0 + e0, (uint32_t)nw * EB, bars + 8 * slot);
      } else {
        mbar_arrive(bars + 8 * slot);
      }
    }
    // (the slot is not touched by the other threads before the barrier below completes a phase
    // that thread 0 arms only after the wait above)
    const bool ok = mbar_wait_bounded(bars + 8 * slot, (it / R) & 1, status);
    if (ok) {
      if (WIDEN) {
        const TH* st = reinterpret_cast<const TH*>(sb);
        float* sw = reinterpret_cast<float*>(sb + (size_t)T * EB);
        for (int i = threadIdx.x * 4; i < nw; i += blockDim.x * 4) {
          float f[4];
          ThetaTraits<TH>::lds_quad(st + i, f);
          *reinterpret_cast<float4*>(sw + i) = make_float4(f[0], f[1], f[2], f[3]);
        }
      }
      // the elements after the last whole piece: straight from theta_0 to every worker's rows
      for (int i = nw + threadIdx.x; i < n; i += blockDim.x) {
        const TH v = theta0[e0 + i];
        for (int k = 0; k < K; ++k) {
          const long long at = (long long)k * ld + e0 + i;
          theta[at] = v;
          omega[at] = ThetaTraits<TH>::widen(v);
          delta[at] = 0.0f;
        }
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (__syncthreads_or(!ok)) break;                    // a wait expired: everybody leaves
    if (threadIdx.x == 0) {
      if (nw > 0) {
        const uint32_t s_th = smem_u32(sb), s_om = WIDEN ? s_th + (uint32_t)T * EB : s_th;
        const uint32_t s_ze = smem_u32(zeros);
        for (int k = 0; k < K; ++k) {
          const long long at = (long long)k * ld + e0;
          asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(theta + at), "r"(s_th), "r"((uint32_t)nw * EB) : "memory");
          asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(omega + at), "r"(s_om), "r"((uint32_t)nw * 4u) : "memory");
          asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(delta + at), "r"(s_ze), "r"((uint32_t)nw * 4u) : "memory");
        }
      }
      asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    }
  }
  if (threadIdx.x == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
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

}  // namespace

#endif  // GBMUF_CSRC_LOCAL_STEP_CUH
