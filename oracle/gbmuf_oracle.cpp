// Oracle for the random-gossip BMUF synchronisation round.
//
// TEST INFRASTRUCTURE, NOT PRODUCT CODE.  This file is the slow, single-threaded, plain CPU
// statement of what the synchronisation step of "A Random Gossip BMUF Process for Neural
// Language Modeling" (Algorithm 1, the body of `if t mod H_i == 0`) computes.  Only the test
// suite, the smoke check and the bench's CPU-baseline leg may call it.  It shares no code,
// header, table or constant generator with the CUDA library; nothing here is tuned.
//
// Build: g++ -std=c++17 -O2 -ffp-contract=off -fno-fast-math -shared -fPIC
// (-ffp-contract=off matters: every product and sum below is rounded to fp32 on its own).
//
// Every floating-point step is fp32, round-to-nearest-even, in the order written in
// Algorithm 1.  bf16 appears only as a storage format of theta (exact widening on load,
// round-to-nearest-even on store).
//
// Pins (tests/test_oracle_*.py): Philox known-answer vectors of the published generator,
// sampler invariants + brute-force enumeration, float64 mixing-matrix brute force of the
// gossip average, the full-average (classic BMUF) and eta=0 (model averaging) closed forms,
// the geometric-series closed form of the block-momentum filter, fixed points, worker-order
// independence, moments of the perturbation noise.  No function here is "parity unpinned".

#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <vector>

namespace {

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3",
// SC'11).  Written from the published round description.
// ---------------------------------------------------------------------------------------------
struct U4 { uint32_t w[4]; };

U4 philox4x32_10(U4 ctr, uint32_t key0, uint32_t key1) {
  const uint64_t M0 = 0xD2511F53ull, M1 = 0xCD9E8D57ull;
  const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
  for (int r = 0; r < 10; ++r) {
    if (r > 0) { key0 += W0; key1 += W1; }
    const uint64_t p0 = M0 * (uint64_t)ctr.w[0];
    const uint64_t p1 = M1 * (uint64_t)ctr.w[2];
    U4 nxt;
    nxt.w[0] = (uint32_t)(p1 >> 32) ^ ctr.w[1] ^ key0;
    nxt.w[1] = (uint32_t)p1;
    nxt.w[2] = (uint32_t)(p0 >> 32) ^ ctr.w[3] ^ key1;
    nxt.w[3] = (uint32_t)p0;
    ctr = nxt;
  }
  return ctr;
}

// ---------------------------------------------------------------------------------------------
// bf16 storage: widening is exact; narrowing rounds to nearest, ties to even.
// ---------------------------------------------------------------------------------------------
float bf16_to_f32(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return f;
}

uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  std::memcpy(&u, &f, 4);
  if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu) != 0u)
    return (uint16_t)((u >> 16) | 0x0040u);          // NaN stays NaN (quiet)
  const uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb;
  return (uint16_t)(u >> 16);
}

enum { DT_F32 = 0, DT_BF16 = 1 };

float load_theta(const void* base, int dtype, int64_t idx) {
  if (dtype == DT_F32) return ((const float*)base)[idx];
  return bf16_to_f32(((const uint16_t*)base)[idx]);
}

// `store` of Algorithm 1's left arrows into theta's storage type; returns the value as stored.
float store_theta(void* base, int dtype, int64_t idx, float v) {
  if (dtype == DT_F32) { ((float*)base)[idx] = v; return v; }
  const uint16_t h = f32_to_bf16_rne(v);
  ((uint16_t*)base)[idx] = h;
  return bf16_to_f32(h);
}

// ---------------------------------------------------------------------------------------------
// Definition 1: node k of an n-node p-symmetric ring is linked to (k-1)%n .. (k-p)%n and
// (k+1)%n .. (k+p)%n.  Listed in that order; a node equal to k, or already listed (possible
// only when 2p > n-1, which the paper's settings never reach), is skipped.
// ---------------------------------------------------------------------------------------------
int candidate_list(int k, int K, int p, int32_t* out) {
  int c = 0;
  for (int side = 0; side < 2; ++side) {
    for (int d = 1; d <= p; ++d) {
      int64_t raw = side == 0 ? (int64_t)k - d : (int64_t)k + d;
      int node = (int)(((raw % K) + K) % K);
      if (node == k) continue;
      bool seen = false;
      for (int j = 0; j < c; ++j) seen = seen || (out[j] == node);
      if (!seen) out[c++] = node;
    }
  }
  return c;
}

}  // namespace

extern "C" {

void gbo_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) {
  U4 c = {{ctr[0], ctr[1], ctr[2], ctr[3]}};
  U4 r = philox4x32_10(c, key[0], key[1]);
  for (int i = 0; i < 4; ++i) out[i] = r.w[i];
}

uint16_t gbo_f32_to_bf16(float f) { return f32_to_bf16_rne(f); }
float gbo_bf16_to_f32(uint16_t h) { return bf16_to_f32(h); }
void gbo_f32_to_bf16_array(const float* in, uint16_t* out, int64_t n) {
  for (int64_t i = 0; i < n; ++i) out[i] = f32_to_bf16_rne(in[i]);
}

// Definition 1.  `out` must hold 2*p entries.  Returns the list length c = min(2p, K-1).
int gbo_candidate_list(int k, int K, int p, int32_t* out) {
  if (K < 1 || k < 0 || k >= K || p < 0) return -1;
  return candidate_list(k, K, p, out);
}

// Algorithm 1, the neighbour-choice line (k_1..k_q): an independent uniform draw of q
// distinct nodes out of worker k's ring neighbours for every (round, worker k, component i).
// Partial Fisher-Yates over the candidate list; the j-th swap index uses one 32-bit Philox
// word reduced to [0, c-j) by multiply-shift.
//   key     = { seed_lo, seed_hi ^ 0x53414D50 }
//   counter = { round_lo, round_hi, comp_base + i, k | (block << 16) },  block = j / 4
// nbr is [K][m][q].  Returns 0, or -1 on bad arguments (q > c included).
int gbo_sample_neighbors(uint64_t seed, uint64_t round, int K, int m, int comp_base, int p, int q,
                         int32_t* nbr) {
  if (K < 1 || K > 65535 || m < 1 || p < 0 || q < 0) return -1;
  std::vector<int32_t> a((size_t)(2 * p > 0 ? 2 * p : 1));
  for (int k = 0; k < K; ++k) {
    for (int i = 0; i < m; ++i) {
      const int c = candidate_list(k, K, p, a.data());
      if (q > c) return -1;
      U4 rnd = {{0, 0, 0, 0}};
      for (int j = 0; j < q; ++j) {
        if (j % 4 == 0) {
          U4 ctr = {{(uint32_t)round, (uint32_t)(round >> 32), (uint32_t)(comp_base + i),
                     (uint32_t)k | ((uint32_t)(j / 4) << 16)}};
          rnd = philox4x32_10(ctr, (uint32_t)seed, (uint32_t)(seed >> 32) ^ 0x53414D50u);
        }
        const uint32_t u = rnd.w[j % 4];
        const int t = j + (int)(((uint64_t)u * (uint64_t)(c - j)) >> 32);
        const int32_t tmp = a[j]; a[j] = a[t]; a[t] = tmp;
        nbr[((size_t)k * m + i) * q + j] = a[j];
      }
    }
  }
  return 0;
}

// One synchronisation round (Algorithm 1, the body of `if t mod H_i == 0`, for every worker k
// and every component i whose sync flag is set).
//
//   theta  [K][ld]  replicas, fp32 or bf16 (dtype); updated in place
//   omega  [K][ld]  per-worker global model, fp32
//   delta  [K][ld]  per-worker block momentum, fp32
//   rst    [K][ld]  theta's dtype: worker k's component value right after its previous sync
//                   (theta_0 before any sync) -- the "theta_{i,t-H_i}^k" of the block-delta line
//   gout   [K][ld]  fp32 or NULL: receives the block delta G (a scratch slot in the paper)
//   off    [m+1]    component i covers elements off[i] .. off[i+1]-1
//   sync   [m] or NULL (= all)
//   nbr    [K][m][q] the chosen neighbours
//   order  [K] or NULL: the order in which workers are processed (results must not depend on it)
//   mode   0 = gossip-BMUF, 1 = gossip-MA
//
// All neighbour reads see the replicas as they were when the round began: every term of the
// averaging line carries the same time index t.
int gbo_sync_round(int K, int64_t N, int64_t ld, int dtype, void* theta, float* omega,
                   float* delta, void* rst, float* gout, int m, const int64_t* off,
                   const uint8_t* sync, const int32_t* nbr, int q, float eta, float zeta,
                   int mode, const int32_t* order) {
  if (K < 1 || N < 0 || ld < N || m < 1 || q < 0) return -1;
  const size_t esz = dtype == DT_F32 ? 4 : 2;
  std::vector<unsigned char> snap((size_t)K * (size_t)ld * esz);
  std::memcpy(snap.data(), theta, snap.size());                  // S <- theta (pre-round)
  const void* S = snap.data();

  for (int kk = 0; kk < K; ++kk) {
    const int k = order ? order[kk] : kk;
    for (int i = 0; i < m; ++i) {
      if (sync && !sync[i]) continue;
      const int32_t* nb = nbr + ((size_t)k * m + i) * q;
      for (int64_t e = off[i]; e < off[i + 1]; ++e) {
        const int64_t at = (int64_t)k * ld + e;
        // averaging line: own value first, then k_1..k_q in draw order
        float s = load_theta(S, dtype, at);
        for (int j = 0; j < q; ++j) s = s + load_theta(S, dtype, (int64_t)nb[j] * ld + e);
        const float avg = s / (float)(q + 1);
        if (mode == 1) {                                          // gossip-MA
          store_theta(theta, dtype, at, avg);
          continue;
        }
        const float g = avg - load_theta(rst, dtype, at);         // G <- avg - theta_{t-H}
        const float md = eta * delta[at];
        const float zg = zeta * g;
        const float d = md + zg;                                  // Delta <- eta Delta + zeta G
        const float w = omega[at] + d;                            // omega <- omega + Delta
        const float nd = eta * d;
        const float t = w + nd;                                   // theta <- omega + eta Delta
        delta[at] = d;
        omega[at] = w;
        const float stored = store_theta(theta, dtype, at, t);
        store_theta(rst, dtype, at, stored);
        if (gout) gout[at] = g;
      }
    }
  }
  return 0;
}

// Initialisation line of Algorithm 1: theta_0^k <- theta_0, omega^k <- theta_0, Delta^k <- 0
// (and the stored block-start value rst <- theta_0).
int gbo_init(int K, int64_t N, int64_t ld, int dtype, const void* theta0, void* theta,
             float* omega, float* delta, void* rst) {
  if (K < 1 || N < 0 || ld < N) return -1;
  for (int k = 0; k < K; ++k) {
    for (int64_t e = 0; e < N; ++e) {
      const int64_t at = (int64_t)k * ld + e;
      const float v = load_theta(theta0, dtype, e);
      store_theta(theta, dtype, at, v);
      store_theta(rst, dtype, at, v);
      omega[at] = v;
      delta[at] = 0.0f;
    }
  }
  return 0;
}

// Synthetic stand-in for the local SGD line theta <- theta - alpha * g, with g = sigma * z and
// z a counter-based approximately standard normal: the sum of the four 16-bit halves of two
// Philox words, centred (mean 131070) and scaled to unit variance (variance (2^32-1)/3).
//   key     = { seed_lo, seed_hi ^ 0x50455254 }
//   counter = { pair_lo, pair_hi, k, step },  pair = (elem_base + e) / 2
//   even element of the pair uses words 0,1; odd element uses words 2,3
// Steps step .. step+nsteps-1 are applied one after another, each stored to theta's dtype.
int gbo_local_perturb(int K, int64_t N, int64_t ld, int dtype, void* theta, uint64_t seed,
                      uint64_t step, float lr, float sigma, int nsteps, int64_t elem_base) {
  if (K < 1 || N < 0 || ld < N || nsteps < 0 || elem_base < 0) return -1;
  if (step + (uint64_t)nsteps > 0xFFFFFFFFull) return -1;
  const float C = 0x1.bb67aep-16f;   // (float)(1 / sqrt((2^32 - 1) / 3))
  for (int k = 0; k < K; ++k) {
    for (int64_t e = 0; e < N; ++e) {
      const uint64_t ge = (uint64_t)(elem_base + e);
      const uint64_t pair = ge >> 1;
      const int64_t at = (int64_t)k * ld + e;
      float v = load_theta(theta, dtype, at);
      for (int s = 0; s < nsteps; ++s) {
        U4 ctr = {{(uint32_t)pair, (uint32_t)(pair >> 32), (uint32_t)k, (uint32_t)(step + s)}};
        const U4 r = philox4x32_10(ctr, (uint32_t)seed, (uint32_t)(seed >> 32) ^ 0x50455254u);
        const uint32_t a = (ge & 1) ? r.w[2] : r.w[0];
        const uint32_t b = (ge & 1) ? r.w[3] : r.w[1];
        const int32_t sum = (int32_t)((a & 0xFFFFu) + (a >> 16) + (b & 0xFFFFu) + (b >> 16));
        const float z = (float)(sum - 131070) * C;
        const float sz = sigma * z;
        const float upd = lr * sz;
        v = v - upd;
        v = store_theta(theta, dtype, at, v);
      }
    }
  }
  return 0;
}

// The local step with the optimiser of the paper's experiments (Section 3.2) in place of the
// plain SGD line of Algorithm 1: Adagrad, with the gradient norm of a group of parameters (there:
// the LSTM weights) clipped to clip_norm.  Per worker k:
//   norm_k = sqrt(sum of g^2 over the elements inside the clip ranges)       (summed in double)
//   g'     = g * (clip_norm / max(norm_k, clip_norm)) inside the ranges, g elsewhere
//   a     <- a + g' * g'
//   theta <- store(theta - (lr * g') / (sqrt(a) + eps))
// grad and accum are fp32 [K][ld]; ranges is nranges pairs [begin, end) of element indices;
// clip_norm <= 0 switches clipping off.
int gbo_local_adagrad(int K, int64_t N, int64_t ld, int dtype, void* theta, const float* grad,
                      float* accum, float lr, float eps, float clip_norm, int nranges,
                      const int64_t* ranges) {
  if (K < 1 || N < 0 || ld < N || nranges < 0) return -1;
  for (int k = 0; k < K; ++k) {
    float scale = 1.0f;
    if (clip_norm > 0.0f && nranges > 0) {
      double ss = 0.0;
      for (int r = 0; r < nranges; ++r)
        for (int64_t e = ranges[2 * r]; e < ranges[2 * r + 1]; ++e) {
          const double g = (double)grad[(int64_t)k * ld + e];
          ss += g * g;
        }
      const float norm = (float)std::sqrt(ss);
      scale = clip_norm / (norm > clip_norm ? norm : clip_norm);
    }
    for (int64_t e = 0; e < N; ++e) {
      const int64_t at = (int64_t)k * ld + e;
      bool inside = false;
      for (int r = 0; r < nranges; ++r) inside = inside || (e >= ranges[2 * r] && e < ranges[2 * r + 1]);
      float g = grad[at];
      if (inside && clip_norm > 0.0f) g = g * scale;
      const float gg = g * g;
      const float a = accum[at] + gg;
      accum[at] = a;
      const float denom = std::sqrt(a) + eps;
      const float num = lr * g;
      const float upd = num / denom;
      store_theta(theta, dtype, at, load_theta(theta, dtype, at) - upd);
    }
  }
  return 0;
}

// Return line of Algorithm 1: theta = (1/n) sum_k theta_T^k.  Sum over k = 0..K-1 in that
// order in fp32, one divide.  out is [N], theta's dtype.
int gbo_final_average(int K, int64_t N, int64_t ld, int dtype, const void* theta, void* out) {
  if (K < 1 || N < 0 || ld < N) return -1;
  for (int64_t e = 0; e < N; ++e) {
    float s = load_theta(theta, dtype, e);
    for (int k = 1; k < K; ++k) s = s + load_theta(theta, dtype, (int64_t)k * ld + e);
    store_theta(out, dtype, e, s / (float)K);
  }
  return 0;
}

}  // extern "C"
