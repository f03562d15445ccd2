// Philox4x32-10 counter-based generator, device side.
// Part of libgbmuf (CUDA, sm_100a); included by gbmuf.cu, which is the only translation unit.
#ifndef GBMUF_CSRC_PHILOX_CUH
#define GBMUF_CSRC_PHILOX_CUH

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

}  // namespace

#endif  // GBMUF_CSRC_PHILOX_CUH
