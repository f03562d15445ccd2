// Bounded mbarrier waits, bulk copies, theta storage types.
// Part of libgbmuf (CUDA, sm_100a); included by gbmuf.cu, which is the only translation unit.
#ifndef GBMUF_CSRC_PRIMITIVES_CUH
#define GBMUF_CSRC_PRIMITIVES_CUH

namespace {

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
// Programmatic dependent launch.  The fused round kernel is launched with the "programmatic
// stream serialization" attribute: it may start while the kernel before it in the stream (the
// round set-up kernel) is still running, so that its prologue -- barrier initialisation, the
// tensor-memory allocation -- overlaps that kernel.  grid_dependency_wait() returns once the
// preceding kernel has completed and its writes are visible; nothing that kernel writes (the
// neighbour table, the work-list) and nothing the kernels before it wrote is read earlier.
// (The set-up kernel says "griddepcontrol.launch_dependents" at its start.)  Launched without
// the attribute, the instruction does nothing.
__device__ __forceinline__ void grid_dependency_wait() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
// Said at the top of the long kernels (the fused round, the local steps): a set-up kernel queued
// behind them may be made resident early; it waits for their completion before doing anything.
__device__ __forceinline__ void grid_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
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
// per box, delivered to this CTA only; completion is counted in bytes on the mbarrier, out-of-range columns
// are zero-filled and still counted.  x * element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_box(uint32_t dst_smem, const CUtensorMap* map, int x, int y,
                                             uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], "
      "[%1, {%2, %3}], [%4];" ::"r"(dst_smem),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
      : "memory");
}

// One-dimensional bulk copy global -> shared through the copy engine (to this CTA only); completion
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
  // the same four elements into shared memory
  static __device__ __forceinline__ void sts_quad(float* p, const float (&x)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
  }
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
  static __device__ __forceinline__ void sts_quad(__nv_bfloat16* p, const float (&x)[4]) {
    uint2 t;
    __nv_bfloat162 h;
    h = __floats2bfloat162_rn(x[0], x[1]); t.x = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2bfloat162_rn(x[2], x[3]); t.y = *reinterpret_cast<uint32_t*>(&h);
    *reinterpret_cast<uint2*>(p) = t;
  }
};

}  // namespace

#endif  // GBMUF_CSRC_PRIMITIVES_CUH
