// Shared device helpers of the ADORE kernels: element types, the device error word,
// warp/block reductions, order-preserving keys.
#pragma once

#include <cstdlib>

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace adore {

// Bits of the device error word.
enum : unsigned {
  ERRW_TIMEOUT = 1u,      // a bounded wait (mbarrier) ran out
  ERRW_BAD_LIST = 2u,     // explicit rebuild entry out of range
  ERRW_BOUNDS = 4u,       // an index check failed; the access was skipped
};

enum : uint8_t { ROLE_EMPTY = 0, ROLE_RETAINED = 1, ROLE_REBUILT = 2 };

__device__ __forceinline__ void set_error(unsigned* word, unsigned bit) { atomicOr(word, bit); }

// fp32 -> uint32 whose unsigned order equals the float order (-inf lowest, +inf highest).
__device__ __forceinline__ uint32_t float_key(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Value order of tokens (higher score first, then the newer token): one 64-bit key.
__device__ __forceinline__ unsigned long long value_key(float score, int tok) {
  return (static_cast<unsigned long long>(float_key(score)) << 32) | static_cast<uint32_t>(tok);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ unsigned long long warp_min(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    unsigned long long t = __shfl_xor_sync(0xffffffffu, v, o);
    v = t < v ? t : v;
  }
  return v;
}
__device__ __forceinline__ int warp_min(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = min(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Element access for the two cache types.
template <typename T> struct Elem;
template <> struct Elem<float> {
  static constexpr int kPer16B = 4;
  __device__ static __forceinline__ void unpack(const uint4& r, float* f) {
    f[0] = __uint_as_float(r.x); f[1] = __uint_as_float(r.y);
    f[2] = __uint_as_float(r.z); f[3] = __uint_as_float(r.w);
  }
  __device__ static __forceinline__ float to_float(float v) { return v; }
  __device__ static __forceinline__ float from_float(float v) { return v; }
};
template <> struct Elem<__nv_bfloat16> {
  static constexpr int kPer16B = 8;
  __device__ static __forceinline__ void unpack(const uint4& r, float* f) {
    // bf16 -> fp32 is a 16-bit shift; the low element of each 32-bit word comes first
    f[0] = __uint_as_float(r.x << 16); f[1] = __uint_as_float(r.x & 0xffff0000u);
    f[2] = __uint_as_float(r.y << 16); f[3] = __uint_as_float(r.y & 0xffff0000u);
    f[4] = __uint_as_float(r.z << 16); f[5] = __uint_as_float(r.z & 0xffff0000u);
    f[6] = __uint_as_float(r.w << 16); f[7] = __uint_as_float(r.w & 0xffff0000u);
  }
  __device__ static __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
  __device__ static __forceinline__ __nv_bfloat16 from_float(float v) { return __float2bfloat16_rn(v); }
};

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  // read-once data: do not allocate in L1 (plain weak load: the same kernel may later write the row)
  uint4 r;
  asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
  return r;
}

// ---- development switches -------------------------------------------------------------------------
// A build with -DADORE_DEVTOOLS reads a few environment variables that turn a launch choice off, for A/B timing of
// the variant that then serves the launch. The ordinary build reads no environment variable at all.
#ifdef ADORE_DEVTOOLS
inline bool dev_switch(const char* name) { return std::getenv(name) != nullptr; }
inline int dev_switch_int(const char* name, int dflt) { const char* v = std::getenv(name); return v ? std::atoi(v) : dflt; }
#else
inline bool dev_switch(const char*) { return false; }
inline int dev_switch_int(const char*, int dflt) { return dflt; }
#endif

// ---- programmatic dependent launch ----------------------------------------------------------------
// A kernel launched with launch_dependent() may be placed on the SMs while the kernel ahead of it in the stream is
// still finishing, which hides its launch latency. Such a kernel calls wait_for_prior_grid() before it reads anything
// an earlier kernel wrote and before it writes anything; the call returns once the earlier kernel has completed and
// its writes are visible (a no-op for an ordinary launch).
__device__ __forceinline__ void wait_for_prior_grid() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Called early by short kernels: lets the next kernel of the stream, if it was launched with launch_dependent(), move
// onto the SMs and run up to its own wait_for_prior_grid() while this one is still working.
__device__ __forceinline__ void let_next_grid_start() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                    Args&&... args) {
  static const bool off = dev_switch("ADORE_NO_DEPENDENT_LAUNCH");
  cudaLaunchConfig_t lc{};
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  lc.gridDim = grid; lc.blockDim = block; lc.dynamicSmemBytes = smem; lc.stream = stream;
  lc.attrs = at; lc.numAttrs = off ? 0 : 1;
  return cudaLaunchKernelEx(&lc, kernel, static_cast<KArgs>(args)...);
}

}  // namespace adore
