// Shared device/host helpers of libssa (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "ssa.h"

namespace ssa {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Per-thread bookkeeping shared by the entry points (defined in ssa_api.cu).
void note_launches(int n);
void take_kernel_events(cudaEvent_t* begin, cudaEvent_t* end);
int sm_count();   // multiprocessors of the current device (cached; no synchronisation)

// Programmatic dependent launch.  Every kernel of the library is launched
// with the programmatic-serialization attribute: its blocks may become
// resident while the preceding kernel of the stream is still draining, and
// they call grid_dependency_wait() before touching any global memory, which
// returns once that kernel has completed and its writes are visible.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_smem(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t dynamic_smem,
                                   cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = dynamic_smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
#ifdef SSA_NO_PDL
  cfg.numAttrs = 0;
#else
  cfg.numAttrs = 1;
#endif
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t stream, Args... args) {
  return launch_pdl_smem(kernel, grid, block, 0, stream, args...);
}

__device__ __forceinline__ float neg_inf() { return __int_as_float(0xff800000); }

// 16-byte read-only load that does not allocate in L1: every K/V row is used once.
__device__ __forceinline__ uint4 ld_stream_16B(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

// A K/V cache stored as 8-bit e4m3 values (1 sign, 4 exponent, 3 mantissa bits; outside the paper).  Queries and
// outputs that go with such a cache are bf16.
struct Fp8E4M3 { uint8_t bits; };
template <typename T> struct Storage { using Query = T; };
template <> struct Storage<Fp8E4M3> { using Query = __nv_bfloat16; };
template <typename T> constexpr bool kIsFp8 = false;
template <> constexpr bool kIsFp8<Fp8E4M3> = true;

// Two e4m3 values (the low 16 bits of `pair`) -> two floats (exact: every e4m3 value is an fp16 value).
__device__ __forceinline__ float2 e4m3x2_to_float2(uint32_t pair) {
  uint32_t h2;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((unsigned short)pair));
  return __half22float2(*reinterpret_cast<const __half2*>(&h2));
}

// Two packed 16-bit storage values -> two floats (exact).
template <typename T>
__device__ __forceinline__ float2 unpack2(uint32_t u);
template <>
__device__ __forceinline__ float2 unpack2<__nv_bfloat16>(uint32_t u) {
  return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
}
template <>
__device__ __forceinline__ float2 unpack2<__half>(uint32_t u) {
  return __half22float2(*reinterpret_cast<const __half2*>(&u));
}

template <typename T>
__device__ __forceinline__ void unpack8(const uint4& r, float (&f)[8]) {
  float2 a = unpack2<T>(r.x), b = unpack2<T>(r.y), c = unpack2<T>(r.z), d = unpack2<T>(r.w);
  f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y;
  f[4] = c.x; f[5] = c.y; f[6] = d.x; f[7] = d.y;
}

template <typename T>
__device__ __forceinline__ T from_float(float x);
template <>
__device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }
template <>
__device__ __forceinline__ __half from_float<__half>(float x) { return __float2half_rn(x); }

// Packed fp32 multiply-add on both halves: a * b + c.
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) {
  float2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;"
      : "=l"(*reinterpret_cast<unsigned long long*>(&d))
      : "l"(*reinterpret_cast<unsigned long long*>(&a)), "l"(*reinterpret_cast<unsigned long long*>(&b)),
        "l"(*reinterpret_cast<unsigned long long*>(&c)));
  return d;
}

// 2^x; 2^-inf = +0.
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

}  // namespace ssa
