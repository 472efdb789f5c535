// Shared definitions of the IST library's device code: status word, launch helpers, types.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ist {

typedef __nv_bfloat16 bf16;

// Sticky device status: word 0 = code (0 = ok, otherwise an ist_status value), word 1 = site
// tag of the first failure, words 2..3 = detail (offending index / value).
struct DeviceStatus {
  int code;
  int site;
  long long detail;
};

enum Site : int {
  SITE_NONE = 0,
  SITE_LABEL = 1,      // label outside [0, N_t)
  SITE_CSR_COL = 2,    // CSR column outside [0, N_0)
  SITE_PART_IDX = 3,   // partition index outside [0, N_l)
  SITE_TC_PIPE = 4,    // bounded wait in the tensor-core pipeline expired
  SITE_CSR_ROW = 5     // CSR row_ptr not monotone
};

__device__ __forceinline__ void report(DeviceStatus* st, int code, int site, long long detail) {
  if (atomicCAS(&st->code, 0, code) == 0) {
    st->site = site;
    st->detail = detail;
  }
}

// Programmatic dependent launch.  A kernel launched with launch_pdl may be scheduled while the
// kernel before it in the stream is still running; it must call pdl_wait() before it touches
// global memory (that waits until the earlier kernel has completed and its writes are visible).
// pdl_trigger() lets the kernel after this one be scheduled as this grid's CTAs retire.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

__host__ __device__ __forceinline__ constexpr int64_t ceil_div(int64_t a, int64_t b) {
  return (a + b - 1) / b;
}
__host__ __device__ __forceinline__ constexpr int64_t round_up(int64_t a, int64_t b) {
  return ceil_div(a, b) * b;
}

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_float(float v);
template <> __device__ __forceinline__ float from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_float<bf16>(float v) { return __float2bfloat16_rn(v); }

// Four adjacent elements as one 16-byte (fp32) or 8-byte (bf16) access; p must be aligned to it.
__device__ __forceinline__ void load4(const float* p, float v[4]) {
  float4 t = *reinterpret_cast<const float4*>(p);
  v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
__device__ __forceinline__ void load4(const bf16* p, float v[4]) {
  uint2 t = *reinterpret_cast<const uint2*>(p);
  __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&t.x);
  __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162*>(&t.y);
  v[0] = __low2float(a); v[1] = __high2float(a); v[2] = __low2float(b); v[3] = __high2float(b);
}
__device__ __forceinline__ void store4(float* p, const float v[4]) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
__device__ __forceinline__ void store4(bf16* p, const float v[4]) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]);
  __nv_bfloat162 b = __floats2bfloat162_rn(v[2], v[3]);
  uint2 t;
  t.x = *reinterpret_cast<uint32_t*>(&a);
  t.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = t;
}

}  // namespace ist
