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

}  // namespace ist
