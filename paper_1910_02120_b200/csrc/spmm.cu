// Sparse (CSR) first layer of the local steps: the paper's extreme-classification network
// takes a 135,909-dimensional sparse feature vector (Sec. 3 "Experimental Settings"), so the
// first-layer product, its weight gradient and the SGD update run over stored nonzeros only.
//
// Mapping: one warp per (subnet g, batch row b) and per chunk of 128 output columns; lane L
// owns columns 4L..4L+3 of the chunk.  The nonzero's column index and value are warp-uniform
// loads; the weight row segment is a contiguous 256/512-byte read per warp.
#include "kernels.h"

namespace ist {
namespace {

constexpr int kRowsPerCta = 4;


// VEC = false: element-wise accesses for leading dimensions that are not multiples of 4
// (the full network's first layer during evaluation).
template <typename T, typename TO, bool VEC>
__global__ void spmm_forward_kernel(const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col,
                                    const float* __restrict__ val, int64_t row0,
                                    int64_t group_row_stride, int B, int64_t N0,
                                    const T* __restrict__ P, int64_t p_ld, int64_t p_sg,
                                    const float* __restrict__ bias, int64_t bias_sg, int n1,
                                    TO* __restrict__ out, int64_t out_ld, int64_t out_sg,
                                    DeviceStatus* st, bool relu) {
  int g = blockIdx.y;
  int b = blockIdx.x * kRowsPerCta + threadIdx.y;
  int cc = blockIdx.z * 128 + threadIdx.x * 4;
  if (b >= B || cc >= out_ld) return;
  int64_t r = row0 + (int64_t)g * group_row_stride + b;
  int lo = row_ptr[r], hi = row_ptr[r + 1];
  if (hi < lo) {
    report(st, -5, SITE_CSR_ROW, r);
    hi = lo;
  }
  const T* Pg = P + (int64_t)g * p_sg + cc;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int p = lo; p < hi; ++p) {
    int c = col[p];
    float x = val[p];
    if (c < 0 || c >= N0) {
      report(st, -5, SITE_CSR_COL, p);
      continue;
    }
    float w[4];
    if (VEC) {
      load4(Pg + (int64_t)c * p_ld, w);
    } else {
#pragma unroll
      for (int u = 0; u < 4; ++u) w[u] = (cc + u) < n1 ? to_float(Pg[(int64_t)c * p_ld + u]) : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) acc[u] = fmaf(x, w[u], acc[u]);
  }
  float o[4];
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    float bv = (cc + u) < n1 ? bias[(int64_t)g * bias_sg + cc + u] : 0.f;
    o[u] = relu ? fmaxf(acc[u] + bv, 0.f) : acc[u] + bv;
  }
  TO* dst = out + (int64_t)g * out_sg + (int64_t)b * out_ld + cc;
  if (VEC) {
    store4(dst, o);
  } else {
#pragma unroll
    for (int u = 0; u < 4; ++u)
      if (cc + u < out_ld) dst[u] = from_float<TO>(o[u]);
  }
}

// Adds four floats to four adjacent words of global memory with one reduction instruction.
__device__ __forceinline__ void red_add_v4(float* p, float a, float b, float c, float d) {
  asm volatile("red.relaxed.gpu.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d)
               : "memory");
}

template <typename T, bool VEC>
__global__ void spmm_backward_kernel(const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col,
                                     const float* __restrict__ val, int64_t row0,
                                     int64_t group_row_stride, int B, int64_t N0,
                                     const T* __restrict__ delta,
                                     int64_t d_ld, int64_t d_sg, float* master, int64_t p_ld,
                                     int64_t p_sg, float lr) {
  int g = blockIdx.y;
  int b = blockIdx.x * kRowsPerCta + threadIdx.y;
  int cc = blockIdx.z * 128 + threadIdx.x * 4;
  if (b >= B || cc >= d_ld) return;
  int64_t r = row0 + (int64_t)g * group_row_stride + b;
  int lo = row_ptr[r], hi = max(lo, row_ptr[r + 1]);
  float d[4];
  load4(delta + (int64_t)g * d_sg + (int64_t)b * d_ld + cc, d);
  float* Mg = master + (int64_t)g * p_sg + cc;
  for (int p = lo; p < hi; ++p) {
    int c = col[p];
    if (c < 0 || c >= N0) continue;   // reported by the forward pass
    float x = -lr * val[p];
    float* dst = Mg + (int64_t)c * p_ld;
    if (VEC) {
      // one 16-byte reduction per lane: the row segment is 16-byte aligned (p_ld % 4 == 0)
      red_add_v4(dst, x * d[0], x * d[1], x * d[2], x * d[3]);
    } else {
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (cc + u < d_ld) atomicAdd(dst + u, x * d[u]);
    }
  }
}

__global__ void spmm_refresh_kernel(const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col,
                                    int64_t row0, int64_t group_row_stride, int B, int64_t N0,
                                    int64_t ld,
                                    const float* __restrict__ master, bf16* __restrict__ opw,
                                    int64_t p_sg) {
  int g = blockIdx.y;
  int b = blockIdx.x * kRowsPerCta + threadIdx.y;
  int cc = blockIdx.z * 128 + threadIdx.x * 4;
  if (b >= B || cc >= ld) return;
  int64_t r = row0 + (int64_t)g * group_row_stride + b;
  int lo = row_ptr[r], hi = max(lo, row_ptr[r + 1]);
  for (int p = lo; p < hi; ++p) {
    int c = col[p];
    if (c < 0 || c >= N0) continue;
    int64_t o = (int64_t)g * p_sg + (int64_t)c * ld + cc;
    float w[4];
    load4(master + o, w);
    store4(opw + o, w);
  }
}

}  // namespace

template <typename T, typename TO>
void spmm_forward(const Launch& L, const int32_t* row_ptr, const int32_t* col, const float* val,
                  int64_t row0, int64_t group_row_stride, int G, int B, int64_t N0, const T* P,
                  int64_t p_ld, int64_t p_sg, const float* bias, int64_t bias_sg, int n1, TO* out,
                  int64_t out_ld, int64_t out_sg, DeviceStatus* st, bool relu) {
  dim3 grid((unsigned)ceil_div(B, kRowsPerCta), G, (unsigned)ceil_div(out_ld, 128));
  if (p_ld % 4 == 0 && out_ld % 4 == 0)
    spmm_forward_kernel<T, TO, true><<<grid, dim3(32, kRowsPerCta), 0, L.stream>>>(
        row_ptr, col, val, row0, group_row_stride, B, N0, P, p_ld, p_sg, bias, bias_sg, n1, out,
        out_ld, out_sg, st, relu);
  else
    spmm_forward_kernel<T, TO, false><<<grid, dim3(32, kRowsPerCta), 0, L.stream>>>(
        row_ptr, col, val, row0, group_row_stride, B, N0, P, p_ld, p_sg, bias, bias_sg, n1, out,
        out_ld, out_sg, st, relu);
  L.count();
}
template void spmm_forward<float, float>(const Launch&, const int32_t*, const int32_t*, const float*,
                                         int64_t, int64_t, int, int, int64_t, const float*, int64_t,
                                         int64_t, const float*, int64_t, int, float*, int64_t, int64_t,
                                         DeviceStatus*, bool);
template void spmm_forward<bf16, float>(const Launch&, const int32_t*, const int32_t*, const float*,
                                        int64_t, int64_t, int, int, int64_t, const bf16*, int64_t,
                                        int64_t, const float*, int64_t, int, float*, int64_t, int64_t,
                                        DeviceStatus*, bool);
template void spmm_forward<bf16, bf16>(const Launch&, const int32_t*, const int32_t*, const float*,
                                       int64_t, int64_t, int, int, int64_t, const bf16*, int64_t,
                                       int64_t, const float*, int64_t, int, bf16*, int64_t, int64_t,
                                       DeviceStatus*, bool);

template <typename T>
void spmm_backward_sgd(const Launch& L, const int32_t* row_ptr, const int32_t* col, const float* val,
                       int64_t row0, int64_t group_row_stride, int G, int B, int64_t N0,
                       const T* delta, int64_t d_ld, int64_t d_sg, int n1, float* master, bf16* opw,
                       int64_t p_ld, int64_t p_sg, float lr) {
  dim3 grid((unsigned)ceil_div(B, kRowsPerCta), G, (unsigned)ceil_div(d_ld, 128));
  if (p_ld % 4 == 0 && ((uintptr_t)master & 15) == 0 && p_sg % 4 == 0)
    spmm_backward_kernel<T, true><<<grid, dim3(32, kRowsPerCta), 0, L.stream>>>(
        row_ptr, col, val, row0, group_row_stride, B, N0, delta, d_ld, d_sg, master, p_ld, p_sg, lr);
  else
    spmm_backward_kernel<T, false><<<grid, dim3(32, kRowsPerCta), 0, L.stream>>>(
        row_ptr, col, val, row0, group_row_stride, B, N0, delta, d_ld, d_sg, master, p_ld, p_sg, lr);
  L.count();
  if (opw) {
    spmm_refresh_kernel<<<grid, dim3(32, kRowsPerCta), 0, L.stream>>>(
        row_ptr, col, row0, group_row_stride, B, N0, p_ld, master, opw, p_sg);
    L.count();
  }
}
template void spmm_backward_sgd<float>(const Launch&, const int32_t*, const int32_t*, const float*,
                                       int64_t, int64_t, int, int, int64_t, const float*, int64_t,
                                       int64_t, int, float*, bf16*, int64_t, int64_t, float);
template void spmm_backward_sgd<bf16>(const Launch&, const int32_t*, const int32_t*, const float*,
                                      int64_t, int64_t, int, int, int64_t, const bf16*, int64_t,
                                      int64_t, int, float*, bf16*, int64_t, int64_t, float);

}  // namespace ist
