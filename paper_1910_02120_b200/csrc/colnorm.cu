// Per-neuron batch standardisation of the hidden layers (paper Sec. 2.2 "Correcting
// Distributional Shift"): the input of every hidden neuron is shifted and scaled by its mean and
// standard deviation over the minibatch before the non-linearity, and the backward pass goes
// through that transform.  No learned scale or shift; biased variance, sigma = sqrt(var + eps).
//
// Layout: z [G][B][ld] fp32 (pre-activations, written by the forward GEMM), statistics [G][ld].
// A block owns 32 adjacent columns of one group; its 8 row lanes walk the batch, so every load
// is a 128-byte row segment.  Means are taken in two passes (mean, then centred squares) and all
// partial sums are combined in a fixed order.  act may alias z (fp32, in place): every thread
// reads an element before it writes that same element.
#include "kernels.h"

namespace ist {
namespace {

constexpr int kCols = 32, kLanes = 8;

// Sum over the 8 row lanes of each column (fixed order); result valid in every thread.
__device__ __forceinline__ float lane_sum(float v, float (*sh)[kCols + 1]) {
  __syncthreads();
  sh[threadIdx.y][threadIdx.x] = v;
  __syncthreads();
  float s = 0.f;
#pragma unroll
  for (int u = 0; u < kLanes; ++u) s += sh[u][threadIdx.x];
  return s;
}

template <typename T>
__global__ void __launch_bounds__(kCols * kLanes) colnorm_forward_kernel(
    const float* z, int64_t ld, int64_t z_sg, int B, int n, float eps, float* __restrict__ mu_out,
    float* __restrict__ rstd_out, int64_t stat_sg, T* act, int64_t act_sg) {
  __shared__ float sh[kLanes][kCols + 1];
  pdl_wait();
  pdl_trigger();
  const int g = blockIdx.y;
  const int col = blockIdx.x * kCols + threadIdx.x;
  const bool live = col < n;                 // pad columns (n..ld) produce zeros
  const float* zc = z + (int64_t)g * z_sg + col;
  float s = 0.f;
  if (live)
    for (int b = threadIdx.y; b < B; b += kLanes) s += zc[(int64_t)b * ld];
  const float mu = lane_sum(s, sh) / (float)B;
  float q = 0.f;
  if (live)
    for (int b = threadIdx.y; b < B; b += kLanes) {
      const float d = zc[(int64_t)b * ld] - mu;
      q = fmaf(d, d, q);
    }
  const float var = lane_sum(q, sh) / (float)B;
  const float rstd = rsqrtf(var + eps);
  if (col < ld) {
    if (threadIdx.y == 0) {
      mu_out[(int64_t)g * stat_sg + col] = live ? mu : 0.f;
      rstd_out[(int64_t)g * stat_sg + col] = live ? rstd : 0.f;
    }
    T* ac = act + (int64_t)g * act_sg + col;
    for (int b = threadIdx.y; b < B; b += kLanes) {
      const float h = live ? (zc[(int64_t)b * ld] - mu) * rstd : 0.f;
      ac[(int64_t)b * ld] = from_float<T>(fmaxf(h, 0.f));
    }
  }
}

// delta holds d_zh = (delta_{l+1} W^T) * [zh > 0] on entry and d_z on exit:
// d_z = (d_zh - mean_b d_zh - zh * mean_b(d_zh * zh)) / sigma.
template <typename T>
__global__ void __launch_bounds__(kCols * kLanes) colnorm_backward_kernel(
    T* __restrict__ delta, int64_t ld, int64_t d_sg, const float* __restrict__ z, int64_t z_sg,
    const float* __restrict__ mu_in, const float* __restrict__ rstd_in, int64_t stat_sg, int B, int n) {
  __shared__ float sh[kLanes][kCols + 1];
  pdl_wait();
  pdl_trigger();
  const int g = blockIdx.y;
  const int col = blockIdx.x * kCols + threadIdx.x;
  const bool live = col < n;
  const float mu = live ? mu_in[(int64_t)g * stat_sg + col] : 0.f;
  const float rstd = live ? rstd_in[(int64_t)g * stat_sg + col] : 0.f;
  const float* zc = z + (int64_t)g * z_sg + col;
  T* dc = delta + (int64_t)g * d_sg + col;
  float s1 = 0.f, s2 = 0.f;
  if (live)
    for (int b = threadIdx.y; b < B; b += kLanes) {
      const float d = to_float(dc[(int64_t)b * ld]);
      const float h = (zc[(int64_t)b * ld] - mu) * rstd;
      s1 += d;
      s2 = fmaf(d, h, s2);
    }
  const float m1 = lane_sum(s1, sh) / (float)B;
  const float m2 = lane_sum(s2, sh) / (float)B;
  if (live)
    for (int b = threadIdx.y; b < B; b += kLanes) {
      const float d = to_float(dc[(int64_t)b * ld]);
      const float h = (zc[(int64_t)b * ld] - mu) * rstd;
      dc[(int64_t)b * ld] = from_float<T>((d - m1 - h * m2) * rstd);
    }
}


// ---- vector kernels for 16-byte aligned rows (ld % 4 == 0): the training path ---------------------
// 8 column threads x 32 row lanes; a thread owns 4 adjacent columns.  The forward kernel keeps its
// rows in registers when the batch fits (B <= 32 * R), so z is read once; the backward kernel reads
// its block's slab twice, the second time from L2.
constexpr int kVecCols = 32, kVecLanes = 32, kVecThreads = 256;

// Sum over the 32 row lanes for each of a thread's 4 columns; result valid in every thread.
__device__ __forceinline__ void lane_sum4(float v[4], float (*sh)[kVecCols]) {
#pragma unroll
  for (int u = 0; u < 4; ++u) {            // a warp holds 4 row lanes x 8 column threads
    v[u] += __shfl_xor_sync(0xffffffffu, v[u], 8);
    v[u] += __shfl_xor_sync(0xffffffffu, v[u], 16);
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tx = threadIdx.x & 7;
  __syncthreads();
  if (lane < 8)
#pragma unroll
    for (int u = 0; u < 4; ++u) sh[warp][tx * 4 + u] = v[u];
  __syncthreads();
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < kVecThreads / 32; ++w) s += sh[w][tx * 4 + u];
    v[u] = s;
  }
}

template <typename T, int R>
__global__ void __launch_bounds__(kVecThreads) colnorm_forward_vec_kernel(
    const float* z, int64_t ld, int64_t z_sg, int B, int n, float eps, float* __restrict__ mu_out,
    float* __restrict__ rstd_out, int64_t stat_sg, T* act, int64_t act_sg) {
  __shared__ float sh[kVecThreads / 32][kVecCols];
  pdl_wait();
  pdl_trigger();
  const int g = blockIdx.y;
  const int tx = threadIdx.x & 7, ty = threadIdx.x >> 3;
  const int col = blockIdx.x * kVecCols + tx * 4;
  const bool in = col < ld;                       // ld % 4 == 0: a thread's 4 columns are in or out together
  const float* zc = z + (int64_t)g * z_sg + col;
  float v[R > 0 ? R : 1][4];
  float s[4] = {0.f, 0.f, 0.f, 0.f};
  if (R > 0) {
#pragma unroll
    for (int i = 0; i < R; ++i) {
      const int b = ty + kVecLanes * i;
      if (in && b < B) load4(zc + (int64_t)b * ld, v[i]);
      else v[i][0] = v[i][1] = v[i][2] = v[i][3] = 0.f;
    }
#pragma unroll
    for (int i = 0; i < R; ++i)
#pragma unroll
      for (int u = 0; u < 4; ++u) s[u] += v[i][u];
  } else if (in) {
#pragma unroll 4
    for (int b = ty; b < B; b += kVecLanes) {
      float t[4];
      load4(zc + (int64_t)b * ld, t);
#pragma unroll
      for (int u = 0; u < 4; ++u) s[u] += t[u];
    }
  }
  lane_sum4(s, sh);
  float mu[4], q[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int u = 0; u < 4; ++u) mu[u] = s[u] / (float)B;
  if (R > 0) {
#pragma unroll
    for (int i = 0; i < R; ++i)
      if (ty + kVecLanes * i < B)
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const float d = v[i][u] - mu[u];
          q[u] = fmaf(d, d, q[u]);
        }
  } else if (in) {
#pragma unroll 4
    for (int b = ty; b < B; b += kVecLanes) {
      float t[4];
      load4(zc + (int64_t)b * ld, t);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const float d = t[u] - mu[u];
        q[u] = fmaf(d, d, q[u]);
      }
    }
  }
  lane_sum4(q, sh);
  float rstd[4];
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const bool live = col + u < n;                // pad columns (n..ld) produce zeros
    rstd[u] = live ? rsqrtf(q[u] / (float)B + eps) : 0.f;
    if (!live) mu[u] = 0.f;
  }
  if (!in) return;
  if (ty == 0) {
    store4(mu_out + (int64_t)g * stat_sg + col, mu);
    store4(rstd_out + (int64_t)g * stat_sg + col, rstd);
  }
  T* ac = act + (int64_t)g * act_sg + col;
  if (R > 0) {
#pragma unroll
    for (int i = 0; i < R; ++i) {
      const int b = ty + kVecLanes * i;
      if (b < B) {
        float o[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) o[u] = fmaxf((v[i][u] - mu[u]) * rstd[u], 0.f);
        store4(ac + (int64_t)b * ld, o);
      }
    }
  } else {
#pragma unroll 4
    for (int b = ty; b < B; b += kVecLanes) {
      float t[4];
      load4(zc + (int64_t)b * ld, t);
#pragma unroll
      for (int u = 0; u < 4; ++u) t[u] = fmaxf((t[u] - mu[u]) * rstd[u], 0.f);
      store4(ac + (int64_t)b * ld, t);
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(kVecThreads) colnorm_backward_vec_kernel(
    T* __restrict__ delta, int64_t ld, int64_t d_sg, const float* __restrict__ z, int64_t z_sg,
    const float* __restrict__ mu_in, const float* __restrict__ rstd_in, int64_t stat_sg, int B) {
  __shared__ float sh[kVecThreads / 32][kVecCols];
  pdl_wait();
  pdl_trigger();
  const int g = blockIdx.y;
  const int tx = threadIdx.x & 7, ty = threadIdx.x >> 3;
  const int col = blockIdx.x * kVecCols + tx * 4;
  const bool in = col < ld;
  float mu[4] = {0.f, 0.f, 0.f, 0.f}, rstd[4] = {0.f, 0.f, 0.f, 0.f};   // pad columns hold rstd = 0
  if (in) {
    load4(mu_in + (int64_t)g * stat_sg + col, mu);
    load4(rstd_in + (int64_t)g * stat_sg + col, rstd);
  }
  const float* zc = z + (int64_t)g * z_sg + col;
  T* dc = delta + (int64_t)g * d_sg + col;
  float s1[4] = {0.f, 0.f, 0.f, 0.f}, s2[4] = {0.f, 0.f, 0.f, 0.f};
  if (in) {
#pragma unroll 4
    for (int b = ty; b < B; b += kVecLanes) {
      float d[4], t[4];
      load4(dc + (int64_t)b * ld, d);
      load4(zc + (int64_t)b * ld, t);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        s1[u] += d[u];
        s2[u] = fmaf(d[u], (t[u] - mu[u]) * rstd[u], s2[u]);
      }
    }
  }
  lane_sum4(s1, sh);
  lane_sum4(s2, sh);
  if (!in) return;
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    s1[u] /= (float)B;
    s2[u] /= (float)B;
  }
#pragma unroll 4
  for (int b = ty; b < B; b += kVecLanes) {
    float d[4], t[4];
    load4(dc + (int64_t)b * ld, d);
    load4(zc + (int64_t)b * ld, t);
#pragma unroll
    for (int u = 0; u < 4; ++u) d[u] = (d[u] - s1[u] - (t[u] - mu[u]) * rstd[u] * s2[u]) * rstd[u];
    store4(dc + (int64_t)b * ld, d);
  }
}

// Deployment: z <- max((z - mu) / sigma, 0) with stored statistics (rows x n, row stride ld).
__global__ void colnorm_apply_kernel(float* __restrict__ z, int64_t ld, int rows, int n,
                                     const float* __restrict__ mu, const float* __restrict__ rstd) {
  const int col = blockIdx.x * blockDim.x + threadIdx.x;
  if (col >= n) return;
  const float m = mu[col], r = rstd[col];
  for (int b = blockIdx.y; b < rows; b += gridDim.y) {
    float* p = z + (int64_t)b * ld + col;
    *p = fmaxf((*p - m) * r, 0.f);
  }
}

}  // namespace

template <typename T>
void colnorm_forward(const Launch& L, const float* z, int64_t ld, int64_t z_sg, int G, int B, int n, float eps,
                     float* mu, float* rstd, int64_t stat_sg, T* act, int64_t act_sg) {
  const bool vec = ld % 4 == 0 && z_sg % 4 == 0 && act_sg % 4 == 0 && stat_sg % 4 == 0 &&
                   ((uintptr_t)z & 15) == 0 && ((uintptr_t)act & 15) == 0 && ((uintptr_t)mu & 15) == 0 &&
                   ((uintptr_t)rstd & 15) == 0;
  const dim3 vgrid((unsigned)ceil_div(ld, kVecCols), G);
  if (vec && B <= kVecLanes * 16)
    launch_pdl(colnorm_forward_vec_kernel<T, 16>, vgrid, dim3(kVecThreads), 0, L.stream, z, ld, z_sg, B, n, eps, mu, rstd,
               stat_sg, act, act_sg);
  else if (vec)
    launch_pdl(colnorm_forward_vec_kernel<T, 0>, vgrid, dim3(kVecThreads), 0, L.stream, z, ld, z_sg, B, n, eps, mu, rstd,
               stat_sg, act, act_sg);
  else
    launch_pdl(colnorm_forward_kernel<T>, dim3((unsigned)ceil_div(ld, kCols), G), dim3(kCols, kLanes), 0, L.stream, z,
               ld, z_sg, B, n, eps, mu, rstd, stat_sg, act, act_sg);
  L.count();
}
template void colnorm_forward<float>(const Launch&, const float*, int64_t, int64_t, int, int, int, float, float*, float*,
                                     int64_t, float*, int64_t);
template void colnorm_forward<bf16>(const Launch&, const float*, int64_t, int64_t, int, int, int, float, float*, float*,
                                    int64_t, bf16*, int64_t);

template <typename T>
void colnorm_backward(const Launch& L, T* delta, int64_t ld, int64_t d_sg, const float* z, int64_t z_sg, const float* mu,
                      const float* rstd, int64_t stat_sg, int G, int B, int n) {
  const bool vec = ld % 4 == 0 && z_sg % 4 == 0 && d_sg % 4 == 0 && stat_sg % 4 == 0 && ((uintptr_t)z & 15) == 0 &&
                   ((uintptr_t)delta & 15) == 0 && ((uintptr_t)mu & 15) == 0 && ((uintptr_t)rstd & 15) == 0;
  if (vec)   // the forward kernel stored mu = rstd = 0 for pad columns, so n is not needed here
    launch_pdl(colnorm_backward_vec_kernel<T>, dim3((unsigned)ceil_div(ld, kVecCols), G), dim3(kVecThreads), 0, L.stream,
               delta, ld, d_sg, z, z_sg, mu, rstd, stat_sg, B);
  else
    launch_pdl(colnorm_backward_kernel<T>, dim3((unsigned)ceil_div(ld, kCols), G), dim3(kCols, kLanes), 0, L.stream,
               delta, ld, d_sg, z, z_sg, mu, rstd, stat_sg, B, n);
  L.count();
}
template void colnorm_backward<float>(const Launch&, float*, int64_t, int64_t, const float*, int64_t, const float*,
                                      const float*, int64_t, int, int, int);
template void colnorm_backward<bf16>(const Launch&, bf16*, int64_t, int64_t, const float*, int64_t, const float*,
                                     const float*, int64_t, int, int, int);

void colnorm_apply(const Launch& L, float* z, int64_t ld, int rows, int n, const float* mu, const float* rstd) {
  dim3 grid((unsigned)ceil_div(n, 256), (unsigned)(rows < 256 ? rows : 256));
  colnorm_apply_kernel<<<grid, 256, 0, L.stream>>>(z, ld, rows, n, mu, rstd);
  L.count();
}

}  // namespace ist
