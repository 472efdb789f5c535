// Row-wise pieces of a local SGD step that are not contractions: softmax cross-entropy and
// its gradient, the bias update, input staging, and the evaluation reductions.
#include <algorithm>

#include "kernels.h"

namespace ist {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ float warp_max(float v) {
  for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Block-wide reductions with a fixed tree (deterministic for a given block size).
__device__ float block_max(float v, float* sh) {
  v = warp_max(v);
  int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) sh[w] = v;
  __syncthreads();
  float r = l < (blockDim.x >> 5) ? sh[l] : -INFINITY;
  return warp_max(r);
}
__device__ float block_sum(float v, float* sh) {
  v = warp_sum(v);
  int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) sh[w] = v;
  __syncthreads();
  float r = l < (blockDim.x >> 5) ? sh[l] : 0.f;
  return warp_sum(r);
}

// One CTA per row (g, b).  loss_row = log(sum exp(z - max)) + max - z[y];
// delta = (exp(z - max)/sum - [n == y]) / B.
template <typename T>
__global__ void softmax_xent_kernel(const float* __restrict__ logits, int64_t ld, int64_t sg, int B,
                                    int Nt, const int32_t* __restrict__ y, int64_t y_sg,
                                    T* __restrict__ delta, int64_t ld_d, int64_t sg_d,
                                    float* __restrict__ row_loss, DeviceStatus* st) {
  __shared__ float sh[32];
  pdl_wait();
  pdl_trigger();
  int g = blockIdx.y, b = blockIdx.x;
  const float* z = logits + (int64_t)g * sg + (int64_t)b * ld;
  T* d = delta + (int64_t)g * sg_d + (int64_t)b * ld_d;
  int label = y[(int64_t)g * y_sg + b];
  if (label < 0 || label >= Nt) {
    if (threadIdx.x == 0) report(st, -5, SITE_LABEL, (long long)g * B + b);
    label = 0;
  }
  float mx = -INFINITY;
  for (int n = threadIdx.x; n < Nt; n += blockDim.x) mx = fmaxf(mx, z[n]);
  mx = block_max(mx, sh);
  float se = 0.f;
  for (int n = threadIdx.x; n < Nt; n += blockDim.x) se += expf(z[n] - mx);
  se = block_sum(se, sh);
  float inv = 1.f / se, invB = 1.f / (float)B;
  for (int n = threadIdx.x; n < ld_d; n += blockDim.x) {
    float v = 0.f;
    if (n < Nt) v = (expf(z[n] - mx) * inv - (n == label ? 1.f : 0.f)) * invB;
    d[n] = from_float<T>(v);
  }
  if (threadIdx.x == 0) row_loss[(int64_t)g * B + b] = logf(se) + mx - z[label];
}

// Wide rows (hundreds of thousands of classes): one pass with a running (max, sum) pair per
// thread and 16-byte loads, then one pass that writes delta.  Row length ld is a multiple of 8.
template <typename T>
__global__ void __launch_bounds__(512) softmax_xent_wide_kernel(
    const float* __restrict__ logits, int64_t ld, int64_t sg, int B, int Nt, const int32_t* __restrict__ y,
    int64_t y_sg, T* __restrict__ delta, int64_t ld_d, int64_t sg_d, float* __restrict__ row_loss,
    DeviceStatus* st) {
  __shared__ float sm[16], ss[16];
  pdl_wait();
  pdl_trigger();
  const int g = blockIdx.y, b = blockIdx.x;
  const float* z = logits + (int64_t)g * sg + (int64_t)b * ld;
  T* d = delta + (int64_t)g * sg_d + (int64_t)b * ld_d;
  int label = y[(int64_t)g * y_sg + b];
  if (label < 0 || label >= Nt) {
    if (threadIdx.x == 0) report(st, -5, SITE_LABEL, (long long)g * B + b);
    label = 0;
  }
  float m = -INFINITY, s = 0.f;
  const int nvec = Nt / 4;
  for (int v = threadIdx.x; v < nvec; v += blockDim.x) {
    float4 t = *reinterpret_cast<const float4*>(z + 4 * v);
    float mx = fmaxf(fmaxf(t.x, t.y), fmaxf(t.z, t.w));
    if (mx > m) { s *= expf(m - mx); m = mx; }
    s += expf(t.x - m) + expf(t.y - m) + expf(t.z - m) + expf(t.w - m);
  }
  for (int n = nvec * 4 + threadIdx.x; n < Nt; n += blockDim.x) {
    float t = z[n];
    if (t > m) { s *= expf(m - t); m = t; }
    s += expf(t - m);
  }
  // combine (m, s) pairs: warp, then block
  for (int o = 16; o; o >>= 1) {
    float om = __shfl_xor_sync(0xffffffffu, m, o), os = __shfl_xor_sync(0xffffffffu, s, o);
    float nm = fmaxf(m, om);
    s = (m == -INFINITY ? 0.f : s * expf(m - nm)) + (om == -INFINITY ? 0.f : os * expf(om - nm));
    m = nm;
  }
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  if (l == 0) { sm[w] = m; ss[w] = s; }
  __syncthreads();
  float M = -INFINITY, S = 0.f;
  for (int u = 0; u < (int)(blockDim.x >> 5); ++u) {   // fixed order, every thread the same
    float nm = fmaxf(M, sm[u]);
    S = (M == -INFINITY ? 0.f : S * expf(M - nm)) + (sm[u] == -INFINITY ? 0.f : ss[u] * expf(sm[u] - nm));
    M = nm;
  }
  const float inv = 1.f / S, invB = 1.f / (float)B;
  const int nvec_d = (int)(ld_d / 4);
  for (int v = threadIdx.x; v < nvec_d; v += blockDim.x) {
    float o[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int n = 4 * v + e;
      o[e] = n < Nt ? (expf(z[n] - M) * inv - (n == label ? 1.f : 0.f)) * invB : 0.f;
    }
    T* dst = d + 4 * v;
    dst[0] = from_float<T>(o[0]); dst[1] = from_float<T>(o[1]);
    dst[2] = from_float<T>(o[2]); dst[3] = from_float<T>(o[3]);
  }
  if (threadIdx.x == 0) row_loss[(int64_t)g * B + b] = logf(S) + M - z[label];
}

// Narrow output layer (Nt <= 64): one warp per row.  The logits may arrive as `ks` partial
// products of a k-split GEMM (slab g * ks + s holds slice s of group g, B rows of ld columns);
// they are summed here together with the bias, so the split costs no extra launch.
template <typename T>
__global__ void __launch_bounds__(256) softmax_xent_small_kernel(
    const float* __restrict__ part, int ks, int64_t ld, int B, int Nt, const float* __restrict__ bias,
    int64_t bias_sg, const int32_t* __restrict__ y, int64_t y_sg, T* __restrict__ delta, int64_t ld_d,
    int64_t sg_d, float* __restrict__ row_loss, DeviceStatus* st) {
  pdl_wait();
  pdl_trigger();
  const int g = blockIdx.y, lane = threadIdx.x & 31;
  const int b = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (b >= B) return;
  int label = y[(int64_t)g * y_sg + b];
  if (label < 0 || label >= Nt) {
    if (lane == 0) report(st, -5, SITE_LABEL, (long long)g * B + b);
    label = 0;
  }
  float z[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int n = lane + 32 * h;
    float v = -INFINITY;
    if (n < Nt) {
      v = bias ? bias[(int64_t)g * bias_sg + n] : 0.f;
      for (int s = 0; s < ks; ++s) v += part[(((int64_t)g * ks + s) * B + b) * ld + n];   // fixed order
    }
    z[h] = v;
  }
  const float mx = warp_max(fmaxf(z[0], z[1]));
  const float e0 = z[0] == -INFINITY ? 0.f : expf(z[0] - mx), e1 = z[1] == -INFINITY ? 0.f : expf(z[1] - mx);
  const float se = warp_sum(e0 + e1);
  const float zl = warp_sum((lane == (label & 31)) ? z[label >> 5] : 0.f);
  const float inv = 1.f / se, invB = 1.f / (float)B;
  T* d = delta + (int64_t)g * sg_d + (int64_t)b * ld_d;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int n = lane + 32 * h;
    if (n < ld_d) {
      const float e = h ? e1 : e0;
      d[n] = from_float<T>(n < Nt ? (e * inv - (n == label ? 1.f : 0.f)) * invB : 0.f);
    }
  }
  if (lane == 0) row_loss[(int64_t)g * B + b] = logf(se) + mx - zl;
}

// Bias gradient and update of every layer in one launch: blockIdx.y = group, blockIdx.x runs over
// the layers' blocks of 64 columns one layer after the other (layer i owns blocks xstart[i] ..
// xstart[i + 1] - 1).  Thread (cx, ry) sums 8 adjacent columns over rows ry, ry + 32, ...; the 32
// partial sums of a column are added in a fixed order.  When a loss is wanted the grid has one
// more column of blocks (one per group) that averages the step's row losses (256 threads, fixed
// summation order).
__device__ __forceinline__ void load8(const float* p, float v[8]) {
  float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8(const bf16* p, float v[8]) {
  uint4 u = *reinterpret_cast<const uint4*>(p);
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
  for (int i = 0; i < 4; ++i) { v[2 * i] = __low2float(h[i]); v[2 * i + 1] = __high2float(h[i]); }
}

template <typename T>
__global__ void __launch_bounds__(256) bias_sgd_kernel(BiasSgdArgs<T> a, int n_layers, int B, float lr, LossReduce lo) {
  __shared__ float part[32][65];
  pdl_wait();
  pdl_trigger();
  if ((int)blockIdx.x == a.xstart[n_layers]) {   // the extra column of blocks
    const int g = blockIdx.y;
    float acc = 0.f;
    for (int b = threadIdx.x; b < B; b += blockDim.x) acc += lo.row_loss[(int64_t)g * B + b];
    acc = block_sum(acc, &part[0][0]);
    if (threadIdx.x == 0) lo.loss_out[(int64_t)g * lo.out_stride + lo.k] = acc / (float)B;
    return;
  }
  int li = 0;
  while (li + 1 < n_layers && (int)blockIdx.x >= a.xstart[li + 1]) ++li;
  const BiasSgdLayer<T> L = a.layer[li];
  const int g = blockIdx.y, bx = blockIdx.x - a.xstart[li];
  const int cx = threadIdx.x & 7, ry = threadIdx.x >> 3;
  const int c0 = bx * 64 + cx * 8;
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  if (c0 < L.ld) {
    const T* d = L.delta + (int64_t)g * L.sg + c0;
#pragma unroll 8
    for (int b = ry; b < B; b += 32) {
      float v[8];
      load8(d + (int64_t)b * L.ld, v);
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] += v[e];
    }
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) part[ry][cx * 8 + e] = acc[e];
  __syncthreads();
  if (threadIdx.x < 64) {
    const int col = bx * 64 + threadIdx.x;
    if (col < L.n) {
      float s = 0.f;
#pragma unroll
      for (int u = 0; u < 32; ++u) s += part[u][threadIdx.x];
      L.bias[(int64_t)g * L.bias_sg + col] -= lr * s;
    }
  }
}

// lse[g][b] = log sum_n exp(z[g][b][n]) from per-tile partials (m, s) = (max of z * log2(e),
// sum of 2^(z * log2(e) - m)).  Block: 32 rows x 32 partial lanes; partials of one index are
// contiguous over rows.
__global__ void __launch_bounds__(1024) lse_combine_kernel(const float2* __restrict__ part, int parts, int B,
                                                            int64_t lse_sg, float* __restrict__ lse,
                                                            const int32_t* __restrict__ y, int64_t y_sg, int Nt,
                                                            DeviceStatus* st) {
  __shared__ float sm[32][33], ss[32][33];
  pdl_wait();
  pdl_trigger();
  const int g = blockIdx.y;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int b = blockIdx.x * 32 + tx;
  float m = -INFINITY, s = 0.f;
  if (b < B) {
    const float2* p = part + (int64_t)g * parts * B + b;
    // eight partials are requested before the first is folded in: a very wide layer has ten
    // thousand of them per row and only a few dozen blocks to read them
    constexpr int kAhead = 8;
    for (int i0 = ty; i0 < parts; i0 += 32 * kAhead) {
      float2 v[kAhead];
#pragma unroll
      for (int u = 0; u < kAhead; ++u) {
        const int i = i0 + 32 * u;
        v[u] = i < parts ? p[(int64_t)i * B] : make_float2(-INFINITY, 0.f);
      }
#pragma unroll
      for (int u = 0; u < kAhead; ++u) {
        if (v[u].x > -INFINITY) {                  // an empty partial carries (-inf, 0)
          const float mn = fmaxf(m, v[u].x);
          s = s * exp2f(m - mn) + v[u].y * exp2f(v[u].x - mn);
          m = mn;
        }
      }
    }
  }
  sm[ty][tx] = m;
  ss[ty][tx] = s;
  __syncthreads();
  if (ty == 0 && b < B) {
    float M = -INFINITY;
    for (int u = 0; u < 32; ++u) M = fmaxf(M, sm[u][tx]);
    float S = 0.f;
    for (int u = 0; u < 32; ++u)
      if (sm[u][tx] > -INFINITY) S += ss[u][tx] * exp2f(sm[u][tx] - M);
    lse[(int64_t)g * lse_sg + b] = (M + log2f(S)) * 0.6931471805599453f;
    const int label = y[(int64_t)g * y_sg + b];
    if (label < 0 || label >= Nt) report(st, -5, SITE_LABEL, (long long)g * B + b);
  }
}

__global__ void lse_row_loss_kernel(const float* __restrict__ lse, const float* __restrict__ zy, int B, int64_t lse_sg,
                                    float* __restrict__ row_loss) {
  pdl_wait();
  pdl_trigger();
  const int g = blockIdx.y, b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b < B) row_loss[(int64_t)g * B + b] = lse[(int64_t)g * lse_sg + b] - zy[(int64_t)g * lse_sg + b];
}

template <typename T>
__global__ void stage_rows_kernel(const float* __restrict__ X, int64_t N0, int64_t group_row_stride,
                                  int B, T* __restrict__ out, int64_t ld, int64_t sg) {
  pdl_wait();
  pdl_trigger();
  int g = blockIdx.z, b = blockIdx.y;
  int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= ld) return;
  float v = j < N0 ? X[((int64_t)g * group_row_stride + b) * N0 + j] : 0.f;
  out[(int64_t)g * sg + (int64_t)b * ld + j] = from_float<T>(v);
}

__global__ void eval_rows_kernel(const float* __restrict__ logits, int64_t ld, int rows, int Nt,
                                 const int32_t* __restrict__ y, double* loss_sum, long long* correct,
                                 DeviceStatus* st) {
  __shared__ float sh[32];
  __shared__ int shi[32];
  int r = blockIdx.x;
  const float* z = logits + (int64_t)r * ld;
  int label = y[r];
  if (label < 0 || label >= Nt) {
    if (threadIdx.x == 0) report(st, -5, SITE_LABEL, r);
    label = 0;
  }
  float mx = -INFINITY;
  int arg = 0x7fffffff;
  for (int n = threadIdx.x; n < Nt; n += blockDim.x) {
    float v = z[n];
    if (v > mx) { mx = v; arg = n; }   // first maximum inside the thread's strided set
  }
  // arg-max with lowest index on ties
  for (int o = 16; o; o >>= 1) {
    float om = __shfl_xor_sync(0xffffffffu, mx, o);
    int oa = __shfl_xor_sync(0xffffffffu, arg, o);
    if (om > mx || (om == mx && oa < arg)) { mx = om; arg = oa; }
  }
  int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  if (l == 0) { sh[w] = mx; shi[w] = arg; }
  __syncthreads();
  if (w == 0) {
    float m2 = l < (blockDim.x >> 5) ? sh[l] : -INFINITY;
    int a2 = l < (blockDim.x >> 5) ? shi[l] : 0x7fffffff;
    for (int o = 16; o; o >>= 1) {
      float om = __shfl_xor_sync(0xffffffffu, m2, o);
      int oa = __shfl_xor_sync(0xffffffffu, a2, o);
      if (om > m2 || (om == m2 && oa < a2)) { m2 = om; a2 = oa; }
    }
    if (l == 0) { sh[0] = m2; shi[0] = a2; }
  }
  __syncthreads();
  mx = sh[0];
  arg = shi[0];
  float se = 0.f;
  for (int n = threadIdx.x; n < Nt; n += blockDim.x) se += expf(z[n] - mx);
  se = block_sum(se, sh);
  if (threadIdx.x == 0) {
    atomicAdd(loss_sum, (double)(logf(se) + mx - z[label]));
    if (arg == label) atomicAdd((unsigned long long*)correct, 1ull);
  }
}

__global__ void eval_finalize_kernel(const double* loss_sum, const long long* correct, int64_t n,
                                     float* mean_loss_out, int64_t* correct_out) {
  *mean_loss_out = (float)(*loss_sum / (double)n);
  *correct_out = (int64_t)*correct;
}

template <typename T>
__global__ void splitk_mask_reduce_kernel(const float* __restrict__ part, int ks, int B, int64_t ld,
                                          const T* __restrict__ mask, int64_t mask_sg, T* __restrict__ out,
                                          int64_t out_sg) {
  pdl_wait();
  pdl_trigger();
  const int g = blockIdx.y;
  const int64_t per = (int64_t)B * ld;
  for (int64_t e = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4; e < per;
       e += (int64_t)gridDim.x * blockDim.x * 4) {
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < ks; ++s) {   // fixed order
      float4 v = *reinterpret_cast<const float4*>(part + ((int64_t)g * ks + s) * per + e);
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    const T* m = mask + (int64_t)g * mask_sg + e;
    T* o = out + (int64_t)g * out_sg + e;
    o[0] = from_float<T>(to_float(m[0]) > 0.f ? acc.x : 0.f);
    o[1] = from_float<T>(to_float(m[1]) > 0.f ? acc.y : 0.f);
    o[2] = from_float<T>(to_float(m[2]) > 0.f ? acc.z : 0.f);
    o[3] = from_float<T>(to_float(m[3]) > 0.f ? acc.w : 0.f);
  }
}

int row_threads(int Nt) { return Nt <= 64 ? 32 : (Nt <= 1024 ? 128 : kThreads); }

}  // namespace

template <typename T>
void softmax_xent(const Launch& L, const float* logits, int64_t ld, int64_t sg, int G, int B, int Nt,
                  const int32_t* y, int64_t y_sg, T* delta, int64_t ld_d, int64_t sg_d,
                  float* row_loss, DeviceStatus* st) {
  if (Nt > 8192 && ld % 4 == 0 && ld_d % 4 == 0)
    launch_pdl(softmax_xent_wide_kernel<T>, dim3(B, G), dim3(512), 0, L.stream, logits, ld, sg, B, Nt, y, y_sg, delta,
               ld_d, sg_d, row_loss, st);
  else
    launch_pdl(softmax_xent_kernel<T>, dim3(B, G), dim3(row_threads(Nt)), 0, L.stream, logits, ld, sg, B, Nt, y, y_sg,
               delta, ld_d, sg_d, row_loss, st);
  L.count();
}
template void softmax_xent<float>(const Launch&, const float*, int64_t, int64_t, int, int, int,
                                  const int32_t*, int64_t, float*, int64_t, int64_t, float*,
                                  DeviceStatus*);
template void softmax_xent<bf16>(const Launch&, const float*, int64_t, int64_t, int, int, int,
                                 const int32_t*, int64_t, bf16*, int64_t, int64_t, float*,
                                 DeviceStatus*);

template <typename T>
void splitk_mask_reduce(const Launch& L, const float* part, int ks, int G, int B, int64_t ld, const T* mask,
                        int64_t mask_sg, T* out, int64_t out_sg) {
  const int64_t vecs = (int64_t)B * ld / 4;
  dim3 grid((unsigned)std::min<int64_t>(ceil_div(vecs, 256), 1024), G);
  launch_pdl(splitk_mask_reduce_kernel<T>, grid, dim3(256), 0, L.stream, part, ks, B, ld, mask, mask_sg, out, out_sg);
  L.count();
}
template void splitk_mask_reduce<bf16>(const Launch&, const float*, int, int, int, int64_t, const bf16*, int64_t,
                                       bf16*, int64_t);

template <typename T>
void softmax_xent_small(const Launch& L, const float* part, int ks, int64_t ld, int G, int B, int Nt,
                        const float* bias, int64_t bias_sg, const int32_t* y, int64_t y_sg, T* delta, int64_t ld_d,
                        int64_t sg_d, float* row_loss, DeviceStatus* st) {
  launch_pdl(softmax_xent_small_kernel<T>, dim3((unsigned)ceil_div(B, 8), G), dim3(256), 0, L.stream, part, ks, ld, B, Nt,
             bias, bias_sg, y, y_sg, delta, ld_d, sg_d, row_loss, st);
  L.count();
}
template void softmax_xent_small<bf16>(const Launch&, const float*, int, int64_t, int, int, int, const float*, int64_t,
                                       const int32_t*, int64_t, bf16*, int64_t, int64_t, float*, DeviceStatus*);

void lse_combine(const Launch& L, const float* lse_part, int parts, int G, int B, int64_t lse_sg, float* lse,
                 const int32_t* y, int64_t y_sg, int Nt, DeviceStatus* st) {
  launch_pdl(lse_combine_kernel, dim3((unsigned)ceil_div(B, 32), G), dim3(1024), 0, L.stream,
             reinterpret_cast<const float2*>(lse_part), parts, B, lse_sg, lse, y, y_sg, Nt, st);
  L.count();
}

void lse_row_loss(const Launch& L, const float* lse, const float* label_logit, int G, int B, int64_t lse_sg,
                  float* row_loss) {
  launch_pdl(lse_row_loss_kernel, dim3((unsigned)ceil_div(B, 256), G), dim3(256), 0, L.stream, lse, label_logit, B,
             lse_sg, row_loss);
  L.count();
}

template <typename T>
void bias_sgd(const Launch& L, const BiasSgdArgs<T>& a, int n_layers, int G, int B, float lr, const LossReduce& loss) {
  BiasSgdArgs<T> b = a;
  b.xstart[0] = 0;
  for (int i = 0; i < n_layers; ++i) b.xstart[i + 1] = b.xstart[i] + (int)ceil_div(a.layer[i].ld, 64);
  launch_pdl(bias_sgd_kernel<T>, dim3((unsigned)b.xstart[n_layers] + (loss.loss_out ? 1 : 0), G), dim3(256), 0, L.stream, b,
             n_layers, B, lr, loss);
  L.count();
}
template void bias_sgd<float>(const Launch&, const BiasSgdArgs<float>&, int, int, int, float, const LossReduce&);
template void bias_sgd<bf16>(const Launch&, const BiasSgdArgs<bf16>&, int, int, int, float, const LossReduce&);

template <typename T>
void stage_rows(const Launch& L, const float* X, int64_t N0, int64_t group_row_stride, int G, int B,
                T* out, int64_t ld, int64_t sg) {
  launch_pdl(stage_rows_kernel<T>, dim3((unsigned)ceil_div(ld, 256), B, G), dim3(256), 0, L.stream, X, N0,
             group_row_stride, B, out, ld, sg);
  L.count();
}
template void stage_rows<float>(const Launch&, const float*, int64_t, int64_t, int, int, float*,
                                int64_t, int64_t);
template void stage_rows<bf16>(const Launch&, const float*, int64_t, int64_t, int, int, bf16*,
                               int64_t, int64_t);

void eval_rows(const Launch& L, const float* logits, int64_t ld, int rows, int Nt, const int32_t* y,
               double* loss_sum, long long* correct, DeviceStatus* st) {
  eval_rows_kernel<<<rows, row_threads(Nt), 0, L.stream>>>(logits, ld, rows, Nt, y, loss_sum, correct,
                                                           st);
  L.count();
}

void eval_finalize(const Launch& L, const double* loss_sum, const long long* correct, int64_t n,
                   float* mean_loss_out, int64_t* correct_out) {
  eval_finalize_kernel<<<1, 1, 0, L.stream>>>(loss_sum, correct, n, mean_loss_out, correct_out);
  L.count();
}

}  // namespace ist
