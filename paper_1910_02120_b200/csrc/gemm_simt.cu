// Grouped GEMM on the CUDA cores with fused epilogues: the fp32 path of the local steps
// (forward, backward and SGD update of all S subnets; paper Sec. 2.1 "Training Subnets",
// App. A Eq. (2) on the slices) and the full-width evaluation pass.
//
// C[g](m, n) = sum_k A[g](m, k) * B[g](n, k) with arbitrary element strides, so the same
// kernel serves x*W (B is n-contiguous), delta*W^T (B is k-contiguous) and a^T*delta
// (both operands contiguous along m / n).  64x64 output tile (4x4 per thread) or, when that
// would leave most SMs without a tile, 32x32 (2x2 per thread); 16-deep k slabs.
#include "kernels.h"

namespace ist {
namespace {

constexpr int BK = 16, kThreads = 256;

template <typename T>
__device__ __forceinline__ void epilogue_store(const GemmArgs<T>& a, int g, int m, int n, float c) {
  switch (a.epi) {
    case EPI_BIAS_RELU: {
      float v = c + a.bias[(int64_t)g * a.bias_sg + n];
      a.out[(int64_t)g * a.out_sg + (int64_t)m * a.out_ld + n] = from_float<T>(fmaxf(v, 0.f));
      break;
    }
    case EPI_BIAS_F32: {
      a.outf[(int64_t)g * a.outf_sg + (int64_t)m * a.outf_ld + n] =
          c + a.bias[(int64_t)g * a.bias_sg + n];
      break;
    }
    case EPI_RELU_MASK: {
      float mk = to_float(a.mask[(int64_t)g * a.mask_sg + (int64_t)m * a.mask_ld + n]);
      a.out[(int64_t)g * a.out_sg + (int64_t)m * a.out_ld + n] = from_float<T>(mk > 0.f ? c : 0.f);
      break;
    }
    case EPI_SGD: {
      int64_t o = (int64_t)g * a.outf_sg + (int64_t)m * a.outf_ld + n;
      float w = a.outf[o] - a.lr * c;
      a.outf[o] = w;
      if (a.opw) a.opw[o] = __float2bfloat16_rn(w);
      break;
    }
    default: {
      a.out[(int64_t)g * a.out_sg + (int64_t)m * a.out_ld + n] = from_float<T>(c);
      break;
    }
  }
}

template <typename T, int BM, int BN>
__global__ void __launch_bounds__(kThreads) gemm_simt_kernel(GemmArgs<T> a) {
  constexpr int TM = BM / 16, TN = BN / 16;      // outputs per thread
  __shared__ float As[BK][BM + 1];
  __shared__ float Bs[BK][BN + 1];
  // blockIdx.x runs over (m tile, n tile) pairs, n fastest: the x dimension of a grid has room
  // for 2^31 - 1 blocks, the y dimension only for 65535
  const int g = blockIdx.z;
  const int n_tiles = (a.N + BN - 1) / BN;
  const int m0 = (int)(blockIdx.x / n_tiles) * BM, n0 = (int)(blockIdx.x % n_tiles) * BN;
  const int tid = threadIdx.x;
  const int ty = tid / 16, tx = tid % 16;
  const T* A = a.A + (int64_t)g * a.a_sg;
  const T* B = a.B + (int64_t)g * a.b_sg;
  const bool a_kmajor = a.a_sk == 1, b_kmajor = a.b_sk == 1;

  float acc[TM][TN];
#pragma unroll
  for (int u = 0; u < TM; ++u)
#pragma unroll
    for (int v = 0; v < TN; ++v) acc[u][v] = 0.f;

  // the next k slab is fetched into registers while the current one is multiplied
  constexpr int NA = BM * BK / kThreads, NB = BN * BK / kThreads;
  float ra[NA], rb[NB];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int u = 0; u < NA; ++u) {
      int e = tid + kThreads * u;
      int kk = a_kmajor ? e % BK : e / BM;
      int mm = a_kmajor ? e / BK : e % BM;
      int m = m0 + mm, k = k0 + kk;
      ra[u] = (m < a.M && k < a.K) ? to_float(A[(int64_t)m * a.a_sm + (int64_t)k * a.a_sk]) : 0.f;
    }
#pragma unroll
    for (int u = 0; u < NB; ++u) {
      int e = tid + kThreads * u;
      int kk = b_kmajor ? e % BK : e / BN;
      int nn = b_kmajor ? e / BK : e % BN;
      int n = n0 + nn, k = k0 + kk;
      rb[u] = (n < a.N && k < a.K) ? to_float(B[(int64_t)n * a.b_sn + (int64_t)k * a.b_sk]) : 0.f;
    }
  };
  fetch(0);
  for (int k0 = 0; k0 < a.K; k0 += BK) {
#pragma unroll
    for (int u = 0; u < NA; ++u) {
      int e = tid + kThreads * u;
      As[a_kmajor ? e % BK : e / BM][a_kmajor ? e / BK : e % BM] = ra[u];
    }
#pragma unroll
    for (int u = 0; u < NB; ++u) {
      int e = tid + kThreads * u;
      Bs[b_kmajor ? e % BK : e / BN][b_kmajor ? e / BK : e % BN] = rb[u];
    }
    __syncthreads();
    if (k0 + BK < a.K) fetch(k0 + BK);
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float av[TM], bv[TN];
#pragma unroll
      for (int u = 0; u < TM; ++u) av[u] = As[kk][ty + 16 * u];
#pragma unroll
      for (int v = 0; v < TN; ++v) bv[v] = Bs[kk][tx + 16 * v];
#pragma unroll
      for (int u = 0; u < TM; ++u)
#pragma unroll
        for (int v = 0; v < TN; ++v) acc[u][v] = fmaf(av[u], bv[v], acc[u][v]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int u = 0; u < TM; ++u) {
    int m = m0 + ty + 16 * u;
    if (m >= a.M) continue;
#pragma unroll
    for (int v = 0; v < TN; ++v) {
      int n = n0 + tx + 16 * v;
      if (n < a.N) epilogue_store(a, g, m, n, acc[u][v]);
    }
  }
}

// The x*W shape of the forward pass (A contiguous along k, B contiguous along n) in fp32 at sizes
// where tiles of 128 x 128 fill the GPU: the full-width evaluation pass and the wide layers of the
// fp32 path.  8 x 8 outputs per thread (rows ty*4..+3 and 64+ty*4..+3, columns likewise), 8-deep
// k slabs held in shared memory with A transposed, every operand read as a 16-byte vector: 64
// multiply-adds per four shared-memory loads instead of 16 per eight in the kernel above.  The
// next slab is fetched into registers while the current one is multiplied.  Sums run over k in
// ascending order, as above.
template <bool VEC>
__global__ void __launch_bounds__(kThreads) gemm_simt_wide_kernel(GemmArgs<float> a) {
  constexpr int BM = 128, BN = 128, BKW = 8;
  __shared__ __align__(16) float As[BKW][BM + 4];   // + 4: the transposing stores of k and k + 4 miss each other's banks
  __shared__ __align__(16) float Bs[BKW][BN];
  const int g = blockIdx.z;
  const int n_tiles = (a.N + BN - 1) / BN;
  const int m0 = (int)(blockIdx.x / n_tiles) * BM, n0 = (int)(blockIdx.x % n_tiles) * BN;
  const int tid = threadIdx.x, ty = tid / 16, tx = tid % 16;
  const float* A = a.A + (int64_t)g * a.a_sg;
  const float* B = a.B + (int64_t)g * a.b_sg;
  // fetch roles: A rows m0 + tid / 2, four k from (tid % 2) * 4; B row k0 + tid / 32, four n from (tid % 32) * 4
  const int am = m0 + tid / 2, ak = (tid % 2) * 4;
  const int bk = tid / 32, bn = n0 + (tid % 32) * 4;
  float acc[8][8];
#pragma unroll
  for (int u = 0; u < 8; ++u)
#pragma unroll
    for (int v = 0; v < 8; ++v) acc[u][v] = 0.f;
  float ra[4], rb[4];
  auto fetch = [&](int k0) {
    const float* pa = A + (int64_t)am * a.a_sm + k0 + ak;
    const float* pb = B + (int64_t)(k0 + bk) * a.b_sk + bn;
    if (VEC && am < a.M && k0 + ak + 3 < a.K) {
      const float4 t = *reinterpret_cast<const float4*>(pa);
      ra[0] = t.x; ra[1] = t.y; ra[2] = t.z; ra[3] = t.w;
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i) ra[i] = (am < a.M && k0 + ak + i < a.K) ? pa[i] : 0.f;
    }
    if (VEC && k0 + bk < a.K && bn + 3 < a.N) {
      const float4 t = *reinterpret_cast<const float4*>(pb);
      rb[0] = t.x; rb[1] = t.y; rb[2] = t.z; rb[3] = t.w;
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i) rb[i] = (k0 + bk < a.K && bn + i < a.N) ? pb[i] : 0.f;
    }
  };
  fetch(0);
  for (int k0 = 0; k0 < a.K; k0 += BKW) {
#pragma unroll
    for (int i = 0; i < 4; ++i) As[ak + i][tid / 2] = ra[i];
    *reinterpret_cast<float4*>(&Bs[bk][(tid % 32) * 4]) = make_float4(rb[0], rb[1], rb[2], rb[3]);
    __syncthreads();
    if (k0 + BKW < a.K) fetch(k0 + BKW);
#pragma unroll
    for (int kk = 0; kk < BKW; ++kk) {
      const float4 a0 = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
      const float4 a1 = *reinterpret_cast<const float4*>(&As[kk][64 + ty * 4]);
      const float4 b0 = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
      const float4 b1 = *reinterpret_cast<const float4*>(&Bs[kk][64 + tx * 4]);
      const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
      for (int u = 0; u < 8; ++u)
#pragma unroll
        for (int v = 0; v < 8; ++v) acc[u][v] = fmaf(av[u], bv[v], acc[u][v]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    const int m = m0 + (u < 4 ? ty * 4 + u : 64 + ty * 4 + u - 4);
    if (m >= a.M) continue;
#pragma unroll
    for (int v = 0; v < 8; ++v) {
      const int n = n0 + (v < 4 ? tx * 4 + v : 64 + tx * 4 + v - 4);
      if (n < a.N) epilogue_store(a, g, m, n, acc[u][v]);
    }
  }
}

// Launches the wide kernel if the product has its shape and enough tiles; false: not launched.
bool launch_wide(const Launch&, const GemmArgs<bf16>&) { return false; }
bool launch_wide(const Launch& L, const GemmArgs<float>& a) {
  if (a.a_sk != 1 || a.b_sn != 1) return false;
  const int64_t tiles = ceil_div(a.N, 128) * ceil_div(a.M, 128) * a.G;
  if (tiles < 148 || ceil_div(a.N, 128) * ceil_div(a.M, 128) > 0x7fffffffll) return false;
  const bool vec = a.a_sm % 4 == 0 && a.b_sk % 4 == 0 && a.a_sg % 4 == 0 && a.b_sg % 4 == 0 &&
                   reinterpret_cast<uintptr_t>(a.A) % 16 == 0 && reinterpret_cast<uintptr_t>(a.B) % 16 == 0;
  const dim3 grid((unsigned)(ceil_div(a.N, 128) * ceil_div(a.M, 128)), 1, (unsigned)a.G);
  if (vec) gemm_simt_wide_kernel<true><<<grid, kThreads, 0, L.stream>>>(a);
  else gemm_simt_wide_kernel<false><<<grid, kThreads, 0, L.stream>>>(a);
  return true;
}

}  // namespace

template <typename T>
void gemm_simt(const Launch& L, const GemmArgs<T>& a) {
  if (a.M <= 0 || a.N <= 0 || a.G <= 0) return;
  if (launch_wide(L, a)) {
    L.count();
    return;
  }
  // few large tiles leave most of the 148 SMs idle: use 32x32 tiles until every SM has two
  const int64_t big = ceil_div(a.N, 64) * ceil_div(a.M, 64) * a.G;
  if (big >= 296) {
    dim3 grid((unsigned)(ceil_div(a.N, 64) * ceil_div(a.M, 64)), 1, (unsigned)a.G);
    gemm_simt_kernel<T, 64, 64><<<grid, kThreads, 0, L.stream>>>(a);
  } else {
    dim3 grid((unsigned)(ceil_div(a.N, 32) * ceil_div(a.M, 32)), 1, (unsigned)a.G);
    gemm_simt_kernel<T, 32, 32><<<grid, kThreads, 0, L.stream>>>(a);
  }
  L.count();
}

template void gemm_simt<float>(const Launch&, const GemmArgs<float>&);
template void gemm_simt<bf16>(const Launch&, const GemmArgs<bf16>&);

}  // namespace ist
