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

}  // namespace

template <typename T>
void gemm_simt(const Launch& L, const GemmArgs<T>& a) {
  if (a.M <= 0 || a.N <= 0 || a.G <= 0) return;
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
