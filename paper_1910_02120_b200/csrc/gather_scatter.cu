// Partition-indexed gather / scatter of weight slices between the full network and the
// per-subnet packed buffers (paper Sec. 2.1: weights are "partitioned accordingly based on the
// active neurons"; "subnet parameters are copied back into the full NN").  Pure data movement:
// fp32 values are moved bit for bit; the bf16 operand copy is a rounding of the moved value.
#include "kernels.h"

namespace ist {
namespace {

constexpr int kThreads = 256;
constexpr int kRowsPerCta = 8;

// Packed element (s, i, j), j = blockIdx.x*256 + tid, i in a block of kRowsPerCta rows.
// Pad rows / columns (beyond the group's true size) are written as zeros so that padded
// neurons stay inert through the local steps.
__global__ void gather_kernel(const float* __restrict__ W, SliceMap m, float* __restrict__ master,
                              bf16* __restrict__ opw) {
  int s = blockIdx.z;
  int64_t j = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  if (j >= m.ld) return;
  int64_t ncols = m.col_idx ? (m.col_off[s + 1] - m.col_off[s]) : m.full_cols;
  int64_t nrows = m.row_idx ? (m.row_off[s + 1] - m.row_off[s]) : m.full_rows;
  int64_t c = -1;
  if (j < ncols) c = m.col_idx ? m.col_idx[m.col_off[s] + j] : j;
  int64_t i0 = (int64_t)blockIdx.y * kRowsPerCta;
  float v[kRowsPerCta];
#pragma unroll
  for (int u = 0; u < kRowsPerCta; ++u) {
    int64_t i = i0 + u;
    v[u] = 0.f;
    if (c >= 0 && i < nrows) {
      int64_t r = m.row_idx ? m.row_idx[m.row_off[s] + i] : i;
      v[u] = __ldg(W + r * m.full_cols + c);
    }
  }
#pragma unroll
  for (int u = 0; u < kRowsPerCta; ++u) {
    int64_t i = i0 + u;
    if (i < m.rows_pad) {
      int64_t o = ((int64_t)s * m.rows_pad + i) * m.ld + j;
      master[o] = v[u];
      if (opw) opw[o] = __float2bfloat16_rn(v[u]);
    }
  }
}

__global__ void scatter_kernel(float* __restrict__ W, SliceMap m, const float* __restrict__ master) {
  int s = blockIdx.z;
  int64_t j = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  int64_t ncols = m.col_idx ? (m.col_off[s + 1] - m.col_off[s]) : m.full_cols;
  int64_t nrows = m.row_idx ? (m.row_off[s + 1] - m.row_off[s]) : m.full_rows;
  if (j >= ncols) return;
  int64_t c = m.col_idx ? m.col_idx[m.col_off[s] + j] : j;
  int64_t i0 = (int64_t)blockIdx.y * kRowsPerCta;
#pragma unroll
  for (int u = 0; u < kRowsPerCta; ++u) {
    int64_t i = i0 + u;
    if (i < nrows) {
      int64_t r = m.row_idx ? m.row_idx[m.row_off[s] + i] : i;
      W[r * m.full_cols + c] = master[((int64_t)s * m.rows_pad + i) * m.ld + j];
    }
  }
}

// ---- first layer: a column permutation, staged through shared memory -------------------------
// W_1[:, G_1^s] keeps whole rows and permutes their columns.  A CTA stages kStageRows rows x
// kStageCols consecutive columns (coalesced float4 accesses on the full-matrix side); because
// indices ascend inside a group, those columns form one contiguous run [lo_s, hi_s) in every
// group's packed row, so the packed side is coalesced as well.  The permutation itself is a
// random-access read (gather) or write (scatter) in shared memory.
constexpr int kStageRows = 8;
constexpr int kStageCols = 2048;
constexpr int kMaxGroupsStaged = 64;

struct ColRuns {                 // per group: packed positions [lo, lo + cnt) fall in the chunk
  int lo[kMaxGroupsStaged];
  int pre[kMaxGroupsStaged + 1]; // prefix sums of cnt
};

// First packed position of group s whose column index is >= c.
__device__ __forceinline__ int lower_bound_idx(const int32_t* idx, int n, int c) {
  int lo = 0, hi = n;
  while (lo < hi) {
    int mid = (lo + hi) >> 1;
    if (idx[mid] < c) lo = mid + 1; else hi = mid;
  }
  return lo;
}

__device__ __forceinline__ void find_runs(const SliceMap& m, int S, int c0, int c1, ColRuns* runs) {
  if (threadIdx.x < S) {
    const int s = threadIdx.x;
    const int32_t* g = m.col_idx + m.col_off[s];
    const int n = m.col_off[s + 1] - m.col_off[s];
    const int lo = lower_bound_idx(g, n, c0);
    runs->lo[s] = lo;
    runs->pre[s + 1] = lower_bound_idx(g, n, c1) - lo;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    runs->pre[0] = 0;
    for (int s = 0; s < S; ++s) runs->pre[s + 1] += runs->pre[s];
  }
  __syncthreads();
}

template <bool GATHER>
__global__ void __launch_bounds__(256) permute_cols_kernel(float* __restrict__ W, SliceMap m, int S,
                                                          float* __restrict__ master,
                                                          bf16* __restrict__ opw) {
  extern __shared__ float tile[];            // [kStageRows][kStageCols]
  __shared__ ColRuns runs;
  const int c0 = blockIdx.x * kStageCols;
  const int c1 = min((int)m.full_cols, c0 + kStageCols);
  const int width = c1 - c0;
  const int64_t k0 = (int64_t)blockIdx.y * kStageRows;
  const int nrows = (int)min((long long)kStageRows, (long long)(m.full_rows - k0));
  find_runs(m, S, c0, c1, &runs);

  if (GATHER) {
    // full matrix -> shared memory, coalesced (float4 where the row start allows it)
    const bool vec = (m.full_cols % 4 == 0);
    for (int r = 0; r < nrows; ++r) {
      const float* src = W + (k0 + r) * m.full_cols + c0;
      float* dst = tile + r * kStageCols;
      if (vec) {
        for (int v = threadIdx.x; v < width / 4; v += blockDim.x)
          reinterpret_cast<float4*>(dst)[v] = __ldg(reinterpret_cast<const float4*>(src) + v);
      } else {
        for (int v = threadIdx.x; v < width; v += blockDim.x) dst[v] = __ldg(src + v);
      }
    }
    __syncthreads();
  }
  // packed side: flattened over (group, position inside the run); one group's run is contiguous
  const int total = runs.pre[S];
  for (int e = threadIdx.x; e < total; e += blockDim.x) {
    int s = 0;
    while (e >= runs.pre[s + 1]) ++s;
    const int j = runs.lo[s] + (e - runs.pre[s]);
    const int col = m.col_idx[m.col_off[s] + j] - c0;
    const int64_t o = ((int64_t)s * m.rows_pad + k0) * m.ld + j;
    if (GATHER) {
#pragma unroll
      for (int r = 0; r < kStageRows; ++r) {
        if (r < nrows) {
          const float v = tile[r * kStageCols + col];
          master[o + (int64_t)r * m.ld] = v;
          if (opw) opw[o + (int64_t)r * m.ld] = __float2bfloat16_rn(v);
        }
      }
    } else {
#pragma unroll
      for (int r = 0; r < kStageRows; ++r)
        if (r < nrows) tile[r * kStageCols + col] = master[o + (int64_t)r * m.ld];
    }
  }
  if (GATHER) {
    // pad columns [|G^s|, ld) of these rows are zero (first column chunk does it)
    if (blockIdx.x == 0) {
      for (int s = 0; s < S; ++s) {
        const int cnt = m.col_off[s + 1] - m.col_off[s];
        const int npad = (int)m.ld - cnt;
        for (int e = threadIdx.x; e < npad * nrows; e += blockDim.x) {
          const int64_t o = ((int64_t)s * m.rows_pad + k0 + e / npad) * m.ld + cnt + e % npad;
          master[o] = 0.f;
          if (opw) opw[o] = __float2bfloat16_rn(0.f);
        }
      }
    }
  } else {
    __syncthreads();
    const bool vec = (m.full_cols % 4 == 0);
    for (int r = 0; r < nrows; ++r) {
      float* dst = W + (k0 + r) * m.full_cols + c0;
      const float* src = tile + r * kStageCols;
      if (vec) {
        for (int v = threadIdx.x; v < width / 4; v += blockDim.x)
          reinterpret_cast<float4*>(dst)[v] = reinterpret_cast<const float4*>(src)[v];
      } else {
        for (int v = threadIdx.x; v < width; v += blockDim.x) dst[v] = src[v];
      }
    }
  }
}

bool staged_ok(const SliceMap& m, int S) {
  return !m.row_idx && m.col_idx && m.full_rows >= kStageRows && S <= kMaxGroupsStaged &&
         m.full_cols >= 256 && ceil_div(m.full_rows, kStageRows) <= 65535;
}

template <bool GATHER>
void launch_permute_cols(const Launch& L, float* W, const SliceMap& m, int S, float* master, bf16* opw) {
  constexpr int smem = kStageRows * kStageCols * (int)sizeof(float);
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(permute_cols_kernel<GATHER>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    configured = true;
  }
  dim3 grid((unsigned)ceil_div(m.full_cols, kStageCols), (unsigned)ceil_div(m.full_rows, kStageRows));
  permute_cols_kernel<GATHER><<<grid, 256, smem, L.stream>>>(W, m, S, master, opw);
  L.count();
}

__global__ void mean_bias_kernel(float* b, int64_t n, int S, const float* __restrict__ packed,
                                 int64_t ld) {
  int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n) return;
  float old = b[j];
  float acc = 0.f;
  for (int s = 0; s < S; ++s) acc += packed[(int64_t)s * ld + j] - old;
  b[j] = old + acc / (float)S;
}

__global__ void copy_out_kernel(const float* __restrict__ packed, int64_t ld, int64_t rows,
                                int64_t cols, float* __restrict__ out) {
  int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int64_t i = blockIdx.y;
  if (j < cols)
    for (; i < rows; i += gridDim.y) out[i * cols + j] = packed[i * ld + j];
}

}  // namespace

void gather_slices(const Launch& L, const float* W, const SliceMap& m, int S, float* master,
                   bf16* opw) {
  if (staged_ok(m, S)) {
    launch_permute_cols<true>(L, const_cast<float*>(W), m, S, master, opw);
    return;
  }
  dim3 grid((unsigned)ceil_div(m.ld, kThreads), (unsigned)ceil_div(m.rows_pad, kRowsPerCta), S);
  gather_kernel<<<grid, kThreads, 0, L.stream>>>(W, m, master, opw);
  L.count();
}

void scatter_slices(const Launch& L, float* W, const SliceMap& m, int S, const float* master) {
  if (staged_ok(m, S)) {
    launch_permute_cols<false>(L, W, m, S, const_cast<float*>(master), nullptr);
    return;
  }
  dim3 grid((unsigned)ceil_div(m.ld, kThreads), (unsigned)ceil_div(m.rows_pad, kRowsPerCta), S);
  scatter_kernel<<<grid, kThreads, 0, L.stream>>>(W, m, master);
  L.count();
}

void scatter_mean_bias(const Launch& L, float* b, int64_t n, int S, const float* packed, int64_t ld) {
  mean_bias_kernel<<<(unsigned)ceil_div(n, 256), 256, 0, L.stream>>>(b, n, S, packed, ld);
  L.count();
}

void copy_out_slice(const Launch& L, const float* packed, int64_t ld, int64_t rows, int64_t cols,
                    float* out) {
  dim3 grid((unsigned)ceil_div(cols, 256), (unsigned)(rows < 1024 ? rows : 1024));
  copy_out_kernel<<<grid, 256, 0, L.stream>>>(packed, ld, rows, cols, out);
  L.count();
}

}  // namespace ist
