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
  dim3 grid((unsigned)ceil_div(m.ld, kThreads), (unsigned)ceil_div(m.rows_pad, kRowsPerCta), S);
  gather_kernel<<<grid, kThreads, 0, L.stream>>>(W, m, master, opw);
  L.count();
}

void scatter_slices(const Launch& L, float* W, const SliceMap& m, int S, const float* master) {
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
