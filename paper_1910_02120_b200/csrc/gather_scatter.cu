// Partition-indexed gather / scatter of weight slices between the full network and the
// per-subnet packed buffers (paper Sec. 2.1 "Constructing Subnets": a subnet's weights are the
// entries whose row and column neurons it owns; "Training Subnets": the trained slices go back
// to the positions they came from).  Pure data movement:
// fp32 values are moved bit for bit; the bf16 operand copy is a rounding of the moved value.
#include <algorithm>
#include <mutex>

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
  int s = m.s_first + blockIdx.z;
  int64_t j = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  if (j >= m.ld) return;
  int64_t ncols = m.col_idx ? (m.col_off[s + 1] - m.col_off[s]) : m.full_cols;
  int64_t nrows = m.row_idx ? (m.row_off[s + 1] - m.row_off[s]) : m.full_rows;
  int64_t c = -1;
  if (j < ncols) c = m.col_idx ? m.col_idx[m.col_off[s] + j] : j;
  // row blocks blockIdx.y, blockIdx.y + gridDim.y, ... (the y dimension of a grid stops at 65535)
  for (int64_t i0 = (int64_t)blockIdx.y * kRowsPerCta; i0 < m.rows_pad; i0 += (int64_t)gridDim.y * kRowsPerCta) {
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
}

__global__ void scatter_kernel(float* __restrict__ W, SliceMap m, const float* __restrict__ master) {
  int s = m.s_first + blockIdx.z;
  int64_t j = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  int64_t ncols = m.col_idx ? (m.col_off[s + 1] - m.col_off[s]) : m.full_cols;
  int64_t nrows = m.row_idx ? (m.row_off[s + 1] - m.row_off[s]) : m.full_rows;
  if (j >= ncols) return;
  int64_t c = m.col_idx ? m.col_idx[m.col_off[s] + j] : j;
  for (int64_t i0 = (int64_t)blockIdx.y * kRowsPerCta; i0 < nrows; i0 += (int64_t)gridDim.y * kRowsPerCta) {
#pragma unroll
    for (int u = 0; u < kRowsPerCta; ++u) {
      int64_t i = i0 + u;
      if (i < nrows) {
        int64_t r = m.row_idx ? m.row_idx[m.row_off[s] + i] : i;
        W[r * m.full_cols + c] = master[((int64_t)s * m.rows_pad + i) * m.ld + j];
      }
    }
  }
}

// ---- last layer: whole rows, picked by the previous hidden layer's partition --------------------
// W_t[G_{t-1}^s, :] keeps every column, so both sides are contiguous along a row and the kernel is a
// strided row copy.  Rows of the full matrix start at any 4-byte offset (N_t is arbitrary), hence
// scalar accesses; a thread keeps kRowU x kColU of them in flight (consecutive lanes on
// consecutive columns), which is what the copy needs to approach the DRAM rate.
constexpr int kRowU = 4, kColU = 4;

template <bool GATHER>
__global__ void __launch_bounds__(kThreads) rows_kernel(float* __restrict__ W, SliceMap m, float* __restrict__ master,
                                                         bf16* __restrict__ opw) {
  const int s = m.s_first + blockIdx.z;
  const int nrows = m.row_off[s + 1] - m.row_off[s];
  const int32_t* rows = m.row_idx + m.row_off[s];
  const int64_t j0 = (int64_t)blockIdx.x * (kThreads * kColU) + threadIdx.x;
  for (int64_t i0 = (int64_t)blockIdx.y * kRowU; i0 < (GATHER ? m.rows_pad : nrows); i0 += (int64_t)gridDim.y * kRowU) {
    float v[kRowU][kColU];
    int64_t src[kRowU];
#pragma unroll
    for (int u = 0; u < kRowU; ++u) src[u] = (i0 + u < nrows) ? (int64_t)rows[i0 + u] * m.full_cols : -1;
    if (GATHER) {
#pragma unroll
      for (int u = 0; u < kRowU; ++u)
#pragma unroll
        for (int c = 0; c < kColU; ++c) {
          const int64_t j = j0 + c * kThreads;
          v[u][c] = (src[u] >= 0 && j < m.full_cols) ? __ldg(W + src[u] + j) : 0.f;   // pad rows / columns are zeros
        }
#pragma unroll
      for (int u = 0; u < kRowU; ++u)
#pragma unroll
        for (int c = 0; c < kColU; ++c) {
          const int64_t j = j0 + c * kThreads;
          if (i0 + u < m.rows_pad && j < m.ld) {
            const int64_t o = ((int64_t)s * m.rows_pad + i0 + u) * m.ld + j;
            master[o] = v[u][c];
            if (opw) opw[o] = __float2bfloat16_rn(v[u][c]);
          }
        }
    } else {
#pragma unroll
      for (int u = 0; u < kRowU; ++u)
#pragma unroll
        for (int c = 0; c < kColU; ++c) {
          const int64_t j = j0 + c * kThreads;
          v[u][c] = (src[u] >= 0 && j < m.full_cols) ? __ldg(master + ((int64_t)s * m.rows_pad + i0 + u) * m.ld + j) : 0.f;
        }
#pragma unroll
      for (int u = 0; u < kRowU; ++u)
#pragma unroll
        for (int c = 0; c < kColU; ++c) {
          const int64_t j = j0 + c * kThreads;
          if (src[u] >= 0 && j < m.full_cols) W[src[u] + j] = v[u][c];
        }
    }
  }
}

bool rows_ok(const SliceMap& m) { return m.row_idx && !m.col_idx && m.full_cols >= 1024; }

template <bool GATHER>
void launch_rows(const Launch& L, float* W, const SliceMap& m, int S, float* master, bf16* opw) {
  dim3 grid((unsigned)ceil_div(m.ld, kThreads * kColU), (unsigned)std::min<int64_t>(ceil_div(m.rows_pad, kRowU), 65535), S);
  rows_kernel<GATHER><<<grid, kThreads, 0, L.stream>>>(W, m, master, opw);
  L.count();
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

struct ColRuns {                 // per group moved (m.s_first + i): packed positions [lo, lo + cnt) fall in the chunk
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
    const int s = m.s_first + threadIdx.x;
    const int32_t* g = m.col_idx + m.col_off[s];
    const int n = m.col_off[s + 1] - m.col_off[s];
    const int lo = lower_bound_idx(g, n, c0);
    runs->lo[threadIdx.x] = lo;
    runs->pre[threadIdx.x + 1] = lower_bound_idx(g, n, c1) - lo;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    runs->pre[0] = 0;
    for (int s = 0; s < S; ++s) runs->pre[s + 1] += runs->pre[s];
  }
  __syncthreads();
}

// ---- bulk-copy helpers (one thread moves whole row segments asynchronously) -------------------
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void bar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void bar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool bar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_addr(dst_smem)), "l"(src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void bulk_store(void* dst, const void* src_smem, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
               ::"l"(dst), "r"(smem_addr(src_smem)), "r"(bytes) : "memory");
}

constexpr int kPermThreads = 512;
constexpr long long kPermWaitCycles = 2000000000ll;   // ~1 s

// Persistent CTA: column chunk blockIdx.x, row blocks blockIdx.y, blockIdx.y + gridDim.y, ...
// The map from a packed position of the chunk to (column inside the chunk, offset in the packed
// buffer) depends on the chunk only, so it is built once and reused for every row block.
// Gather: row blocks arrive through double-buffered bulk copies (the next block loads while
// this one is permuted).  Scatter: packed values are read into the permuted tile, which leaves
// through bulk stores.  Requires full_cols % 4 == 0 (16-byte row segments).
template <bool GATHER>
__global__ void __launch_bounds__(kPermThreads, 1) permute_cols_kernel(float* __restrict__ W, SliceMap m, int S,
                                                                      float* __restrict__ master,
                                                                      bf16* __restrict__ opw, DeviceStatus* st) {
  extern __shared__ __align__(128) unsigned char perm_smem[];
  float* tile = reinterpret_cast<float*>(perm_smem);                                  // [2][rows][cols]
  long long* map_off = reinterpret_cast<long long*>(tile + 2 * kStageRows * kStageCols);   // [cols]
  uint16_t* map_col = reinterpret_cast<uint16_t*>(map_off + kStageCols);                   // [cols]
  __shared__ ColRuns runs;
  __shared__ uint64_t full[2];
  const int c0 = blockIdx.x * kStageCols;
  const int c1 = min((int)m.full_cols, c0 + kStageCols);
  const int width = c1 - c0;
  const int64_t n_blocks = ceil_div(m.full_rows, kStageRows);
  if (threadIdx.x == 0) {
    bar_init(&full[0], 1);
    bar_init(&full[1], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  find_runs(m, S, c0, c1, &runs);      // contains the barriers that publish the mbarrier init
  const int total = runs.pre[S];
  for (int e = threadIdx.x; e < total; e += kPermThreads) {
    int i = 0;
    while (e >= runs.pre[i + 1]) ++i;
    const int s = m.s_first + i;
    const int j = runs.lo[i] + (e - runs.pre[i]);
    map_col[e] = (uint16_t)(m.col_idx[m.col_off[s] + j] - c0);
    map_off[e] = (long long)s * m.rows_pad * m.ld + j;
  }
  __syncthreads();

  auto issue_load = [&](int64_t rb, int buf) {   // thread 0 only
    const int64_t k0 = rb * kStageRows;
    const int nrows = (int)min((long long)kStageRows, (long long)(m.full_rows - k0));
    bar_expect_tx(&full[buf], (uint32_t)(nrows * width * 4));
    for (int r = 0; r < nrows; ++r)
      bulk_load(tile + (buf * kStageRows + r) * kStageCols, W + (k0 + r) * m.full_cols + c0, (uint32_t)(width * 4),
                &full[buf]);
  };

  if (GATHER && threadIdx.x == 0 && blockIdx.y < n_blocks) issue_load(blockIdx.y, 0);
  int it = 0;
  for (int64_t rb = blockIdx.y; rb < n_blocks; rb += gridDim.y, ++it) {
    const int buf = it & 1;
    const int64_t k0 = rb * kStageRows;
    const int nrows = (int)min((long long)kStageRows, (long long)(m.full_rows - k0));
    float* t = tile + buf * kStageRows * kStageCols;
    if (GATHER) {
      // the other buffer was last read in the previous iteration, which ended with a barrier
      if (threadIdx.x == 0 && rb + gridDim.y < n_blocks) issue_load(rb + gridDim.y, buf ^ 1);
      bool ok = true;
      const long long t0 = clock64();
      while (!bar_try_wait(&full[buf], (it >> 1) & 1)) {
        if (clock64() - t0 > kPermWaitCycles) { ok = false; break; }
      }
      if (!__syncthreads_and(ok)) {
        if (threadIdx.x == 0) report(st, -6, SITE_TC_PIPE, 100);
        return;
      }
      for (int e = threadIdx.x; e < total; e += kPermThreads) {
        const int col = map_col[e];
        const long long o = map_off[e] + k0 * m.ld;
#pragma unroll
        for (int r = 0; r < kStageRows; ++r) {
          if (r < nrows) {
            const float v = t[r * kStageCols + col];
            master[o + (long long)r * m.ld] = v;
            if (opw) opw[o + (long long)r * m.ld] = __float2bfloat16_rn(v);
          }
        }
      }
      if (blockIdx.x == 0) {   // pad columns [|G^s|, ld) of these rows are zero
        for (int s = m.s_first; s < m.s_first + S; ++s) {
          const int cnt = m.col_off[s + 1] - m.col_off[s];
          const int npad = (int)m.ld - cnt;
          for (int e = threadIdx.x; e < npad * nrows; e += kPermThreads) {
            const long long o = ((long long)s * m.rows_pad + k0 + e / npad) * m.ld + cnt + e % npad;
            master[o] = 0.f;
            if (opw) opw[o] = __float2bfloat16_rn(0.f);
          }
        }
      }
      __syncthreads();
    } else {
      // this buffer's previous stores (two iterations ago) must have read it
      if (threadIdx.x == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
      __syncthreads();
      for (int e = threadIdx.x; e < total; e += kPermThreads) {
        const int col = map_col[e];
        const long long o = map_off[e] + k0 * m.ld;
        float v[kStageRows];
#pragma unroll
        for (int r = 0; r < kStageRows; ++r) v[r] = r < nrows ? master[o + (long long)r * m.ld] : 0.f;
#pragma unroll
        for (int r = 0; r < kStageRows; ++r) t[r * kStageCols + col] = v[r];
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncthreads();
      if (threadIdx.x == 0) {
        for (int r = 0; r < nrows; ++r)
          bulk_store(W + (k0 + r) * m.full_cols + c0, t + r * kStageCols, (uint32_t)(width * 4));
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      }
    }
  }
  if (!GATHER && threadIdx.x == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

bool staged_ok(const SliceMap& m, int S) {
  return !m.row_idx && m.col_idx && m.full_rows >= kStageRows && S <= kMaxGroupsStaged &&
         m.full_cols >= 256 && m.full_cols % 4 == 0;
}

template <bool GATHER>
bool launch_permute_cols(const Launch& L, float* W, const SliceMap& m, int S, float* master, bf16* opw,
                         DeviceStatus* st) {
  constexpr int smem = 2 * kStageRows * kStageCols * (int)sizeof(float) + kStageCols * 8 + kStageCols * 2;
  static std::once_flag once;     // one instance per direction; any host thread may come first
  static bool configured = false;
  std::call_once(once, [] {
    configured = cudaFuncSetAttribute(permute_cols_kernel<GATHER>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      smem) == cudaSuccess;
  });
  if (!configured) return false;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int64_t chunks = ceil_div(m.full_cols, kStageCols), blocks = ceil_div(m.full_rows, kStageRows);
  int64_t y = sms / chunks;
  if (y < 1) y = 1;
  if (y > blocks) y = blocks;
  if (y > 65535) y = 65535;
  dim3 grid((unsigned)chunks, (unsigned)y);
  permute_cols_kernel<GATHER><<<grid, kPermThreads, smem, L.stream>>>(W, m, S, master, opw, st);
  L.count();
  return true;
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
                   bf16* opw, DeviceStatus* st) {
  if (staged_ok(m, S) && launch_permute_cols<true>(L, const_cast<float*>(W), m, S, master, opw, st)) return;
  if (rows_ok(m)) return launch_rows<true>(L, const_cast<float*>(W), m, S, master, opw);
  dim3 grid((unsigned)ceil_div(m.ld, kThreads), (unsigned)std::min<int64_t>(ceil_div(m.rows_pad, kRowsPerCta), 65535), S);
  gather_kernel<<<grid, kThreads, 0, L.stream>>>(W, m, master, opw);
  L.count();
}

void scatter_slices(const Launch& L, float* W, const SliceMap& m, int S, const float* master,
                    DeviceStatus* st) {
  if (staged_ok(m, S) && launch_permute_cols<false>(L, W, m, S, const_cast<float*>(master), nullptr, st)) return;
  if (rows_ok(m)) return launch_rows<false>(L, W, m, S, const_cast<float*>(master), nullptr);
  dim3 grid((unsigned)ceil_div(m.ld, kThreads), (unsigned)std::min<int64_t>(ceil_div(m.rows_pad, kRowsPerCta), 65535), S);
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
