// Grouped bf16 GEMM on the 5th-generation tensor cores (tcgen05.mma, accumulators in tensor
// memory, operands staged in shared memory by TMA) with the local-step epilogues fused in:
// bias + ReLU (forward), logits, ReLU mask (delta back-propagation) and the SGD update of the
// fp32 master slice with its bf16 operand copy (paper Sec. 2.1 "Training Subnets"; App. A
// Eq. (2) on the slices).  All S subnets run as the third grid dimension of one launch.
//
//   C[g](m, n) = sum_k A[g](m, k) * B[g](n, k),   fp32 accumulation
//
// One CTA computes one 128 x BN tile.  Warp 0 (one lane) issues TMA loads into a ring of
// STAGES shared-memory slots; warp 1 (one lane) issues the MMAs and owns the tensor-memory
// allocation; warps 2..5 read the accumulator back (tcgen05.ld: warp w may touch lanes
// 32*(w%4)..+31) and apply the epilogue straight from registers.
//
// Either operand may be contiguous along k ("K-major": activations in x*W, weights in
// delta*W^T) or along m/n ("MN-major": weights in x*W, both operands of a^T*delta); the shared
// memory tile is 128-byte swizzled in both cases and the UMMA descriptors say which.
// Rows/columns beyond the tensor extents are zero-filled by TMA, so ragged shapes need no
// special casing in the main loop; the epilogue masks its stores.
//
// Every wait is bounded: after about a second without progress a role records
// IST_ERR_DEVICE_TIMEOUT in the status word, raises the CTA's abort flag and all roles fall
// through to the common exit, where tensor memory is released.
#include <cuda.h>

#include <cstdio>
#include <map>
#include <mutex>
#include <tuple>

#include "kernels.h"

namespace ist {
namespace {

constexpr int BM = 128;
constexpr int BK = 64;                   // 64 bf16 = 128 bytes = one swizzle row
constexpr int kThreads = 192;
constexpr long long kWaitLimitCycles = 2000000000ll;   // ~1 s at 2 GHz

// ---- small PTX wrappers ------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false (and raises the abort flag) if the phase did not complete in time
// or another role has already aborted.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          DeviceStatus* st, int where) {
  if (mbar_try_wait(bar, parity)) return true;
  long long t0 = clock64();
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > kWaitLimitCycles) {
      *abort_flag = 1;
      report(st, -6, SITE_TC_PIPE, where);
      return false;
    }
  }
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0,
                                            int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// 32 lanes x 32 consecutive 32-bit columns: thread i of the warp gets lane (row) i.
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t* v) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor for a 128-byte-swizzled tile.
//   bits  0..13 start address >> 4      bits 16..29 leading byte offset >> 4
//   bits 32..45 stride byte offset >> 4 bits 46..47 descriptor version (1)
//   bits 61..63 swizzle mode (2 = 128 B)
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// Instruction descriptor: D = f32 (bits 4..5 = 1), A and B = bf16 (bits 7..9, 10..12 = 1),
// operand majors (bit 15 / 16: 1 = MN-major), N >> 3 at bits 17..22, M >> 4 at bits 24..28.
__host__ __device__ constexpr uint32_t make_idesc(int a_mn, int b_mn, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

struct TcArgs {
  int M, N, K;            // M, N: bounds of the output rows / columns the epilogue may touch
  int a_gmul, b_gmul;     // 1 if the operand has one slab per group, 0 if all groups share it
  int epi;
  const float* bias; long long bias_sg;
  bf16* out; long long out_ld, out_sg;
  float* outf; long long outf_ld, outf_sg;
  const bf16* mask; long long mask_ld, mask_sg;
  bf16* opw;
  float lr;
  DeviceStatus* status;
};

__device__ __forceinline__ uint2 pack4(float a, float b, float c, float d) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  uint2 r;
  r.x = *reinterpret_cast<uint32_t*>(&lo);
  r.y = *reinterpret_cast<uint32_t*>(&hi);
  return r;
}

// Applies the epilogue to 32 consecutive columns [n, n+32) of output row m (thread-private).
template <int EPI>
__device__ __forceinline__ void epilogue_row32(const TcArgs& a, int g, int m, int n, const uint32_t* acc) {
#pragma unroll
  for (int v = 0; v < 8; ++v) {
    const int nn = n + 4 * v;
    if (nn >= a.N) break;
    float c0 = __uint_as_float(acc[4 * v]), c1 = __uint_as_float(acc[4 * v + 1]);
    float c2 = __uint_as_float(acc[4 * v + 2]), c3 = __uint_as_float(acc[4 * v + 3]);
    if (EPI == EPI_BIAS_RELU) {
      float4 b = *reinterpret_cast<const float4*>(a.bias + (long long)g * a.bias_sg + nn);
      *reinterpret_cast<uint2*>(a.out + (long long)g * a.out_sg + (long long)m * a.out_ld + nn) =
          pack4(fmaxf(c0 + b.x, 0.f), fmaxf(c1 + b.y, 0.f), fmaxf(c2 + b.z, 0.f), fmaxf(c3 + b.w, 0.f));
    } else if (EPI == EPI_BIAS_F32) {
      float4 b = *reinterpret_cast<const float4*>(a.bias + (long long)g * a.bias_sg + nn);
      *reinterpret_cast<float4*>(a.outf + (long long)g * a.outf_sg + (long long)m * a.outf_ld + nn) =
          make_float4(c0 + b.x, c1 + b.y, c2 + b.z, c3 + b.w);
    } else if (EPI == EPI_RELU_MASK) {
      uint2 mk = *reinterpret_cast<const uint2*>(a.mask + (long long)g * a.mask_sg + (long long)m * a.mask_ld + nn);
      __nv_bfloat162 m01 = *reinterpret_cast<__nv_bfloat162*>(&mk.x);
      __nv_bfloat162 m23 = *reinterpret_cast<__nv_bfloat162*>(&mk.y);
      *reinterpret_cast<uint2*>(a.out + (long long)g * a.out_sg + (long long)m * a.out_ld + nn) =
          pack4(__low2float(m01) > 0.f ? c0 : 0.f, __high2float(m01) > 0.f ? c1 : 0.f,
                __low2float(m23) > 0.f ? c2 : 0.f, __high2float(m23) > 0.f ? c3 : 0.f);
    } else if (EPI == EPI_SGD) {
      long long o = (long long)g * a.outf_sg + (long long)m * a.outf_ld + nn;
      float4 w = *reinterpret_cast<float4*>(a.outf + o);
      w.x -= a.lr * c0; w.y -= a.lr * c1; w.z -= a.lr * c2; w.w -= a.lr * c3;
      *reinterpret_cast<float4*>(a.outf + o) = w;
      *reinterpret_cast<uint2*>(a.opw + o) = pack4(w.x, w.y, w.z, w.w);
    } else {
      *reinterpret_cast<uint2*>(a.out + (long long)g * a.out_sg + (long long)m * a.out_ld + nn) =
          pack4(c0, c1, c2, c3);
    }
  }
}

template <int A_MN, int B_MN, int BN, int STAGES, int EPI>
__global__ void __launch_bounds__(kThreads)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, TcArgs a) {
  constexpr uint32_t A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  __shared__ uint64_t full_bar[STAGES], empty_bar[STAGES], acc_bar;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN, g = blockIdx.z;
  const int num_kb = (a.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    mbar_init(&acc_bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                 "r"((uint32_t)BN)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  volatile int* abortp = &abort_flag;

  if (warp == 0) {
    if (lane == 0) {
      int issued = 0;
      for (int kb = 0; kb < num_kb; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (kb / STAGES) & 1;
        if (!mbar_wait(&empty_bar[s], ph ^ 1, abortp, a.status, 1)) break;
        uint8_t* sa = smem + s * STAGE_BYTES;
        uint8_t* sb = sa + A_BYTES;
        mbar_expect_tx(&full_bar[s], STAGE_BYTES);
        if (A_MN) {
#pragma unroll
          for (int j = 0; j < BM / 64; ++j)
            tma_load_3d(sa + j * (BK * 128), &tmA, &full_bar[s], m0 + 64 * j, kb * BK, g * a.a_gmul);
        } else {
          tma_load_3d(sa, &tmA, &full_bar[s], kb * BK, m0, g * a.a_gmul);
        }
        if (B_MN) {
#pragma unroll
          for (int j = 0; j < BN / 64; ++j)
            tma_load_3d(sb + j * (BK * 128), &tmB, &full_bar[s], n0 + 64 * j, kb * BK, g * a.b_gmul);
        } else {
          tma_load_3d(sb, &tmB, &full_bar[s], kb * BK, n0, g * a.b_gmul);
        }
        issued = kb + 1;
      }
      if (*abortp) {
        // let copies already in flight land before the CTA's shared memory goes away
        for (int kb = max(0, issued - STAGES); kb < issued; ++kb) {
          long long t0 = clock64();
          while (!mbar_try_wait(&full_bar[kb % STAGES], (kb / STAGES) & 1) && clock64() - t0 < kWaitLimitCycles) {}
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(A_MN, B_MN, BN);
      bool ok = true;
      for (int kb = 0; kb < num_kb && ok; ++kb) {
        const int s = kb % STAGES;
        const uint32_t ph = (kb / STAGES) & 1;
        ok = mbar_wait(&full_bar[s], ph, abortp, a.status, 2);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sa = smem_u32(smem + s * STAGE_BYTES), sb = sa + A_BYTES;
#pragma unroll
        for (int k = 0; k < BK / 16; ++k) {
          // K-major: 16 k-elements = 32 bytes inside the swizzle row; 8-row groups 1024 B apart.
          // MN-major: 16 k-rows = 2048 B; 64-element MN chunks (one TMA box each) 8192 B apart.
          const uint64_t ad = A_MN ? make_desc(sa + k * 2048, BK * 128, 1024) : make_desc(sa + k * 32, 16, 1024);
          const uint64_t bd = B_MN ? make_desc(sb + k * 2048, BK * 128, 1024) : make_desc(sb + k * 32, 16, 1024);
          tc_mma(tmem_base, ad, bd, idesc, (kb | k) != 0);
        }
        tc_commit(&empty_bar[s]);   // frees the slot once these MMAs have read it
      }
      if (ok) tc_commit(&acc_bar);  // accumulator complete
    }
  } else {
    if (mbar_wait(&acc_bar, 0, abortp, a.status, 3)) {
      tc_fence_after();
      const int q = warp & 3;
      const int m = m0 + q * 32 + lane;
#pragma unroll 1
      for (int c = 0; c < BN; c += 32) {
        if (n0 + c >= a.N) break;   // warp-uniform
        uint32_t acc[32];
        tc_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)c, acc);
        if (m < a.M) epilogue_row32<EPI>(a, g, m, n0 + c, acc);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)BN)
                 : "memory");
  }
}

// ---- host side ---------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

// bf16 tensor [groups][outer][inner] (inner contiguous), box {64, box_outer, 1}, 128-byte swizzle.
using MapKey = std::tuple<const void*, long long, long long, long long, long long, long long, int>;
std::map<MapKey, CUtensorMap>& map_cache() {
  static std::map<MapKey, CUtensorMap> c;
  return c;
}
std::mutex& map_mutex() {
  static std::mutex m;
  return m;
}

bool make_map(CUtensorMap* out, const bf16* base, long long inner, long long outer, long long groups,
              long long outer_stride, long long group_stride, int box_outer) {
  MapKey key{base, inner, outer, groups, outer_stride, group_stride, box_outer};
  std::lock_guard<std::mutex> lk(map_mutex());
  auto& cache = map_cache();
  auto it = cache.find(key);
  if (it != cache.end()) {
    *out = it->second;
    return true;
  }
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)outer, (cuuint64_t)groups};
  cuuint64_t strides[2] = {(cuuint64_t)outer_stride * 2,
                           (cuuint64_t)(groups > 1 ? group_stride : outer_stride * outer) * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)box_outer, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<bf16*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  if (cache.size() > 4096) cache.clear();
  cache[key] = *out;
  return true;
}

template <int A_MN, int B_MN, int BN, int STAGES, int EPI>
bool launch(const Launch& L, const CUtensorMap& ma, const CUtensorMap& mb, const TcArgs& t, int m_tiles, int n_tiles,
            int G) {
  constexpr int smem = STAGES * (BM * BK * 2 + BN * BK * 2) + 1024;
  auto kern = gemm_tc_kernel<A_MN, B_MN, BN, STAGES, EPI>;
  static bool configured = false;
  if (!configured) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return false;
    configured = true;
  }
  kern<<<dim3(m_tiles, n_tiles, G), kThreads, smem, L.stream>>>(ma, mb, t);
  L.count();
  return true;
}

template <int A_MN, int B_MN, int EPI>
bool launch_bn(const Launch& L, const CUtensorMap& ma, const CUtensorMap& mb, const TcArgs& t, int bn, int m_tiles,
               int n_tiles, int G) {
  switch (bn) {
    case 64: return launch<A_MN, B_MN, 64, 4, EPI>(L, ma, mb, t, m_tiles, n_tiles, G);
    case 128: return launch<A_MN, B_MN, 128, 3, EPI>(L, ma, mb, t, m_tiles, n_tiles, G);
    default: return launch<A_MN, B_MN, 256, 4, EPI>(L, ma, mb, t, m_tiles, n_tiles, G);
  }
}

}  // namespace

// Tile width: the widest of 256 / 128 / 64 that still gives every SM a tile; the weight-update
// epilogue moves 10 bytes per output element, so it prefers two resident CTAs of width 128.
int pick_bn(int M, int N, int G, int epi) {
  const long long m_tiles = ceil_div(M, BM);
  auto tiles = [&](int bn) { return m_tiles * ceil_div(N, bn) * G; };
  if (epi == EPI_SGD) return (N > 64 && tiles(128) >= 148) ? 128 : 64;
  if (N > 128 && tiles(256) >= 148) return 256;
  if (N > 64 && tiles(128) >= 148) return 128;
  return 64;
}

bool gemm_tc(const Launch& L, const GemmArgs<bf16>& a, DeviceStatus* st) {
  const int n_store = a.N_store > 0 ? a.N_store : a.N;
  const bool a_mn = a.a_sm == 1 && a.a_sk != 1, b_mn = a.b_sn == 1 && a.b_sk != 1;
  if (!a_mn && a.a_sk != 1) return false;
  if (!b_mn && a.b_sk != 1) return false;
  const int bn = pick_bn(a.M, n_store, a.G, a.epi);
  const int m_tiles = (int)ceil_div(a.M, BM), n_tiles = (int)ceil_div(n_store, bn);
  if (n_tiles > 65535 || a.G > 65535) return false;
  CUtensorMap ma, mb;
  // K-major operand: inner = K, outer = rows (M or N).  MN-major: inner = rows, outer = K.
  const long long ga = (a.G > 1 && a.a_sg != 0) ? a.G : 1, gb = (a.G > 1 && a.b_sg != 0) ? a.G : 1;
  const bool ok_a = a_mn ? make_map(&ma, a.A, a.M, a.K, ga, a.a_sk, a.a_sg, BK)
                         : make_map(&ma, a.A, a.K, a.M, ga, a.a_sm, a.a_sg, BM);
  const bool ok_b = b_mn ? make_map(&mb, a.B, a.N, a.K, gb, a.b_sk, a.b_sg, BK)
                         : make_map(&mb, a.B, a.K, a.N, gb, a.b_sn, a.b_sg, bn);
  if (!ok_a || !ok_b) return false;
  TcArgs t{};
  t.M = a.M; t.N = n_store; t.K = a.K;
  t.a_gmul = (a.G > 1 && a.a_sg != 0) ? 1 : 0;
  t.b_gmul = (a.G > 1 && a.b_sg != 0) ? 1 : 0;
  t.epi = a.epi;
  t.bias = a.bias; t.bias_sg = a.bias_sg;
  t.out = a.out; t.out_ld = a.out_ld; t.out_sg = a.out_sg;
  t.outf = a.outf; t.outf_ld = a.outf_ld; t.outf_sg = a.outf_sg;
  t.mask = a.mask; t.mask_ld = a.mask_ld; t.mask_sg = a.mask_sg;
  t.opw = a.opw;
  t.lr = a.lr;
  t.status = st;
  switch (a.epi) {
    case EPI_BIAS_RELU:
      if (!a_mn && b_mn) return launch_bn<0, 1, EPI_BIAS_RELU>(L, ma, mb, t, bn, m_tiles, n_tiles, a.G);
      break;
    case EPI_BIAS_F32:
      if (!a_mn && b_mn) return launch_bn<0, 1, EPI_BIAS_F32>(L, ma, mb, t, bn, m_tiles, n_tiles, a.G);
      break;
    case EPI_RELU_MASK:
      if (!a_mn && !b_mn) return launch_bn<0, 0, EPI_RELU_MASK>(L, ma, mb, t, bn, m_tiles, n_tiles, a.G);
      break;
    case EPI_SGD:
      if (a_mn && b_mn && a.opw) return launch_bn<1, 1, EPI_SGD>(L, ma, mb, t, bn, m_tiles, n_tiles, a.G);
      break;
    default:
      break;
  }
  return false;
}

}  // namespace ist
