// Grouped bf16 GEMM on the 5th-generation tensor cores (tcgen05.mma, accumulators in tensor
// memory, operands staged in shared memory by TMA) with the local-step epilogues fused in:
// bias + ReLU (forward), logits, ReLU mask (delta back-propagation) and the SGD update of the
// fp32 master slice together with its bf16 operand copy (paper Sec. 2.1 "Training Subnets";
// App. A Eq. (2) on the slices).  All S subnets are tiles of one persistent launch.
//
//   C[g](m, n) = sum_k A[g](m, k) * B[g](n, k),   fp32 accumulation
//
// One CTA per SM walks over 128 x BN output tiles (tile = blockIdx.x + i * gridDim.x).
//   warp 0 (one lane)  TMA loads of the A / B k-slabs into a ring of STAGES slots
//   warp 1 (one lane)  tcgen05.mma issue; owns the tensor-memory allocation (2 accumulators,
//                      so the MMAs of tile i+1 overlap the epilogue of tile i)
//   then the epilogue warps, groups of four that take the 32-column chunks in turn (two groups;
//                      four for the softmax passes over a very wide output layer):
//                      tcgen05.ld (warp w reads lanes 32*(w%4)..+31, one row per thread), apply
//                      the epilogue, write the chunk into a swizzled shared-memory slot
//   then one warp (one lane), where the epilogue has input chunks: their TMA loads into the
//                      slots (the fp32 master slice for the SGD update, the ReLU mask for the
//                      delta GEMM)
//   then the storers (one lane each; four, two beside sixteen epilogue warps, none where the
//                      epilogue stores no chunks): TMA stores of finished slots (coalesced,
//                      clipped at the tensor edge); slot i belongs to storer i % (their number),
//                      which hands the slot back as soon as its own store has read it, without
//                      waiting for a later chunk
//   then two warps, weight-update launches on single CTAs only: column sums of the B operand
//                      (the deltas) as its k-slabs pass through shared memory, which is the bias
//                      gradient; the bias update then needs no pass of its own over the deltas
// The epilogue has no CTA-wide barrier: slots move between loader, epilogue warps and storer
// through mbarriers (slot_full -> chunk_done -> slot_empty), so warps work on different chunks
// at the same time and a slow chunk does not hold the others back.
// The weight-update epilogue is the HBM-heavy part of a step (10 bytes per weight against
// 2*B flops): its fp32 master chunks are prefetched through the slot ring while earlier chunks
// are updated in place in shared memory and stored back.
//
// PAIR = 2 runs two CTAs of a cluster as one unit (tcgen05 cta_group::2): the pair computes a
// 256 x BN tile, each CTA loads its own 128 rows of A and its half (BN/2 rows) of B and keeps its
// own 128 x BN accumulator, and the leader CTA (cluster rank 0) issues one MMA that reads both
// CTAs' shared memory.  Every B byte then enters shared memory once per 256 output rows instead
// of once per 128, which is what the L2-to-SM path needs to keep the tensor pipe fed.
//
// Either operand may be contiguous along k ("K-major") or along m/n ("MN-major"); the shared
// memory tile is 128-byte swizzled in both cases and the UMMA descriptors say which.  Rows and
// columns beyond the tensor extents are zero-filled by TMA loads and dropped by TMA stores.
//
// One launch may run several products of the same kind ("problems": the same operand layouts, tile
// shape and epilogue, e.g. the weight updates of all layers of a step).  Their tiles form one flat
// list that the CTAs walk in order, so that a small product costs a few tiles instead of a launch
// and no SM idles between one product's last wave and the next one's first.  A problem may be
// chained to the one before it in the list (its A operand is that problem's output, as in
// a_l = relu(a_{l-1} W_l + b_l) or delta_{l-1} = (delta_l W_l^T) * mask): its tiles then wait
// until the rows they read are complete, through one counter per (group, block of tile rows)
// that the storing threads of the producer bump after their stores have completed.  Tiles are
// claimed in list order by CTAs that are all resident at once, and a tile depends only on
// earlier tiles, so the waits always end; they are bounded like every other wait here.
//
// Every wait is bounded: after about a second without progress a role records
// IST_ERR_DEVICE_TIMEOUT in the status word, raises the CTA's abort flag and all roles fall
// through to the common exit, where tensor memory is released.
#include <cuda.h>

#include <map>
#include <mutex>
#include <tuple>

#include "kernels.h"

namespace ist {
namespace {

constexpr int BM = 128;
constexpr int BK = 64;                   // 64 bf16 = 128 bytes = one swizzle row
constexpr int CH = 32;                   // epilogue chunk: 32 output columns
// Warps of a CTA, see the role list above: loader, MMA issuer, the epilogue warps (two groups of
// four; four groups for the two softmax passes over a very wide output layer, whose epilogues are
// long chains of dependent instructions and need more warps to hide them), the epilogue input
// loader, four storers, and two summing warps for weight-update launches (bias gradient).
constexpr int kSumWarps = 2;
constexpr bool sums_in_kernel(int epi, int pair) { return epi == 3 /* EPI_SGD */ && pair == 1; }   // sums from the B stages
constexpr bool has_sum_warps(int epi) { return epi == 3 /* EPI_SGD */; }
constexpr int epi_warps(int epi) { return (epi == 5 /* EPI_LSE_PART */ || epi == 6 /* EPI_SOFTMAX_DELTA */) ? 16 : 8; }
constexpr bool has_aux(int epi) { return epi == 2 /* EPI_RELU_MASK */ || epi == 3; }   // EpiTraits::kAux
// storers: none where the epilogue stores no chunks (EpiTraits::k32 || k16), two beside sixteen
// epilogue warps (20 warps leave a thread 96 registers, 22 would leave 80), else four
constexpr int store_warps(int epi) { return epi == 5 ? 0 : epi == 6 ? 2 : 4; }
constexpr int threads_for(int epi, int pair) {
  return (2 + epi_warps(epi) + (has_aux(epi) ? 1 : 0) + store_warps(epi) + (has_sum_warps(epi) ? kSumWarps : 0)) * 32;
}
constexpr long long kWaitLimitCycles = 2000000000ll;   // ~1 s at 2 GHz
constexpr uint32_t kSuspendHintNs = 20000;             // a waiting thread may sleep this long inside one try_wait

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
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(kSuspendHintNs)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false (and raises the abort flag) if the phase did not complete in time
// or another role has already aborted.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          DeviceStatus* st, int where, long long limit_cycles = kWaitLimitCycles) {
  if (mbar_try_wait(bar, parity)) return true;
  long long t0 = clock64();
  while (true) {
    // A try_wait comes back after a fraction of a microsecond whatever its hint says, so a waiting
    // warp goes round this loop millions of times per second: the abort flag and the clock are
    // looked at once in 32 rounds, which keeps a round at a few instructions (in the softmax
    // passes over a very wide output layer, sixteen waiting epilogue warps otherwise issue more
    // instructions in this loop than in their arithmetic; no measurable difference in time).
#pragma unroll 1
    for (int i = 0; i < 32; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > limit_cycles) {
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
// Same copy issued by a CTA of a pair; the mbarrier may live in the peer CTA (shared::cluster
// address), which is how both CTAs' loads complete on the leader's "full" barrier.
__device__ __forceinline__ void tma_load_3d_pair(void* dst, const CUtensorMap* map, uint32_t bar_cluster_addr,
                                                 int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(bar_cluster_addr), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(const void* p, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(p)), "r"(rank));
  return r;
}
// Arrival on a barrier of another CTA of the cluster, which hands back a tensor-memory
// accumulator whose reads have completed (tcgen05.wait::ld, then
// tcgen05.fence::before_thread_sync); no data in memory goes with it.  CLUSTER_SCOPE: release at
// cluster scope, which stalls the arriving warp for most of a microsecond per tile; otherwise
// the instruction's default, release at CTA scope.  The softmax passes over a very wide output
// layer, whose tiles are short, take the cheap form (670,091 classes behind 128 hidden neurons per
// subnet: the two passes 2.4 -> 2.2 ms per local step); the weight update measured 4 % slower with it than with the stall and keeps the
// cluster scope, as do the other epilogues, where it makes no difference.
template <bool CLUSTER_SCOPE>
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
  if (CLUSTER_SCOPE)
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
  else
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, const void* src, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(map), "r"(smem_u32(src)), "r"(c0), "r"(c1), "r"(c2)
               : "memory");
}
// Asks for a box to be brought into L2 only (no shared-memory destination, nothing to wait for).
__device__ __forceinline__ void tma_prefetch_l2_3d(const CUtensorMap* map, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];"
               ::"l"(map), "r"(c0), "r"(c1), "r"(c2)
               : "memory");
}
// Brings a tensor map (a kernel parameter) into the descriptor cache ahead of its first copy.
__device__ __forceinline__ void prefetch_map(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
__device__ __forceinline__ void tma_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void tma_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void tma_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
// Pair forms: one commit arrives on the barrier at the same offset in both CTAs; one MMA
// reads both CTAs' operand tiles and writes both accumulators.
__device__ __forceinline__ void tc_commit_pair(uint64_t* bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(smem_u32(bar)), "h"((uint16_t)3)
      : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
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

// 32 lanes x 16 consecutive 32-bit columns.
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t* v) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
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
__host__ __device__ constexpr uint32_t make_idesc(int a_mn, int b_mn, int n, int m) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

constexpr int kMaxProblems = 4;

// One product of a launch.  Tiles tile_end(previous) .. tile_end - 1 of the flat list are its.
struct TcProblem {
  int M, N, K;            // M, N: bounds of the output rows / columns the epilogue touches
  int n_true;             // columns of the product proper (<= N; the rest pads the rows): the softmax passes count only these
  int m_tiles, n_tiles, G;
  uint32_t m_div, m_sh, n_div, n_sh;   // division by m_tiles / n_tiles as a multiplication, see div_by
  int k_splits, kb_per_split;   // the k range may be cut into slices that run as separate tiles
  int a_gmul, b_gmul;     // 1 if the operand has one slab per group, 0 if all groups share it
  int tile_end;
  // true extents of the groups (null: every group fills M / N / K), see GemmArgs
  const int32_t* m_off; const int32_t* n_off; const int32_t* k_off;
  // weight-update launches: bias[g * bias_upd_sg + n] -= lr * sum_k B[g](n, k) for n < bias_n (null: none),
  // summed from the B stages in shared memory (single CTAs only) ...
  float* bias_upd; long long bias_upd_sg; int bias_n;
  // ... or the same from B as it lies in memory (bias_mem null: none): dmem[g * dmem_sg + k * dmem_ld + n];
  // the work is cut into items of 64 columns of one group, items bias_item_end(previous) ..
  // bias_item_end - 1 of the launch belong to this problem
  float* bias_mem; const bf16* dmem; long long dmem_ld, dmem_sg; int bias_item_end;
  int head_f32;           // EPI_BIAS_RELU launches only: this problem writes plain fp32 products in
                          // 16-column chunks through the c32 map (a narrow output layer riding on the
                          // hidden layers' launch); 0 = the launch's ordinary epilogue
  const float* bias; long long bias_sg;
  // chaining: counters [G][m_tiles]; a tile of (g, mt) may load A once wait_ctr[g * m_tiles + mt]
  // has reached wait_target; a storer adds the chunks it has stored for (g, mt) to signal_ctr
  const unsigned* wait_ctr; unsigned wait_target;
  unsigned* signal_ctr;
};

struct TcArgs {
  int n_problems, total_tiles;
  TcProblem p[kMaxProblems];
  // weight-update launches: the step's mean losses, loss.loss_out[g * out_stride + k] = mean of
  // loss.row_loss[g][0 .. loss_B) for g < loss_G (loss_out null: none)
  LossReduce loss;
  int loss_B, loss_G;
  int n_bias_items;        // bias items of all problems (see TcProblem::bias_mem)
  float lr;
  DeviceStatus* status;
  // wide softmax head (see GemmArgs); single-problem launches only
  float2* lse_part;
  const float* lse; long long lse_sg;
  const int32_t* labels; long long labels_sg;
  float* label_logit;
  float inv_rows;
};

struct TcMaps {
  CUtensorMap a[kMaxProblems], b[kMaxProblems];
  CUtensorMap c32[kMaxProblems];     // fp32 chunks: logits out, master in/out
  CUtensorMap c16[kMaxProblems];     // bf16 chunks out: activations, delta, weights
  CUtensorMap aux16[kMaxProblems];   // bf16 chunks in: ReLU mask
};

// Where a tile of the flat list lies: problem, tile row / column, output slab (group and k slice).
struct TileAt {
  int pi, mt, nt, slab;
};
// n / d for 0 <= n < 2^31 with mul = floor(2^(31 + sh) / d) + 1, sh = ceil(log2 d) (set_div): the
// product over-estimates n / d by less than n / 2^31 / d < 1 / d, so the floor is exact.  Every
// role of the kernel locates every tile; two hardware divisions per tile were a large share of the
// instructions of launches with short tiles.
__device__ __forceinline__ int div_by(int n, uint32_t mul, uint32_t sh) {
  return (int)(((unsigned long long)(uint32_t)n * mul) >> (31 + sh));
}
__device__ __forceinline__ TileAt locate(const TcArgs& a, int tile, int& pi) {
  while (tile >= a.p[pi].tile_end) ++pi;       // tiles are visited in increasing order
  const TcProblem& pr = a.p[pi];
  const int lt = tile - (pi ? a.p[pi - 1].tile_end : 0);
  TileAt t;
  t.pi = pi;
  const int q = div_by(lt, pr.m_div, pr.m_sh);       // lt / m_tiles
  t.mt = lt - q * pr.m_tiles;
  t.slab = div_by(q, pr.n_div, pr.n_sh);             // lt / (m_tiles * n_tiles)
  t.nt = q - t.slab * pr.n_tiles;
  return t;
}

// Group and k slice of an output slab; launches without k slices (nearly all) skip the division.
__device__ __forceinline__ int group_of(const TcProblem& pr, int slab) { return pr.k_splits == 1 ? slab : slab / pr.k_splits; }
__device__ __forceinline__ int kslice_of(const TcProblem& pr, int slab) { return pr.k_splits == 1 ? 0 : slab % pr.k_splits; }

// Whether tile (mt, nt) of group g has any output inside the group's true extents, and how many
// 64-deep k blocks its contraction really needs (at least one, so that the accumulator is
// written: the operands beyond a group's depth are zeros).  Every role asks the same question
// about every tile, so all of them skip the same tiles.
// Weight-update launches on single CTAs: the tiles of the first tile row also sum their column
// block's deltas for the bias update.
__device__ __forceinline__ bool sums_bias(const TcProblem& pr, const TileAt& at) {
  return pr.bias_upd != nullptr && at.mt == 0;
}

template <int TILE_M, int TILE_N>
__device__ __forceinline__ bool tile_live(const TcProblem& pr, const TileAt& at, int g, int* kb_limit) {
  *kb_limit = 0x7fffffff;
  if (!pr.m_off && !pr.n_off && !pr.k_off) return true;
  if (pr.n_off && at.nt * TILE_N >= __ldg(pr.n_off + g + 1) - __ldg(pr.n_off + g)) return false;
  // a tile that carries its columns' bias update runs even if it lies beyond the group's rows
  if (pr.m_off && at.mt * TILE_M >= __ldg(pr.m_off + g + 1) - __ldg(pr.m_off + g) && !sums_bias(pr, at))
    return false;
  if (pr.k_off) *kb_limit = max(1, (__ldg(pr.k_off + g + 1) - __ldg(pr.k_off + g) + BK - 1) / BK);
  return true;
}

__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_add(unsigned* p, unsigned v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

// Chunk staging: a ring of fp32 areas ([128][32] floats, 128-byte swizzle) and / or a ring of
// bf16 areas ([128][32] bf16, 64-byte swizzle); kAux says whether chunks are loaded before use
// (the fp32 ring for the SGD update, the bf16 ring for the ReLU mask).
template <int EPI> struct EpiTraits;
template <> struct EpiTraits<EPI_BIAS_RELU> { static constexpr bool k32 = false, k16 = true, kAux = false; };
template <> struct EpiTraits<EPI_BIAS_F32> { static constexpr bool k32 = true, k16 = false, kAux = false; };
template <> struct EpiTraits<EPI_RELU_MASK> { static constexpr bool k32 = false, k16 = true, kAux = true; };
template <> struct EpiTraits<EPI_SGD> { static constexpr bool k32 = true, k16 = true, kAux = true; };
template <> struct EpiTraits<EPI_LSE_PART> { static constexpr bool k32 = false, k16 = false, kAux = false; };
template <> struct EpiTraits<EPI_SOFTMAX_DELTA> { static constexpr bool k32 = false, k16 = true, kAux = false; };

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint4 pack8(const float* v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
  __nv_bfloat162 c = __floats2bfloat162_rn(v[4], v[5]), d = __floats2bfloat162_rn(v[6], v[7]);
  uint4 r;
  r.x = *reinterpret_cast<uint32_t*>(&a);
  r.y = *reinterpret_cast<uint32_t*>(&b);
  r.z = *reinterpret_cast<uint32_t*>(&c);
  r.w = *reinterpret_cast<uint32_t*>(&d);
  return r;
}
__device__ __forceinline__ void unpack8(uint4 u, float* v) {
  __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&u.x), b = *reinterpret_cast<__nv_bfloat162*>(&u.y);
  __nv_bfloat162 c = *reinterpret_cast<__nv_bfloat162*>(&u.z), d = *reinterpret_cast<__nv_bfloat162*>(&u.w);
  v[0] = __low2float(a); v[1] = __high2float(a); v[2] = __low2float(b); v[3] = __high2float(b);
  v[4] = __low2float(c); v[5] = __high2float(c); v[6] = __low2float(d); v[7] = __high2float(d);
}

// Row r of a chunk slot.  fp32 area: 128-byte rows, 16-byte unit u stored at u ^ (r & 7).
// bf16 area: 64-byte rows, 16-byte unit u stored at u ^ ((r >> 1) & 3).
__device__ __forceinline__ float4* f32_unit(uint8_t* area, int r, int u) {
  return reinterpret_cast<float4*>(area + r * 128 + ((u ^ (r & 7)) << 4));
}
__device__ __forceinline__ uint4* b16_unit(uint8_t* area, int r, int u) {
  return reinterpret_cast<uint4*>(area + r * 64 + ((u ^ ((r >> 1) & 3)) << 4));
}

template <int A_MN, int B_MN, int BN, int STAGES, int NS, int EPI, int PAIR>
__global__ void __launch_bounds__(threads_for(EPI, PAIR), 1)
gemm_tc_kernel(const __grid_constant__ TcMaps maps, const __grid_constant__ TcArgs a) {
  using ET = EpiTraits<EPI>;
  constexpr int BNL = BN / PAIR;   // rows of the B tile this CTA loads
  constexpr uint32_t A_BYTES = BM * BK * 2, B_BYTES = BNL * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
  // a slot holds one 128 x 32 chunk: an fp32 area and / or a bf16 area, as the epilogue needs
  constexpr uint32_t F32_BYTES = ET::k32 ? BM * CH * 4 : 0, B16_BYTES = ET::k16 ? BM * CH * 2 : 0;
  constexpr uint32_t SLOT_BYTES = F32_BYTES + B16_BYTES;
  constexpr uint32_t AUX_BYTES = EPI == EPI_SGD ? F32_BYTES : B16_BYTES;
  constexpr uint32_t TMEM_COLS = 2 * BN;
  constexpr int NCH = BN / CH;
  constexpr bool kStore = ET::k32 || ET::k16;   // the epilogue writes chunks through the slot ring
  constexpr bool kSums = sums_in_kernel(EPI, PAIR);   // two more warps sum the deltas for the bias update
  static_assert(EPI_RELU_MASK == 2 && EPI_SGD == 3 && EPI_LSE_PART == 5 && EPI_SOFTMAX_DELTA == 6 &&
                    has_aux(EPI) == ET::kAux && (store_warps(EPI) > 0) == kStore,
                "the role layout functions name epilogues by value");
  constexpr int kEpiWarps = epi_warps(EPI), NG = kEpiWarps / 4;   // epilogue warps; groups of four
  // first warp after the epilogue warps: the input loader if the epilogue has one, then the storers
  constexpr int kAuxWarp = 2 + kEpiWarps, kStoreWarp0 = kAuxWarp + (ET::kAux ? 1 : 0), kStoreWarps = store_warps(EPI);
  constexpr float kLog2e = 1.4426950408889634f;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* slots = smem + STAGES * STAGE_BYTES;
  __shared__ uint64_t full_bar[STAGES], empty_bar[STAGES], acc_full[2], acc_empty[2];
  __shared__ uint64_t slot_full[NS], chunk_done[NS], slot_empty[NS];
  // weight update on single CTAs: "stage is full" passed on to the summing warps, and their "stage has been read"
  __shared__ uint64_t stage_here[STAGES], sum_done[STAGES];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_tiles = a.total_tiles;             // tiles of (128 * PAIR) x BN x k slice, all problems
  const int rank = PAIR == 2 ? (int)cluster_ctarank() : 0;
  const int unit = blockIdx.x / PAIR, n_units = gridDim.x / PAIR;   // a unit = a CTA or a pair

  if (threadIdx.x == 32) {   // the maps this instance copies through; they do not depend on the previous kernel
    for (int i = 0; i < a.n_problems; ++i) {
      prefetch_map(&maps.a[i]);
      prefetch_map(&maps.b[i]);
      if (ET::k32 || (EPI == EPI_BIAS_RELU && a.p[i].head_f32)) prefetch_map(&maps.c32[i]);
      if (ET::k16) prefetch_map(&maps.c16[i]);
      if (EPI == EPI_RELU_MASK) prefetch_map(&maps.aux16[i]);
    }
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&stage_here[s], 1);
      mbar_init(&empty_bar[s], 1);                 // the MMA commit
      mbar_init(&sum_done[s], kSumWarps);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&acc_full[b], 1);
      mbar_init(&acc_empty[b], PAIR * kEpiWarps);   // one arrival per epilogue warp of the unit
    }
    for (int s = 0; s < NS; ++s) {
      mbar_init(&slot_full[s], 1);               // loader's TMA bytes
      mbar_init(&chunk_done[s], 4);              // the four warps that worked on the chunk
      mbar_init(&slot_empty[s], 1);              // storer: the store has read the slot
    }
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  if (warp == 1) {
    if (PAIR == 2) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                   "r"(TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                   "r"(TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR == 2) cluster_sync_all();   // the peer's barriers are initialised before anyone signals them
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  volatile int* abortp = &abort_flag;
  // Programmatic dependent launch: everything above touched only this CTA's own shared and tensor
  // memory, so it may run while the previous kernel in the stream is still draining.  From here on
  // global memory written by that kernel is read (and buffers it reads are overwritten), so wait
  // until it has completed and its writes are visible; then let the next kernel's CTAs be
  // scheduled as this grid's CTAs retire.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == 0) {
    // ---------------------------------------------------------------- operand loads
    if (lane == 0) {
      int it = 0, pi = 0;
      uint32_t sum_pending = 0, sum_parity = 0;
      bool ok = true;
      for (int tile = unit; tile < total_tiles && ok; tile += n_units) {
        const TileAt at = locate(a, tile, pi);
        const TcProblem& pr = a.p[pi];
        const CUtensorMap* tmA = &maps.a[pi];
        const CUtensorMap* tmB = &maps.b[pi];
        const int m0 = at.mt * (BM * PAIR) + rank * BM;     // this CTA's rows of A
        const int n0 = at.nt * BN + rank * BNL;             // this CTA's rows of B
        const int g = group_of(pr, at.slab);
        int kb_limit;
        if (!tile_live<BM * PAIR, BN>(pr, at, g, &kb_limit)) continue;
        const int num_kb = min((pr.K + BK - 1) / BK, kb_limit);
        const int kb0 = kslice_of(pr, at.slab) * pr.kb_per_split, kb1 = min(num_kb, kb0 + pr.kb_per_split);
        const int ga = g * pr.a_gmul, gb = g * pr.b_gmul;
        if (pr.wait_ctr) {
          // A is the output of the problem before this one: wait until every chunk of these rows
          // has been stored (the storers count them), then order the copies below after that
          const unsigned* ctr = pr.wait_ctr + (long long)g * pr.m_tiles + at.mt;
          const long long t0 = clock64();
          while ((int)(ld_acquire(ctr) - pr.wait_target) < 0) {
            if (*abortp) { ok = false; break; }
            if (clock64() - t0 > kWaitLimitCycles) {
              *abortp = 1;
              report(a.status, -6, SITE_TC_PIPE, 8);
              ok = false;
              break;
            }
            __nanosleep(64);
          }
          if (!ok) break;
          fence_proxy_async_all();
        }
        const bool sums = kSums && sums_bias(pr, at);   // the summing warps read this tile's B stages
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % STAGES;
          ok = mbar_wait(&empty_bar[s], ((it / STAGES) & 1) ^ 1, abortp, a.status, 1);
          if (!ok) break;
          if (kSums) {
            // a stage that a summing tile filled last is free once the summing warps have read it
            // too; they signal per stage, so bit s of sum_parity is the phase to wait for next
            if ((sum_pending >> s) & 1u) {
              ok = mbar_wait(&sum_done[s], (sum_parity >> s) & 1u, abortp, a.status, 12);
              if (!ok) break;
              sum_parity ^= 1u << s;
              sum_pending &= ~(1u << s);
            }
            if (sums) sum_pending |= 1u << s;
          }
          uint8_t* sa = smem + s * STAGE_BYTES;
          uint8_t* sb = sa + A_BYTES;
          if (PAIR == 2) {
            // both CTAs' copies complete on the leader's barrier, which expects the bytes of both
            const uint32_t bar = map_to_cta(&full_bar[s], 0);
            if (rank == 0) mbar_expect_tx(&full_bar[s], 2 * STAGE_BYTES);
            if (A_MN) {
#pragma unroll
              for (int j = 0; j < BM / 64; ++j)
                tma_load_3d_pair(sa + j * (BK * 128), tmA, bar, m0 + 64 * j, kb * BK, ga);
            } else {
              tma_load_3d_pair(sa, tmA, bar, kb * BK, m0, ga);
            }
            if (B_MN) {
#pragma unroll
              for (int j = 0; j < BNL / 64; ++j)
                tma_load_3d_pair(sb + j * (BK * 128), tmB, bar, n0 + 64 * j, kb * BK, gb);
            } else {
              tma_load_3d_pair(sb, tmB, bar, kb * BK, n0, gb);
            }
          } else {
            mbar_expect_tx(&full_bar[s], STAGE_BYTES);
            if (A_MN) {
#pragma unroll
              for (int j = 0; j < BM / 64; ++j)
                tma_load_3d(sa + j * (BK * 128), tmA, &full_bar[s], m0 + 64 * j, kb * BK, ga);
            } else {
              tma_load_3d(sa, tmA, &full_bar[s], kb * BK, m0, ga);
            }
            if (B_MN) {
#pragma unroll
              for (int j = 0; j < BNL / 64; ++j)
                tma_load_3d(sb + j * (BK * 128), tmB, &full_bar[s], n0 + 64 * j, kb * BK, gb);
            } else {
              tma_load_3d(sb, tmB, &full_bar[s], kb * BK, n0, gb);
            }
          }
        }
      }
      if (!ok && rank == 0) {
        // let copies already in flight land before the CTA's shared memory goes away (a peer CTA
        // is held by the closing cluster barrier until the leader has got here)
        for (int j = max(0, it - STAGES); j < it; ++j) {
          long long t0 = clock64();
          while (!mbar_try_wait(&full_bar[j % STAGES], (j / STAGES) & 1) && clock64() - t0 < kWaitLimitCycles) {}
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issue
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = make_idesc(A_MN, B_MN, BN, BM * PAIR);
      int it = 0, j = 0, pi = 0, sit = 0;
      bool ok = true;
      for (int tile = unit; tile < total_tiles && ok; tile += n_units) {
        const TileAt at = locate(a, tile, pi);
        const TcProblem& pr = a.p[pi];
        int kb_limit;
        if (!tile_live<BM * PAIR, BN>(pr, at, group_of(pr, at.slab), &kb_limit)) continue;
        const int b = j & 1;
        ok = mbar_wait(&acc_empty[b], ((j >> 1) & 1) ^ 1, abortp, a.status, 2);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(b * BN);
        const int num_kb = min((pr.K + BK - 1) / BK, kb_limit);
        const int kb0 = kslice_of(pr, at.slab) * pr.kb_per_split;
        const int kb1 = min(num_kb, kb0 + pr.kb_per_split);
        const bool sums = kSums && sums_bias(pr, at);   // the summing warps follow this tile
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % STAGES;
          ok = mbar_wait(&full_bar[s], (it / STAGES) & 1, abortp, a.status, 3);
          if (!ok) break;
          tc_fence_after();
          if (kSums && sums) {
            // tell the summing warps that the stage is full; they have a ring of their own,
            // stepped once per stage of a summing tile, so that its phases stay in step with
            // them although they skip the other tiles
            mbar_arrive(&stage_here[sit % STAGES]);
            ++sit;
          }
          const uint32_t sa = smem_u32(smem + s * STAGE_BYTES), sb = sa + A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            // K-major: 16 k-elements = 32 bytes inside the swizzle row; 8-row groups 1024 B apart.
            // MN-major: 16 k-rows = 2048 B; 64-element MN chunks (one TMA box each) 8192 B apart.
            const uint64_t ad = A_MN ? make_desc(sa + k * 2048, BK * 128, 1024) : make_desc(sa + k * 32, 16, 1024);
            const uint64_t bd = B_MN ? make_desc(sb + k * 2048, BK * 128, 1024) : make_desc(sb + k * 32, 16, 1024);
            if (PAIR == 2) tc_mma_pair(d_tmem, ad, bd, idesc, ((kb - kb0) | k) != 0);
            else tc_mma(d_tmem, ad, bd, idesc, ((kb - kb0) | k) != 0);
          }
          // frees the slot (in both CTAs of a pair) once these MMAs have read it
          if (PAIR == 2) tc_commit_pair(&empty_bar[s]); else tc_commit(&empty_bar[s]);

        }
        if (ok) {
          if (PAIR == 2) tc_commit_pair(&acc_full[b]); else tc_commit(&acc_full[b]);
        }
        ++j;
      }
    }
  } else if (warp < kAuxWarp) {
    // ---------------------------------------------------------------- epilogue
    const int q = warp & 3;                           // tensor-memory lane quarter of this warp
    const int wg = (warp - 2) >> 2;                   // this warp's group takes chunks with cq % NG == wg
    const int r = q * 32 + lane;                      // row of the tile owned by this thread
    int cq = 0, j = 0, pi = 0, pi_next = 0;
    bool ok = true;
    float run_max = -INFINITY;                        // EPI_LSE_PART: the reference exponent, see there
    // per-tile epilogue inputs, requested one tile ahead (see below)
    float next_bias[NCH];
    float next_lse = 0.f;
    int next_label = -1;
    TileAt at_next{};                                 // the tile the last prefetch located: the next one to work on
    auto prefetch_tile_inputs = [&](int tile) {
      const TileAt at = at_next = locate(a, tile, pi_next);
      const TcProblem& pr = a.p[pi_next];
      const int n0 = at.nt * BN;
      if (EPI == EPI_BIAS_RELU || EPI == EPI_BIAS_F32) {
        const float* bias = pr.bias ? pr.bias + (long long)group_of(pr, at.slab) * pr.bias_sg : nullptr;
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
          const int n = n0 + c * CH + lane;
          next_bias[c] = (bias && n < pr.N) ? __ldg(bias + n) : 0.f;
        }
      }
      if (EPI == EPI_LSE_PART || EPI == EPI_SOFTMAX_DELTA) {
        // the softmax passes read the chunk's bias values straight from memory (warp-uniform
        // 16-byte loads): one warp asks for the next tile's eight lines into L1 a tile ahead
        if (warp == 2 && lane < BN * 4 / 128 && pr.bias && n0 + 32 * lane < pr.N)
          asm volatile("prefetch.global.L1 [%0];" ::"l"(pr.bias + (long long)at.slab * pr.bias_sg + n0 + 32 * lane));
      }
      if (EPI == EPI_SOFTMAX_DELTA) {
        const int row = at.mt * (BM * PAIR) + rank * BM + r;
        next_lse = row < pr.M ? __ldg(a.lse + (long long)at.slab * a.lse_sg + row) : 0.f;
        next_label = row < pr.M ? __ldg(a.labels + (long long)at.slab * a.labels_sg + row) : -1;
      }
    };
#pragma unroll
    for (int c = 0; c < NCH; ++c) next_bias[c] = 0.f;
    if (unit < total_tiles) prefetch_tile_inputs(unit);
    for (int tile = unit; tile < total_tiles && ok; tile += n_units) {
      const TileAt at = at_next;                      // located when its inputs were requested
      pi = at.pi;
      {
        int kb_limit;
        if (!tile_live<BM * PAIR, BN>(a.p[pi], at, group_of(a.p[pi], at.slab), &kb_limit)) {
          // the inputs requested for this tile are dropped; ask for the next tile's
          if (tile + n_units < total_tiles) prefetch_tile_inputs(tile + n_units);
          continue;
        }
      }
      const int pN = a.p[pi].N, pNt = a.p[pi].n_true, pM = a.p[pi].M, p_ntiles = a.p[pi].n_tiles;
      // a narrow fp32 head works in 16-column chunks: 128 x 16 floats fill the bf16 area of a slot
      const bool head = EPI == EPI_BIAS_RELU && a.p[pi].head_f32;
      const int cw = head ? CH / 2 : CH, nch = head ? 2 * NCH : NCH;
      const int n0 = at.nt * BN;
      const int g = at.slab;                          // output slab (group, k slice)
      const int b = j & 1;
      // Bias of the tile's columns: lane l keeps column 32 * c + l of every chunk c, and the chunk
      // code reads the 32 values of its chunk with warp shuffles.  The values (and the per-row
      // inputs of the softmax pass) were requested one tile ahead, so that their L2 round trip is
      // not paid inside a tile; the requests for the next tile go out now.
      float bias_reg[NCH];
#pragma unroll
      for (int c = 0; c < NCH; ++c) bias_reg[c] = next_bias[c];
      const int row = at.mt * (BM * PAIR) + rank * BM + r;   // this thread's row of the output
      float run_sum = 0.f;                            // EPI_LSE_PART: over this warp group's chunks of the tile
      // softmax pass: log-sum-exp in the log2 domain, with the division by the batch size folded in
      const float row_lse = EPI == EPI_SOFTMAX_DELTA ? next_lse * kLog2e - log2f(a.inv_rows) : 0.f;
      const int row_label = next_label;
      if (tile + n_units < total_tiles) prefetch_tile_inputs(tile + n_units);
      // warp-uniform outcome: the tensor-memory loads below need the whole warp
      ok = __all_sync(0xffffffffu, mbar_wait(&acc_full[b], (j >> 1) & 1, abortp, a.status, 4));
      if (!ok) break;
      tc_fence_after();
#pragma unroll 1
      for (int c = 0; c < nch; ++c, ++cq) {
        const int nc = n0 + c * cw;
        if (nc >= pN) break;                          // CTA-uniform
        // A slot always belongs to the same warp group, so that the group sees the slot's barrier
        // phases in order (a parity wait cannot tell phase p from phase p + 2); every configuration
        // that stores through the ring has a multiple of NG slots, so the groups take turns.
        static_assert(!kStore || NS % NG == 0, "slot ring: a whole number of slots per warp group");
        if ((cq % NG) != wg) continue;
        const int slot = cq % NS;
        uint8_t* f32 = slots + slot * SLOT_BYTES;
        uint8_t* b16 = f32 + F32_BYTES;
        // the slot is ready: loaded (input chunk) or drained by the store of an earlier chunk
        if (kStore) {
          if (ET::kAux) ok = mbar_wait(&slot_full[slot], (cq / NS) & 1, abortp, a.status, 5);
          else ok = mbar_wait(&slot_empty[slot], ((cq / NS) & 1) ^ 1, abortp, a.status, 5);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
        }
        uint32_t acc[32];
        if (head) {
          // plain product (a k slice of the logits; bias and the sum over slices come later)
          tc_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * BN + c * cw), acc);
#pragma unroll
          for (int u = 0; u < 4; ++u)
            *b16_unit(b16, r, u) = make_uint4(acc[4 * u], acc[4 * u + 1], acc[4 * u + 2], acc[4 * u + 3]);
          fence_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive(&chunk_done[slot]);
          continue;
        }
        tc_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * BN + c * CH), acc);
        if (EPI == EPI_SGD) {
#pragma unroll
          for (int u = 0; u < 4; ++u) {               // 8 columns per iteration
            float w[8];
            float4* p0 = f32_unit(f32, r, 2 * u);
            float4* p1 = f32_unit(f32, r, 2 * u + 1);
            float4 w0 = *p0, w1 = *p1;
            w[0] = w0.x - a.lr * __uint_as_float(acc[8 * u + 0]);
            w[1] = w0.y - a.lr * __uint_as_float(acc[8 * u + 1]);
            w[2] = w0.z - a.lr * __uint_as_float(acc[8 * u + 2]);
            w[3] = w0.w - a.lr * __uint_as_float(acc[8 * u + 3]);
            w[4] = w1.x - a.lr * __uint_as_float(acc[8 * u + 4]);
            w[5] = w1.y - a.lr * __uint_as_float(acc[8 * u + 5]);
            w[6] = w1.z - a.lr * __uint_as_float(acc[8 * u + 6]);
            w[7] = w1.w - a.lr * __uint_as_float(acc[8 * u + 7]);
            *p0 = make_float4(w[0], w[1], w[2], w[3]);
            *p1 = make_float4(w[4], w[5], w[6], w[7]);
            *b16_unit(b16, r, u) = pack8(w);
          }
        } else if (EPI == EPI_RELU_MASK) {
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            float mk[8], o[8];
            uint4* pm = b16_unit(b16, r, u);
            unpack8(*pm, mk);
#pragma unroll
            for (int e = 0; e < 8; ++e) o[e] = mk[e] > 0.f ? __uint_as_float(acc[8 * u + e]) : 0.f;
            *pm = pack8(o);
          }
        } else if (EPI == EPI_LSE_PART || EPI == EPI_SOFTMAX_DELTA) {
          // z = C + bias; every exponential is one ex2 of z * log2(e) minus a per-row constant,
          // which is the multiply-add that follows the bias addition.  The bias values of the
          // chunk are the same for every row: warp-uniform 16-byte loads, served by L1.
          float z[32];
          {
            const float* bias = a.p[pi].bias ? a.p[pi].bias + (long long)g * a.p[pi].bias_sg + nc : nullptr;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const float4 bv = (bias && nc + 4 * u < pN) ? __ldg(reinterpret_cast<const float4*>(bias) + u)
                                                          : make_float4(0.f, 0.f, 0.f, 0.f);
              z[4 * u + 0] = __uint_as_float(acc[4 * u + 0]) + bv.x;
              z[4 * u + 1] = __uint_as_float(acc[4 * u + 1]) + bv.y;
              z[4 * u + 2] = __uint_as_float(acc[4 * u + 2]) + bv.z;
              z[4 * u + 3] = __uint_as_float(acc[4 * u + 3]) + bv.w;
            }
          }
          if (EPI == EPI_LSE_PART) {
            // (ref, sum of 2^(z log2e - ref)) of this row over the chunks this warp group sees.
            // ref need not be the maximum: it only has to keep the sum inside the fp32 range.  It
            // stays where it is, from chunk to chunk and from tile to tile (another row's logits
            // are of the same size as a rule), while a chunk's sum comes out moderate, and moves
            // to the chunk's maximum otherwise (always for a thread's first chunk, where it is
            // still -inf).  The common case costs no comparison per element.
            if (nc + CH > pNt) {                         // CTA-uniform: the last, ragged chunk
#pragma unroll
              for (int e = 0; e < 32; ++e)
                if (nc + e >= pNt) z[e] = -INFINITY;     // pad columns do not count
            }
            // four independent chains, so that the ex2 and the sums overlap
            float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int e = 0; e < 32; ++e) s4[e & 3] += ex2_approx(fmaf(z[e], kLog2e, -run_max));
            float cs = (s4[0] + s4[1]) + (s4[2] + s4[3]);
            // Too large (2^64 or more; the exponent field also catches infinities and NaN, inf - inf
            // on the pad columns of a thread's first chunk), or too small (below 2^-64) at the
            // start of a tile: take the reference from this chunk.  A small chunk sum later in a
            // tile is simply added: the tile's sum so far is at least 2^-64 and dwarfs what a
            // flush to zero could lose.
            const uint32_t cs_exp = (__float_as_uint(cs) >> 23) & 0xffu;
            if (cs_exp >= 127u + 64u || (cs_exp < 127u - 64u && run_sum == 0.f)) {
              float m4[4] = {z[0], z[1], z[2], z[3]};
#pragma unroll
              for (int e = 4; e < 32; ++e) m4[e & 3] = fmaxf(m4[e & 3], z[e]);
              // finite: column nc is a column of the product (N is padded by less than a chunk)
              const float mn = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])) * kLog2e;
              // the tile's sum so far moves to the new reference, which is higher if there is a sum
              if (run_sum != 0.f) run_sum *= ex2_approx(run_max - mn);
              run_max = mn;
              s4[0] = s4[1] = s4[2] = s4[3] = 0.f;
#pragma unroll
              for (int e = 0; e < 32; ++e) s4[e & 3] += ex2_approx(fmaf(z[e], kLog2e, -mn));
              cs = (s4[0] + s4[1]) + (s4[2] + s4[3]);
            }
            run_sum += cs;
          } else {
            // softmax / rows = 2^(z log2e - (lse log2e + log2 rows))
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              float o[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) o[e] = ex2_approx(fmaf(z[8 * u + e], kLog2e, -row_lse));
              *b16_unit(b16, r, u) = pack8(o);
            }
            if (nc + CH > pNt) {                         // zero the pad columns of the ragged chunk
#pragma unroll
              for (int e = 0; e < 32; ++e)
                if (nc + e >= pNt)
                  reinterpret_cast<bf16*>(b16_unit(b16, r, e >> 3))[e & 7] = __float2bfloat16_rn(0.f);
            }
            const int lat = row_label - nc;              // the label's column, if it is in this chunk
            if (lat >= 0 && lat < CH && row < pM) {
              float zl = 0.f;
#pragma unroll
              for (int e = 0; e < 32; ++e)
                if (e == lat) zl = z[e];
              reinterpret_cast<bf16*>(b16_unit(b16, r, lat >> 3))[lat & 7] =
                  __float2bfloat16_rn(ex2_approx(fmaf(zl, kLog2e, -row_lse)) - a.inv_rows);
              a.label_logit[(long long)g * a.lse_sg + row] = zl;
            }
          }
        } else {
          float bl = 0.f;   // this lane's bias value of chunk c (zero for a k slice of a split product)
#pragma unroll
          for (int i = 0; i < NCH; ++i)
            if (i == c) bl = bias_reg[i];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            float o[8];
#pragma unroll
            for (int e = 0; e < 8; ++e)
              o[e] = __uint_as_float(acc[8 * u + e]) + __shfl_sync(0xffffffffu, bl, 8 * u + e);
            if (EPI == EPI_BIAS_RELU) {
#pragma unroll
              for (int e = 0; e < 8; ++e) o[e] = fmaxf(o[e], 0.f);
              *b16_unit(b16, r, u) = pack8(o);
            } else {
              *f32_unit(f32, r, 2 * u) = make_float4(o[0], o[1], o[2], o[3]);
              *f32_unit(f32, r, 2 * u + 1) = make_float4(o[4], o[5], o[6], o[7]);
            }
          }
        }
        if (kStore) {
          fence_async_smem();          // generic-proxy writes -> visible to the TMA store
          __syncwarp();
          if (lane == 0) mbar_arrive(&chunk_done[slot]);
        }
      }
      if (!ok) break;
      if (EPI == EPI_LSE_PART && row < pM) {
        // one partial per tile and warp group, combined by lse_combine
        a.lse_part[((long long)g * (NG * p_ntiles) + NG * at.nt + wg) * pM + row] = make_float2(run_max, run_sum);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {   // the accumulator is free again: tell the CTA that issues the MMAs
        if (PAIR == 2) mbar_arrive_cluster<!(EPI == EPI_LSE_PART || EPI == EPI_SOFTMAX_DELTA)>(map_to_cta(&acc_empty[b], 0));
        else mbar_arrive(&acc_empty[b]);
      }
      ++j;
    }
  } else if (ET::kAux && warp == kAuxWarp) {
    // ---------------------------------------------------------------- epilogue input loads
    if (lane == 0) {
      int cq = 0, pi = 0;
      bool ok = true;
      for (int tile = unit; tile < total_tiles && ok; tile += n_units) {
        const TileAt at = locate(a, tile, pi);
        {
          int kb_limit;
          if (!tile_live<BM * PAIR, BN>(a.p[pi], at, group_of(a.p[pi], at.slab), &kb_limit)) continue;
        }
        const int pN = a.p[pi].N;
        const int m0 = at.mt * (BM * PAIR) + rank * BM;
        const int n0 = at.nt * BN;
        const int g = at.slab;
        for (int c = 0; c < NCH; ++c, ++cq) {
          const int nc = n0 + c * CH;
          if (nc >= pN) break;
          const int slot = cq % NS;
          ok = mbar_wait(&slot_empty[slot], ((cq / NS) & 1) ^ 1, abortp, a.status, 6);
          if (!ok) break;
          mbar_expect_tx(&slot_full[slot], AUX_BYTES);
          if (EPI == EPI_SGD) tma_load_3d(slots + slot * SLOT_BYTES, &maps.c32[pi], &slot_full[slot], nc, m0, g);
          else tma_load_3d(slots + slot * SLOT_BYTES + F32_BYTES, &maps.aux16[pi], &slot_full[slot], nc, m0, g);
        }
      }
      if (!ok) {
        for (int jq = max(0, cq - NS); jq < cq; ++jq) {
          long long t0 = clock64();
          while (!mbar_try_wait(&slot_full[jq % NS], (jq / NS) & 1) && clock64() - t0 < kWaitLimitCycles) {}
        }
      }
    }
  } else if (warp < kStoreWarp0 + kStoreWarps) {
    // ---------------------------------------------------------------- chunk stores
    if (kStore && lane == 0) {
      const int sj = warp - kStoreWarp0;
      int cq = 0, pi = 0, pi_next = 0;
      bool ok = true;
      for (int tile = unit; tile < total_tiles && ok; tile += n_units) {
        const TileAt at = locate(a, tile, pi);
        const TcProblem& pr = a.p[pi];
        {
          int kb_limit;
          if (!tile_live<BM * PAIR, BN>(pr, at, group_of(pr, at.slab), &kb_limit)) {
            // A skipped tile still counts towards its row block, so that the rows' readers wait for
            // the same total whatever the group's extent (they never read behind the extent).
            if (pr.signal_ctr && sj == 0) {
              const int live = min(NCH, (pr.N - at.nt * BN + CH - 1) / CH);
              if (live > 0)
                red_release_add(pr.signal_ctr + (long long)group_of(pr, at.slab) * pr.m_tiles + at.mt, (unsigned)live);
            }
            continue;
          }
        }
        const int m0 = at.mt * (BM * PAIR) + rank * BM;
        const int n0 = at.nt * BN;
        const int g = at.slab;
        unsigned stored = 0;                 // chunks of this tile this thread has stored
        const bool head = EPI == EPI_BIAS_RELU && pr.head_f32;
        const int cw = head ? CH / 2 : CH, nch = head ? 2 * NCH : NCH;
        for (int c = 0; c < nch; ++c, ++cq) {
          const int nc = n0 + c * cw;
          if (nc >= pr.N) break;
          const int slot = cq % NS;
          // a slot always belongs to the same storer, so that storer sees the slot's barrier
          // phases in order (a parity wait cannot tell phase p from phase p + 2)
          if (slot % kStoreWarps != sj) continue;
          ok = mbar_wait(&chunk_done[slot], (cq / NS) & 1, abortp, a.status, 7);
          if (!ok) break;
          uint8_t* f32 = slots + slot * SLOT_BYTES;
          if (head) {
            tma_store_3d(&maps.c32[pi], f32 + F32_BYTES, nc, m0, g);
          } else {
            if (ET::k32) tma_store_3d(&maps.c32[pi], f32, nc, m0, g);
            if (ET::k16) tma_store_3d(&maps.c16[pi], f32 + F32_BYTES, nc, m0, g);
          }
          tma_commit_group();
          ++stored;
          if (EPI == EPI_SGD && PAIR == 2) {
            // The same chunk of this unit's next tile is asked into L2 now, one tile ahead of its
            // load, so that the load finds it there.  The request is issued here, where the
            // thread would wait for its store anyway; issued by the loader it delayed the loads.
            // Only on CTA pairs: with single-CTA tiles (short contractions over slices one tile
            // high) the requests measured slower than going without.
            const int nt = tile + n_units;
            if (nt < total_tiles) {
              const TileAt nx = locate(a, nt, pi_next);
              const int pn = nx.nt * BN + c * CH;
              if (pn < a.p[pi_next].N)
                tma_prefetch_l2_3d(&maps.c32[pi_next], pn, nx.mt * (BM * PAIR) + rank * BM, nx.slab);
            }
          }
          // once the store has read the slot it can be refilled (by the loader) or rewritten (by
          // the epilogue warps); the write to global memory completes in the background
          tma_wait_read<0>();
          mbar_arrive(&slot_empty[slot]);
        }
        if (ok && pr.signal_ctr && stored) {
          // a later problem of this launch reads these rows: once this thread's stores of the tile
          // have completed, add them to the row block's count (release: the reader acquires it)
          tma_wait_all();
          fence_proxy_async_all();
          red_release_add(pr.signal_ctr + (long long)group_of(pr, g) * pr.m_tiles + at.mt, stored);
        }
      }
      tma_wait_all();                // all stores complete before the CTA exits
    }
  }
  if (has_sum_warps(EPI) && warp >= kStoreWarp0 + kStoreWarps) {
    // ---------------------------------------------------------------- bias gradient (and loss means)
    // Two ways, chosen by the host per launch.  From memory (bias_mem): while the deltas of a step
    // are small enough to be still in L2, the summing warps of all CTAs share out (group, 64
    // columns) items and read them with plain loads, sixteen rows in flight per lane, at their own
    // pace beside the tiles: no barrier of the pipeline knows of them.  From shared memory
    // (bias_upd, single CTAs): deltas that no longer fit in L2 would come from DRAM a second time,
    // so there the warps read them out of the B stages as they pass:
    // summing warp sw owns the 64-column box sw of the B tile (MN-major: row k of a box holds 64
    // consecutive columns, 128 bytes, 16-byte units swizzled by k % 8); lane l adds up columns
    // 8 (l % 8) .. + 7 over the rows k = l / 8 (mod 4), and the four lanes of a column combine
    // their sums at the end of the tile.  Only the first tile row carries a bias update
    // (sums_bias); the summing warps step over the stages of all other tiles.  A stage of a
    // summing tile is released by the MMA commit and by both summing warps (sum_done, which the
    // loading thread waits for before it refills such a stage).  The MMA thread, which sees every
    // stage fill up, passes the completions of a summing tile on through the stage_here ring.
    // The ring is stepped once per stage of a summing tile and the MMA thread cannot be STAGES
    // steps ahead (refilling a stage needs the summing warps' arrival), so a parity wait on it
    // is unambiguous, which one on full_bar would not be for warps that skip tiles.
    const int sw = warp - (kStoreWarp0 + kStoreWarps);
    if (rank == 0 && sw == kSumWarps - 1 && a.loss.loss_out) {
      for (int g = unit; g < a.loss_G; g += n_units) {
        float acc = 0.f;
        for (int b = lane; b < a.loss_B; b += 32) acc += __ldg(a.loss.row_loss + (long long)g * a.loss_B + b);
#pragma unroll
        for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) a.loss.loss_out[(long long)g * a.loss.out_stride + a.loss.k] = acc / (float)a.loss_B;
      }
    }
    if (a.n_bias_items > 0) {
      const int n_workers = (int)gridDim.x * kSumWarps;
      int pj = 0;
      for (int item = (int)blockIdx.x * kSumWarps + sw; item < a.n_bias_items; item += n_workers) {
        while (item >= a.p[pj].bias_item_end) ++pj;
        const TcProblem& pr = a.p[pj];
        const int li = item - (pj ? a.p[pj - 1].bias_item_end : 0);
        const int blocks = (pr.bias_n + 63) / 64;            // column blocks of a group
        const int g = li / blocks, c0 = (li - g * blocks) * 64 + 2 * lane;   // this lane's two columns
        if (c0 >= pr.bias_n) continue;                       // rows are padded to an even length
        const uint32_t* dp = reinterpret_cast<const uint32_t*>(pr.dmem + (long long)g * pr.dmem_sg + c0);
        const long long ld2 = pr.dmem_ld / 2;
        float acc0 = 0.f, acc1 = 0.f;
        for (int r0 = 0; r0 < pr.K; r0 += 16) {              // the contraction of a weight update runs over the batch
          uint32_t v[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) v[i] = r0 + i < pr.K ? __ldg(dp + (long long)(r0 + i) * ld2) : 0u;
#pragma unroll
          for (int i = 0; i < 16; ++i) {                     // rows in ascending order: a fixed sum
            acc0 += __uint_as_float(v[i] << 16);
            acc1 += __uint_as_float(v[i] & 0xffff0000u);
          }
        }
        float* bp = pr.bias_mem + (long long)g * pr.bias_upd_sg + c0;
        bp[0] -= a.lr * acc0;
        if (c0 + 1 < pr.bias_n) bp[1] -= a.lr * acc1;
      }
    }
    constexpr int kBoxes = BNL / 64;
    static_assert(!kSums || kBoxes <= kSumWarps, "one summing warp per 64-column box");
    int it = 0, pi = 0, sit = 0;
    bool ok = true;
    for (int tile = unit; kSums && tile < total_tiles && ok; tile += n_units) {
      const TileAt at = locate(a, tile, pi);
      const TcProblem& pr = a.p[pi];
      int kb_limit;
      if (!tile_live<BM * PAIR, BN>(pr, at, at.slab, &kb_limit)) continue;
      const int num_kb = min((pr.K + BK - 1) / BK, kb_limit);
      if (!sums_bias(pr, at)) {
        it += num_kb;
        continue;
      }
      const bool sum = sw < kBoxes;
      const int u = lane & 7, rq = lane >> 3;   // this lane's 16-byte unit (8 columns) and row quarter
      float acc[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] = 0.f;
      for (int kb = 0; kb < num_kb; ++kb, ++it, ++sit) {
        const int s = it % STAGES;
        const uint32_t par = (sit / STAGES) & 1;
        ok = mbar_wait(&stage_here[sit % STAGES], par, abortp, a.status, 10);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        if (sum) {
          // one instruction reads four rows of the box (512 contiguous bytes, every bank once)
          const uint8_t* box = smem + s * STAGE_BYTES + A_BYTES + sw * (BK * 128);
#pragma unroll
          for (int i = 0; i < BK / 4; ++i) {
            const int k = 4 * i + rq;
            float v[8];
            unpack8(*reinterpret_cast<const uint4*>(box + k * 128 + ((u ^ (k & 7)) << 4)), v);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] += v[e];
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sum_done[s]);
      }
      if (ok && sum) {
#pragma unroll
        for (int e = 0; e < 8; ++e) {             // the four row quarters of a column, in a fixed order
          acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], 8);
          acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], 16);
        }
        if (rq == 0) {
          const int n = at.nt * BN + rank * BNL + sw * 64 + 8 * u;
          float* bp = pr.bias_upd + (long long)at.slab * pr.bias_upd_sg + n;
#pragma unroll
          for (int e = 0; e < 8; ++e)
            if (n + e < pr.bias_n) bp[e] -= a.lr * acc[e];
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR == 2) cluster_sync_all();   // neither CTA leaves while the other may still touch its memory
  if (warp == 1) {
    __syncwarp();
    if (PAIR == 2)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS)
                   : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS)
                   : "memory");
  }
}

// Self-test of the bounded wait: one thread waits on a barrier that nothing ever signals, with
// the given limit, so the wait has to give up, record the status and return.  where = 99.
__global__ void wait_expiry_kernel(DeviceStatus* st, long long limit_cycles) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) mbar_wait(&bar, 0, &abort_flag, st, 99, limit_cycles);
  __syncthreads();
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

int sm_count() {
  static int n = 0;
  static std::once_flag once;
  std::call_once(once, [] {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
      n = 148;
  });
  return n;
}

// Tensor [groups][outer][inner] (inner contiguous, strides in elements) with box
// {box_inner, box_outer, 1}.  elem_bytes 2 = bf16, 4 = fp32.  swizzle_bytes 128 or 64.
using MapKey = std::tuple<const void*, long long, long long, long long, long long, long long, int, int, int, int>;
std::map<MapKey, CUtensorMap>& map_cache() {
  static std::map<MapKey, CUtensorMap> c;
  return c;
}
std::mutex& map_mutex() {
  static std::mutex m;
  return m;
}

bool make_map(CUtensorMap* out, const void* base, int elem_bytes, long long inner, long long outer,
              long long groups, long long outer_stride, long long group_stride, int box_inner, int box_outer,
              int swizzle_bytes) {
  if (!base) return false;
  MapKey key{base, inner, outer, groups, outer_stride, group_stride, elem_bytes, box_inner, box_outer, swizzle_bytes};
  std::lock_guard<std::mutex> lk(map_mutex());
  auto& cache = map_cache();
  auto it = cache.find(key);
  if (it != cache.end()) {
    *out = it->second;
    return true;
  }
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  // The encoder is a driver call and wants the device's context current on the calling thread; a
  // thread that has made no runtime call yet has none (the launches that follow would bind it, but
  // they come after this).
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaSetDevice(dev) != cudaSuccess) return false;
  cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)outer, (cuuint64_t)groups};
  cuuint64_t strides[2] = {(cuuint64_t)outer_stride * elem_bytes,
                           (cuuint64_t)(groups > 1 ? group_stride : outer_stride * outer) * elem_bytes};
  cuuint32_t box[3] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(out, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3,
                  const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  if (cache.size() > 4096) cache.clear();
  cache[key] = *out;
  return true;
}

template <int A_MN, int B_MN, int BN, int STAGES, int NS, int EPI, int PAIR>
bool launch(const Launch& L, const TcMaps& m, const TcArgs& t) {
  using ET = EpiTraits<EPI>;
  constexpr int slot_bytes = (ET::k32 ? BM * CH * 4 : 0) + (ET::k16 ? BM * CH * 2 : 0);
  constexpr int smem = STAGES * (BM * BK * 2 + (BN / PAIR) * BK * 2) + NS * slot_bytes + 1024;
  static_assert(smem <= 227 * 1024 - 512, "shared memory budget exceeded");
  auto kern = gemm_tc_kernel<A_MN, B_MN, BN, STAGES, NS, EPI, PAIR>;
  // CTAs (PAIR = 1) or clusters (PAIR = 2) that can be resident at once; looked up by whichever
  // host thread launches this instance first
  static int max_units = 0;
  static std::once_flag once;
  std::call_once(once, [&] {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return;
    if (PAIR == 2) {
      cudaLaunchConfig_t probe{};
      probe.gridDim = dim3(2 * (sm_count() / 2));
      probe.blockDim = dim3(threads_for(EPI, PAIR));
      probe.dynamicSmemBytes = smem;
      cudaLaunchAttribute attr{};
      attr.id = cudaLaunchAttributeClusterDimension;
      attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
      probe.attrs = &attr;
      probe.numAttrs = 1;
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, kern, &probe) != cudaSuccess || n <= 0) return;
      max_units = n < sm_count() / 2 ? n : sm_count() / 2;
    } else {
      max_units = sm_count();
    }
  });
  if (max_units <= 0) return false;
  const int total = t.total_tiles;
  const int units = total < max_units ? total : max_units;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(PAIR * units);
  cfg.blockDim = dim3(threads_for(EPI, PAIR));
  cfg.dynamicSmemBytes = smem;
  cfg.stream = L.stream;
  cudaLaunchAttribute attrs[2];
  int n_attrs = 0;
  // the kernel's prologue may overlap the tail of the kernel before it (see griddepcontrol.wait)
  attrs[n_attrs].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attrs[n_attrs].val.programmaticStreamSerializationAllowed = 1;
  ++n_attrs;
  if (PAIR == 2) {
    attrs[n_attrs].id = cudaLaunchAttributeClusterDimension;
    attrs[n_attrs].val.clusterDim.x = 2; attrs[n_attrs].val.clusterDim.y = 1; attrs[n_attrs].val.clusterDim.z = 1;
    ++n_attrs;
  }
  cfg.attrs = attrs;
  cfg.numAttrs = n_attrs;
  if (cudaLaunchKernelEx(&cfg, kern, m, t) != cudaSuccess) return false;
  L.count();
  return true;
}

}  // namespace

bool gemm_tc_wait_selftest(const Launch& L, DeviceStatus* st, long long limit_cycles) {
  wait_expiry_kernel<<<1, 32, 0, L.stream>>>(st, limit_cycles);
  L.count();
  return cudaGetLastError() == cudaSuccess;
}

// Tile shape.  Pairs of CTAs (256 x 256 tiles) are used when the problem has enough of them to
// give every SM pair work; otherwise single CTAs with the widest of 256 / 128 / 64 columns that
// still gives every SM a tile.  The weight-update epilogue keeps a chunk ring in shared memory
// and stays at 128 columns when it runs on single CTAs.  A batch of problems is judged by the
// tiles of all of them together and must have one problem that qualifies for pairs by itself
// (more than 128 rows and columns); the small ones then ride along on the same shape.
struct TileChoice { int bn, pair; };
TileChoice pick_tile(const GemmArgs<bf16>* a, int n, int epi) {
  const int sms = sm_count();
  auto n_store = [&](int i) { return a[i].N_store > 0 ? a[i].N_store : a[i].N; };
  auto tiles = [&](int bm, int bn) {
    int64_t s = 0;
    for (int i = 0; i < n; ++i)
      s += ceil_div(a[i].M, bm) * ceil_div(n_store(i), bn) * a[i].G * (a[i].k_splits > 1 ? a[i].k_splits : 1);
    return s;
  };
  bool pair_ok = false, wide = false, mid = false;
  for (int i = 0; i < n; ++i) {
    pair_ok |= a[i].M > BM && n_store(i) > 128;
    wide |= n_store(i) > 128;
    mid |= n_store(i) > 64;
  }
  if (pair_ok && 4 * tiles(2 * BM, 256) >= 3 * (sms / 2)) return {256, 2};
  if (epi == EPI_SGD) return {(mid && tiles(BM, 128) >= sms) ? 128 : 64, 1};
  if (wide && tiles(BM, 256) >= sms) return {256, 1};
  if (mid && tiles(BM, 128) >= sms) return {128, 1};
  return {64, 1};
}

// Partials per row the EPI_LSE_PART epilogue writes: one per 256-column tile and warp group.
int gemm_tc_lse_parts(int64_t n_store) { return (epi_warps(EPI_LSE_PART) / 4) * (int)ceil_div(n_store, 256); }

// Number of k slices gemm_tc will really use when `want` are asked for (slices hold whole
// 64-deep k blocks, so the count can come out smaller).
int gemm_tc_splits(int K, int want) {
  if (want <= 1) return 1;
  const int64_t nkb = ceil_div(K, BK);
  return (int)ceil_div(nkb, ceil_div(nkb, want));
}

int gemm_tc_max_batch() { return kMaxProblems; }

// Whether a weight-update launch of these products would run on single CTAs, whose extra warps
// can sum the deltas for the bias update (GemmArgs::bias_upd) and reduce the step's losses.
bool gemm_tc_update_sums_bias(const GemmArgs<bf16>* a, int n) {
  return n >= 1 && n <= kMaxProblems && pick_tile(a, n, EPI_SGD).pair == 1;
}

// Counters a chain of n problems over G groups and up to max_rows output rows needs.
size_t gemm_tc_chain_counters(int n, int G, int max_rows) { return (size_t)n * G * ceil_div(max_rows, BM); }

// Multiplier and shift of div_by for the divisor d >= 1.
static void set_div(int d, uint32_t* mul, uint32_t* sh) {
  uint32_t s = 0;
  while ((1ull << s) < (unsigned long long)d) ++s;
  *sh = s;
  *mul = (uint32_t)((1ull << (31 + s)) / (unsigned long long)d + 1);
}

bool gemm_tc_batch(const Launch& L, const GemmArgs<bf16>* ga, int n, const GemmChain* chain, const LossReduce* loss,
                   DeviceStatus* st) {
  if (n < 1 || n > kMaxProblems) return false;
  const GemmArgs<bf16>& a0 = ga[0];
  const int epi = a0.epi;
  const bool a_mn = a0.a_sm == 1 && a0.a_sk != 1, b_mn = a0.b_sn == 1 && a0.b_sk != 1;
  // A narrow output layer may close a list of hidden forward layers: plain fp32 products (k slices
  // allowed) of at most 64 columns, written in 16-column chunks by the same kernel instance.
  const bool head = n > 1 && epi == EPI_BIAS_RELU && ga[n - 1].epi == EPI_BIAS_F32;
  if (head) {
    const GemmArgs<bf16>& h = ga[n - 1];
    if (h.bias || !h.outf || (h.N_store > 0 ? h.N_store : h.N) > 64) return false;
  }
  for (int i = 0; i < n; ++i) {
    const GemmArgs<bf16>& a = ga[i];
    const bool ai = a.a_sm == 1 && a.a_sk != 1, bi = a.b_sn == 1 && a.b_sk != 1;
    const bool is_head = head && i == n - 1;
    if ((a.epi != epi && !is_head) || ai != a_mn || bi != b_mn) return false;   // one kernel instance serves the batch
    if (!ai && a.a_sk != 1) return false;
    if (!bi && a.b_sk != 1) return false;
    if (n > 1 && a.k_splits > 1 && !is_head) return false;
  }
  if (n > 1 && epi != EPI_BIAS_RELU && epi != EPI_RELU_MASK && epi != EPI_SGD) return false;
  if (chain && (epi == EPI_SGD || n < 2 || !chain->counters || !chain->totals)) return false;
  TileChoice tc = pick_tile(ga, n, epi);
  if (epi == EPI_LSE_PART || epi == EPI_SOFTMAX_DELTA)   // the partials are laid out per 256-column tile
    tc = TileChoice{256, a0.M > BM ? 2 : 1};
  const int bn = tc.bn, pair = tc.pair;

  TcArgs t{};
  TcMaps m{};
  t.n_problems = n;
  t.lr = a0.lr;
  t.status = st;
  t.lse_part = reinterpret_cast<float2*>(a0.lse_part);
  t.lse = a0.lse; t.lse_sg = a0.lse_sg;
  t.labels = a0.labels; t.labels_sg = a0.labels_sg;
  t.label_logit = a0.label_logit;
  t.inv_rows = a0.inv_rows;
  if (loss && epi != EPI_SGD) return false;
  if (loss) {
    t.loss = *loss;
    t.loss_B = a0.K;          // the contraction of a weight update runs over the batch
    t.loss_G = a0.G;
  }
  int64_t tiles = 0, bias_items = 0;
  for (int i = 0; i < n; ++i) {
    const GemmArgs<bf16>& a = ga[i];
    const int n_store = a.N_store > 0 ? a.N_store : a.N;
    TcProblem& p = t.p[i];
    p.M = a.M; p.N = n_store; p.n_true = a.N; p.K = a.K;
    p.m_tiles = (int)ceil_div(a.M, BM * pair);
    p.n_tiles = (int)ceil_div(n_store, bn);
    set_div(p.m_tiles, &p.m_div, &p.m_sh);
    set_div(p.n_tiles, &p.n_div, &p.n_sh);
    p.G = a.G;
    p.k_splits = 1;
    p.kb_per_split = (int)ceil_div(a.K, BK);
    const bool is_head = head && i == n - 1;
    p.head_f32 = is_head ? 1 : 0;
    if (a.k_splits > 1) {
      if (a.epi != EPI_BIAS_F32 || a.bias) return false;   // slices are plain fp32 partial products
      p.kb_per_split = (int)ceil_div(ceil_div(a.K, BK), a.k_splits);
      p.k_splits = (int)ceil_div(ceil_div(a.K, BK), p.kb_per_split);
      if (p.k_splits != a.k_splits) return false;           // caller sizes its buffer with gemm_tc_splits()
    }
    p.a_gmul = (a.G > 1 && a.a_sg != 0) ? 1 : 0;
    p.b_gmul = (a.G > 1 && a.b_sg != 0) ? 1 : 0;
    p.bias = a.bias; p.bias_sg = a.bias_sg;
    p.m_off = a.m_off; p.n_off = a.n_off; p.k_off = a.k_off;
    if (a.bias_upd && epi != EPI_SGD) return false;
    p.bias_upd_sg = a.bias_upd_sg; p.bias_n = a.bias_n;
    p.bias_item_end = bias_items;
    if (a.bias_upd && a.bias_upd_from_memory) {
      if (!b_mn || a.b_sk % 2 != 0 || a.b_sg % 2 != 0 || reinterpret_cast<uintptr_t>(a.B) % 4 != 0) return false;
      p.bias_mem = a.bias_upd; p.dmem = a.B; p.dmem_ld = a.b_sk; p.dmem_sg = a.G > 1 ? a.b_sg : 0;
      bias_items += (int64_t)a.G * ceil_div(a.bias_n, 64);
      if (bias_items > 0x7fffffffll) return false;
      p.bias_item_end = (int)bias_items;
    } else if (a.bias_upd) {
      if (pair != 1) return false;   // sums from the B stages: single CTAs only, see gemm_tc_update_sums_bias
      p.bias_upd = a.bias_upd;
    }
    if (a.k_off && p.k_splits > 1) return false;
    tiles += (int64_t)p.m_tiles * p.n_tiles * p.G * p.k_splits;
    if (tiles > 0x7fffffffll) return false;
    p.tile_end = (int)tiles;
    if (a.lr != a0.lr) return false;

    // K-major operand: inner = K, outer = rows (M or N).  MN-major: inner = rows, outer = K.
    const long long gga = p.a_gmul ? a.G : 1, ggb = p.b_gmul ? a.G : 1;
    const bool ok_a = a_mn ? make_map(&m.a[i], a.A, 2, a.M, a.K, gga, a.a_sk, a.a_sg, 64, BK, 128)
                           : make_map(&m.a[i], a.A, 2, a.K, a.M, gga, a.a_sm, a.a_sg, 64, BM, 128);
    const bool ok_b = b_mn ? make_map(&m.b[i], a.B, 2, a.N, a.K, ggb, a.b_sk, a.b_sg, 64, BK, 128)
                           : make_map(&m.b[i], a.B, 2, a.K, a.N, ggb, a.b_sn, a.b_sg, 64, bn / pair, 128);
    if (!ok_a || !ok_b) return false;
    m.c32[i] = m.a[i]; m.c16[i] = m.a[i]; m.aux16[i] = m.a[i];   // placeholders for the maps an epilogue does not use
    // Output / epilogue-input chunks: [G][M][n_store] row-major, boxes of 128 rows x 32 columns.
    switch (epi) {
      case EPI_BIAS_RELU:
        if (a_mn || !b_mn) return false;
        if (is_head) {   // 128 x 16 fp32 chunks: 64-byte rows, like the bf16 chunks of the other problems
          if (!make_map(&m.c32[i], a.outf, 4, n_store, a.M, (long long)a.G * p.k_splits, a.outf_ld, a.outf_sg, CH / 2, BM, 64))
            return false;
        } else if (!make_map(&m.c16[i], a.out, 2, n_store, a.M, a.G, a.out_ld, a.out_sg, CH, BM, 64)) {
          return false;
        }
        break;
      case EPI_BIAS_F32:
        if (a_mn) return false;
        if (!make_map(&m.c32[i], a.outf, 4, n_store, a.M, (long long)a.G * p.k_splits, a.outf_ld, a.outf_sg, CH, BM, 128))
          return false;
        break;
      case EPI_LSE_PART:
        if (a_mn || !b_mn || a.k_splits > 1 || !a.lse_part) return false;
        break;
      case EPI_SOFTMAX_DELTA:
        if (a_mn || !b_mn || a.k_splits > 1 || !a.lse || !a.labels || !a.label_logit) return false;
        if (!make_map(&m.c16[i], a.out, 2, n_store, a.M, a.G, a.out_ld, a.out_sg, CH, BM, 64)) return false;
        break;
      case EPI_RELU_MASK:
        if (a_mn || b_mn) return false;
        if (!make_map(&m.c16[i], a.out, 2, n_store, a.M, a.G, a.out_ld, a.out_sg, CH, BM, 64)) return false;
        if (!make_map(&m.aux16[i], a.mask, 2, n_store, a.M, a.G, a.mask_ld, a.mask_sg, CH, BM, 64)) return false;
        break;
      case EPI_SGD:
        if (!a_mn || !b_mn || !a.opw) return false;
        if (!make_map(&m.c32[i], a.outf, 4, n_store, a.M, a.G, a.outf_ld, a.outf_sg, CH, BM, 128)) return false;
        if (!make_map(&m.c16[i], a.opw, 2, n_store, a.M, a.G, a.outf_ld, a.outf_sg, CH, BM, 64)) return false;
        break;
      default:
        return false;
    }
  }
  t.total_tiles = (int)tiles;
  t.n_bias_items = (int)bias_items;
  if (chain) {
    // Problem i + 1 reads problem i's output rows: same groups, same rows, hence the same tile rows.
    // Every CTA of a unit stores ceil(N / 32) chunks per (group, tile row) and launch; the running
    // totals are kept by the caller, who clears counters and totals together.
    for (int i = 0; i + 1 < n; ++i) {
      if (ga[i + 1].M != ga[i].M || ga[i + 1].G != ga[i].G || ga[i + 1].A != ga[i].out) return false;
      unsigned* ctr = chain->counters + (size_t)i * chain->stride;
      if ((size_t)t.p[i].G * t.p[i].m_tiles > chain->stride) return false;
      chain->totals[i] += (unsigned)(pair * ceil_div(t.p[i].N, CH));
      t.p[i].signal_ctr = ctr;
      t.p[i + 1].wait_ctr = ctr;
      t.p[i + 1].wait_target = chain->totals[i];
    }
  }

  switch (epi) {
    case EPI_BIAS_RELU:
      if (pair == 2) return launch<0, 1, 256, 6, 4, EPI_BIAS_RELU, 2>(L, m, t);
      if (bn == 256) return launch<0, 1, 256, 4, 4, EPI_BIAS_RELU, 1>(L, m, t);
      if (bn == 128) return launch<0, 1, 128, 6, 4, EPI_BIAS_RELU, 1>(L, m, t);
      return launch<0, 1, 64, 8, 4, EPI_BIAS_RELU, 1>(L, m, t);
    case EPI_BIAS_F32:
      if (!a_mn && !b_mn) {   // both operands K-major: k slices of delta * W^T
        if (pair == 2) return launch<0, 0, 256, 6, 2, EPI_BIAS_F32, 2>(L, m, t);
        if (bn == 256) return launch<0, 0, 256, 4, 2, EPI_BIAS_F32, 1>(L, m, t);
        if (bn == 128) return launch<0, 0, 128, 5, 4, EPI_BIAS_F32, 1>(L, m, t);
        return launch<0, 0, 64, 6, 4, EPI_BIAS_F32, 1>(L, m, t);
      }
      // a short contraction (wide output layer fed by a narrow hidden layer) is bound by writing
      // the logits: fewer operand stages, a deeper ring of output chunks
      if (pair == 2 && ceil_div(a0.K, BK) <= 4) return launch<0, 1, 256, 3, 6, EPI_BIAS_F32, 2>(L, m, t);
      if (pair == 2) return launch<0, 1, 256, 6, 2, EPI_BIAS_F32, 2>(L, m, t);
      if (bn == 256) return launch<0, 1, 256, 4, 2, EPI_BIAS_F32, 1>(L, m, t);
      if (bn == 128) return launch<0, 1, 128, 5, 4, EPI_BIAS_F32, 1>(L, m, t);
      return launch<0, 1, 64, 6, 4, EPI_BIAS_F32, 1>(L, m, t);
    case EPI_LSE_PART:
      if (pair == 2) return launch<0, 1, 256, 4, 1, EPI_LSE_PART, 2>(L, m, t);
      return launch<0, 1, 256, 3, 1, EPI_LSE_PART, 1>(L, m, t);
    case EPI_SOFTMAX_DELTA:
      if (pair == 2) return launch<0, 1, 256, 4, 8, EPI_SOFTMAX_DELTA, 2>(L, m, t);
      return launch<0, 1, 256, 3, 8, EPI_SOFTMAX_DELTA, 1>(L, m, t);
    case EPI_RELU_MASK:
      if (pair == 2) return launch<0, 0, 256, 6, 4, EPI_RELU_MASK, 2>(L, m, t);
      if (bn == 256) return launch<0, 0, 256, 4, 4, EPI_RELU_MASK, 1>(L, m, t);
      if (bn == 128) return launch<0, 0, 128, 6, 4, EPI_RELU_MASK, 1>(L, m, t);
      return launch<0, 0, 64, 8, 4, EPI_RELU_MASK, 1>(L, m, t);
    case EPI_SGD:
      if (pair == 2) return launch<1, 1, 256, 4, 4, EPI_SGD, 2>(L, m, t);
      if (bn == 128) return launch<1, 1, 128, 4, 4, EPI_SGD, 1>(L, m, t);
      return launch<1, 1, 64, 5, 4, EPI_SGD, 1>(L, m, t);
    default:
      return false;
  }
}

bool gemm_tc(const Launch& L, const GemmArgs<bf16>& a, DeviceStatus* st) {
  return gemm_tc_batch(L, &a, 1, nullptr, nullptr, st);
}

}  // namespace ist
