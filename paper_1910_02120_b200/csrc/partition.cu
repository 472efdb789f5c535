// Random balanced partition of a hidden layer's neurons into S groups (paper Sec. 2.1
// "Constructing Subnets"; App. A: sum_s m^(s)_{l,i} = 1).  Integer work only, and the result
// does not depend on scheduling (atomics are used only for counts and for placement inside a
// bucket, whose order does not enter the result).
//
// key_i   = (i+1)-th output of SplitMix64 seeded with the layer's stream seed
// rank_i  = #{ j : (key_j, j) < (key_i, i) }
// group_i = the group whose rank interval contains rank_i (sizes floor(N/S), +1 for the
//           first N mod S groups)
// pos_i   = #{ j < i : group_j = group_i }      (ascending order inside a group)
// idx[off[group_i] + pos_i] = i
//
// rank: the keys are uniform 64-bit numbers, so their top bits spread them evenly over ~N/8
// buckets; rank_i = (#keys in lower buckets) + (#smaller keys in i's own bucket).
// pos: neurons are walked in index order in blocks of 1024; a block counts its members per
// group (warp match + per-warp counters), and pos_i = members in earlier blocks + members
// earlier in this block.
#include "kernels.h"

namespace ist {
namespace {

constexpr int kThreads = 256;
constexpr int kPosBlock = 1024;

__device__ __forceinline__ uint64_t splitmix64_mix(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
__device__ __forceinline__ int bucket_of(uint64_t key, int log_buckets) {
  return log_buckets ? (int)(key >> (64 - log_buckets)) : 0;
}

__global__ void clear_kernel(int32_t* p, int n) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = 0;
}

__global__ void keys_kernel(uint64_t layer_seed, int N, int log_buckets, uint64_t* keys, int32_t* hist) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < N) {
    uint64_t k = splitmix64_mix(layer_seed + 0x9E3779B97F4A7C15ull * (uint64_t)(i + 1));
    keys[i] = k;
    atomicAdd(&hist[bucket_of(k, log_buckets)], 1);
  }
}

// One CTA: start[b] = sum of hist[0..b), start[nb] = N; cursor[b] = 0.
__global__ void bucket_scan_kernel(const int32_t* __restrict__ hist, int nb, int32_t* start, int32_t* cursor) {
  __shared__ int32_t warp_tot[32];
  __shared__ int32_t carry;
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  for (int base = 0; base < nb; base += blockDim.x) {
    int b = base + threadIdx.x;
    int v = b < nb ? hist[b] : 0;
    int incl = v;
    for (int o = 1; o < 32; o <<= 1) {
      int t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) warp_tot[w] = incl;
    __syncthreads();
    int woff = 0;
    for (int u = 0; u < w; ++u) woff += warp_tot[u];
    if (b < nb) {
      start[b] = carry + woff + incl - v;
      cursor[b] = 0;
    }
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) carry += woff + incl;
    __syncthreads();
  }
  if (threadIdx.x == 0) start[nb] = carry;
}

__global__ void place_kernel(int N, int log_buckets, const uint64_t* __restrict__ keys,
                             const int32_t* __restrict__ start, int32_t* cursor, uint64_t* skey, int32_t* sidx) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= N) return;
  uint64_t k = keys[i];
  int b = bucket_of(k, log_buckets);
  int at = start[b] + atomicAdd(&cursor[b], 1);
  skey[at] = k;
  sidx[at] = i;
}

// One CTA of kPosBlock threads per kPosBlock consecutive neurons: rank, group, position of each
// neuron among the block's members of its group (lp), and the block's member count per group.
__global__ void __launch_bounds__(kPosBlock) rank_group_kernel(
    int N, int S, int log_buckets, const uint64_t* __restrict__ keys, const int32_t* __restrict__ start,
    const uint64_t* __restrict__ skey, const int32_t* __restrict__ sidx, int32_t* grp, int32_t* lp,
    int32_t* blkcnt, int32_t* off) {
  extern __shared__ int32_t wcnt[];          // [32 warps][S]
  const int i = blockIdx.x * kPosBlock + threadIdx.x;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int q = N / S, r = N % S;
  for (int e = threadIdx.x; e < 32 * S; e += kPosBlock) wcnt[e] = 0;
  if (blockIdx.x == 0)
    for (int e = threadIdx.x; e <= S; e += kPosBlock) off[e] = e * q + min(e, r);
  __syncthreads();
  int g = -1;
  if (i < N) {
    const uint64_t ki = keys[i];
    const int b = bucket_of(ki, log_buckets);
    const int lo = start[b], hi = start[b + 1];
    int rk = lo;
    for (int p = lo; p < hi; ++p) {
      const uint64_t kj = skey[p];
      rk += (kj < ki) || (kj == ki && sidx[p] < i);
    }
    const int big = r * (q + 1);
    g = rk < big ? rk / (q + 1) : r + (rk - big) / q;
    grp[i] = g;
  }
  // members of the same group among the lower lanes of this warp
  const unsigned same = __match_any_sync(0xffffffffu, g);
  const int wpos = __popc(same & ((1u << lane) - 1u));
  if (g >= 0 && wpos == 0) wcnt[w * S + g] = __popc(same);   // one writer per (warp, group)
  __syncthreads();
  if (i < N) {
    int before = 0;
    for (int u = 0; u < w; ++u) before += wcnt[u * S + g];
    lp[i] = before + wpos;
  }
  for (int s = threadIdx.x; s < S; s += kPosBlock) {
    int tot = 0;
    for (int u = 0; u < 32; ++u) tot += wcnt[u * S + s];
    blkcnt[(int64_t)blockIdx.x * S + s] = tot;
  }
}

__global__ void emit_kernel(int N, int S, const int32_t* __restrict__ grp, const int32_t* __restrict__ lp,
                            const int32_t* __restrict__ blkcnt, int32_t* idx, DeviceStatus* st) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= N) return;
  const int q = N / S, r = N % S;
  const int g = grp[i];
  if (g < 0 || g >= S) {
    report(st, -5, SITE_PART_IDX, i);
    return;
  }
  int pos = lp[i];
  const int blk = i / kPosBlock;
  for (int u = 0; u < blk; ++u) pos += blkcnt[(int64_t)u * S + g];
  const int at = g * q + min(g, r) + pos;
  const int end = (g + 1) * q + min(g + 1, r);
  if (at < 0 || at >= end) {
    report(st, -5, SITE_PART_IDX, i);
    return;
  }
  idx[at] = i;
}

// ---- independent uniform assignment -----------------------------------------------------------
// group_i = floor(key_i * S / 2^64) with the same keys; group sizes are Binomial(N, 1/S).  The
// position of a neuron inside its group is found exactly as above (blocks of 1024 neurons in
// index order); the group offsets come from the block counts instead of a formula.
__global__ void __launch_bounds__(kPosBlock) iid_group_kernel(uint64_t layer_seed, int N, int S, int32_t* grp,
                                                               int32_t* lp, int32_t* blkcnt) {
  extern __shared__ int32_t wcnt[];          // [32 warps][S]
  const int i = blockIdx.x * kPosBlock + threadIdx.x;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  for (int e = threadIdx.x; e < 32 * S; e += kPosBlock) wcnt[e] = 0;
  __syncthreads();
  int g = -1;
  if (i < N) {
    const uint64_t k = splitmix64_mix(layer_seed + 0x9E3779B97F4A7C15ull * (uint64_t)(i + 1));
    g = (int)__umul64hi(k, (uint64_t)S);
    grp[i] = g;
  }
  const unsigned same = __match_any_sync(0xffffffffu, g);
  const int wpos = __popc(same & ((1u << lane) - 1u));
  if (g >= 0 && wpos == 0) wcnt[w * S + g] = __popc(same);
  __syncthreads();
  if (i < N) {
    int before = 0;
    for (int u = 0; u < w; ++u) before += wcnt[u * S + g];
    lp[i] = before + wpos;
  }
  for (int s = threadIdx.x; s < S; s += kPosBlock) {
    int tot = 0;
    for (int u = 0; u < 32; ++u) tot += wcnt[u * S + s];
    blkcnt[(int64_t)blockIdx.x * S + s] = tot;
  }
}

// One CTA: off[g] = number of neurons in groups below g.
__global__ void iid_offsets_kernel(int S, int n_blocks, const int32_t* __restrict__ blkcnt, int32_t* off) {
  extern __shared__ int32_t tot[];           // [S]
  for (int s = threadIdx.x; s < S; s += blockDim.x) {
    int t = 0;
    for (int u = 0; u < n_blocks; ++u) t += blkcnt[(int64_t)u * S + s];
    tot[s] = t;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int at = 0;
    for (int s = 0; s < S; ++s) {
      off[s] = at;
      at += tot[s];
    }
    off[S] = at;
  }
}

__global__ void iid_emit_kernel(int N, int S, const int32_t* __restrict__ grp, const int32_t* __restrict__ lp,
                                const int32_t* __restrict__ blkcnt, const int32_t* __restrict__ off, int32_t* idx,
                                DeviceStatus* st) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= N) return;
  const int g = grp[i];
  if (g < 0 || g >= S) {
    report(st, -5, SITE_PART_IDX, i);
    return;
  }
  int pos = lp[i];
  const int blk = i / kPosBlock;
  for (int u = 0; u < blk; ++u) pos += blkcnt[(int64_t)u * S + g];
  const int at = off[g] + pos;
  if (at < off[g] || at >= off[g + 1]) {
    report(st, -5, SITE_PART_IDX, i);
    return;
  }
  idx[at] = i;
}

}  // namespace

bool partition_layer_iid(const Launch& L, uint64_t layer_seed, int N, int S, const PartitionScratch& sc, int32_t* idx,
                         int32_t* off, DeviceStatus* st) {
  const int smem = 32 * S * (int)sizeof(int32_t);
  if (smem > 96 * 1024) return false;
  static bool configured = false;
  if (!configured) {
    if (cudaFuncSetAttribute(iid_group_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024) != cudaSuccess)
      return false;
    configured = true;
  }
  const int n_blocks = (int)ceil_div(N, kPosBlock);
  iid_group_kernel<<<n_blocks, kPosBlock, smem, L.stream>>>(layer_seed, N, S, sc.grp, sc.lp, sc.blkcnt);
  iid_offsets_kernel<<<1, 256, S * sizeof(int32_t), L.stream>>>(S, n_blocks, sc.blkcnt, off);
  iid_emit_kernel<<<(unsigned)ceil_div(N, kThreads), kThreads, 0, L.stream>>>(N, S, sc.grp, sc.lp, sc.blkcnt, off, idx, st);
  L.count(3);
  return true;
}

// Host copy of the same rule: group sizes only (the host needs them to size copies and to refuse
// a draw that does not fit the packed layout).
void partition_iid_counts_host(uint64_t layer_seed, int N, int S, int64_t* counts) {
  for (int s = 0; s < S; ++s) counts[s] = 0;
  for (int i = 0; i < N; ++i) {
    uint64_t z = layer_seed + 0x9E3779B97F4A7C15ull * (uint64_t)(i + 1);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    z ^= z >> 31;
    counts[(int)(((unsigned __int128)z * (unsigned __int128)(uint64_t)S) >> 64)]++;
  }
}

size_t partition_scratch_bytes(int N, int S) {
  PartitionScratch s{};
  return partition_scratch_carve(nullptr, N, S, &s);
}

// Lays the scratch arrays out in `base` (may be null to just measure).  Returns bytes used.
size_t partition_scratch_carve(void* base, int N, int S, PartitionScratch* out) {
  size_t at = 0;
  auto take = [&](size_t bytes) {
    void* p = base ? (char*)base + at : nullptr;
    at += (size_t)round_up((int64_t)bytes, 256);
    return p;
  };
  int nb = 1, lb = 0;
  while (nb * 8 < N && lb < 24) { nb <<= 1; ++lb; }
  out->log_buckets = lb;
  out->n_buckets = nb;
  out->keys = (uint64_t*)take((size_t)N * 8);
  out->skey = (uint64_t*)take((size_t)N * 8);
  out->sidx = (int32_t*)take((size_t)N * 4);
  out->hist = (int32_t*)take((size_t)nb * 4);
  out->start = (int32_t*)take((size_t)(nb + 1) * 4);
  out->cursor = (int32_t*)take((size_t)nb * 4);
  out->grp = (int32_t*)take((size_t)N * 4);
  out->lp = (int32_t*)take((size_t)N * 4);
  out->blkcnt = (int32_t*)take((size_t)ceil_div(N, kPosBlock) * S * 4);
  return at;
}

bool partition_layer(const Launch& L, uint64_t layer_seed, int N, int S, const PartitionScratch& sc,
                     int32_t* idx, int32_t* off, DeviceStatus* st) {
  const int smem = 32 * S * (int)sizeof(int32_t);
  if (smem > 96 * 1024) return false;
  static bool configured = false;
  if (!configured) {
    if (cudaFuncSetAttribute(rank_group_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024) !=
        cudaSuccess)
      return false;
    configured = true;
  }
  const int nb = (int)ceil_div(N, kThreads);
  clear_kernel<<<(unsigned)ceil_div(sc.n_buckets, kThreads), kThreads, 0, L.stream>>>(sc.hist, sc.n_buckets);
  keys_kernel<<<nb, kThreads, 0, L.stream>>>(layer_seed, N, sc.log_buckets, sc.keys, sc.hist);
  bucket_scan_kernel<<<1, 1024, 0, L.stream>>>(sc.hist, sc.n_buckets, sc.start, sc.cursor);
  place_kernel<<<nb, kThreads, 0, L.stream>>>(N, sc.log_buckets, sc.keys, sc.start, sc.cursor, sc.skey, sc.sidx);
  rank_group_kernel<<<(unsigned)ceil_div(N, kPosBlock), kPosBlock, smem, L.stream>>>(
      N, S, sc.log_buckets, sc.keys, sc.start, sc.skey, sc.sidx, sc.grp, sc.lp, sc.blkcnt, off);
  emit_kernel<<<nb, kThreads, 0, L.stream>>>(N, S, sc.grp, sc.lp, sc.blkcnt, idx, st);
  L.count(6);
  return true;
}

}  // namespace ist
