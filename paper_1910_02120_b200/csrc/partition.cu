// Random balanced partition of a hidden layer's neurons into S groups (paper Sec. 2.1
// "Constructing Subnets"; App. A: sum_s m^(s)_{l,i} = 1).  Integer work only.
//
// key_i   = (i+1)-th output of SplitMix64 seeded with the layer's stream seed
// rank_i  = #{ j : (key_j, j) < (key_i, i) }
// group_i = the group whose rank interval contains rank_i (sizes floor(N/S), +1 for the
//           first N mod S groups)
// pos_i   = #{ j < i : group_j = group_i }      (ascending order inside a group)
// idx[off[group_i] + pos_i] = i
//
// rank and pos are counted by brute force over (i, j) pairs, spread over a 2-D grid with
// integer atomics, so the result does not depend on scheduling.
#include "kernels.h"

namespace ist {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ uint64_t splitmix64_mix(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

__global__ void keys_kernel(uint64_t layer_seed, int N, uint64_t* keys, int32_t* rank, int32_t* pos) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < N) {
    keys[i] = splitmix64_mix(layer_seed + 0x9E3779B97F4A7C15ull * (uint64_t)(i + 1));
    rank[i] = 0;
    pos[i] = 0;
  }
}

// blockIdx.x: block of 256 neurons i; blockIdx.y: chunk of the j range.
__global__ void rank_kernel(int N, int jchunk, const uint64_t* __restrict__ keys, int32_t* rank) {
  __shared__ uint64_t tile[kThreads];
  int i = blockIdx.x * kThreads + threadIdx.x;
  uint64_t ki = i < N ? keys[i] : 0;
  int j0 = blockIdx.y * jchunk;
  int j1 = min(N, j0 + jchunk);
  int cnt = 0;
  for (int jb = j0; jb < j1; jb += kThreads) {
    int j = jb + threadIdx.x;
    tile[threadIdx.x] = j < j1 ? keys[j] : ~0ull;
    __syncthreads();
    int lim = min(kThreads, j1 - jb);
    for (int u = 0; u < lim; ++u) {
      uint64_t kj = tile[u];
      cnt += (kj < ki) || (kj == ki && (jb + u) < i);
    }
    __syncthreads();
  }
  if (i < N && cnt) atomicAdd(&rank[i], cnt);
}

__global__ void group_kernel(int N, int S, const int32_t* __restrict__ rank, int32_t* grp,
                             int32_t* off) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  int q = N / S, r = N % S;
  if (i < N) {
    int rk = rank[i];
    int big = r * (q + 1);
    grp[i] = rk < big ? rk / (q + 1) : r + (rk - big) / q;
  }
  if (i <= S) off[i] = i * q + min(i, r);
}

__global__ void pos_kernel(int N, int jchunk, const int32_t* __restrict__ grp, int32_t* pos) {
  __shared__ int32_t tile[kThreads];
  int i = blockIdx.x * kThreads + threadIdx.x;
  int gi = i < N ? grp[i] : -1;
  int j0 = blockIdx.y * jchunk;
  int j1 = min(N, j0 + jchunk);
  j1 = min(j1, (int)(blockIdx.x + 1) * kThreads);  // only j < i can count
  int cnt = 0;
  for (int jb = j0; jb < j1; jb += kThreads) {
    int j = jb + threadIdx.x;
    tile[threadIdx.x] = j < j1 ? grp[j] : -2;
    __syncthreads();
    int lim = min(kThreads, j1 - jb);
    for (int u = 0; u < lim; ++u) cnt += (tile[u] == gi) && (jb + u) < i;
    __syncthreads();
  }
  if (i < N && cnt) atomicAdd(&pos[i], cnt);
}

__global__ void emit_kernel(int N, int S, const int32_t* __restrict__ grp,
                            const int32_t* __restrict__ pos, int32_t* idx, DeviceStatus* st) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= N) return;
  int q = N / S, r = N % S;
  int g = grp[i];
  int at = g * q + min(g, r) + pos[i];
  int end = (g + 1) * q + min(g + 1, r);
  if (g < 0 || g >= S || at < 0 || at >= end) {
    report(st, -5, SITE_PART_IDX, i);
    return;
  }
  idx[at] = i;
}

}  // namespace

void partition_layer(const Launch& L, uint64_t layer_seed, int N, int S, uint64_t* keys,
                     int32_t* rank, int32_t* grp, int32_t* pos, int32_t* idx, int32_t* off,
                     DeviceStatus* st) {
  int nb = (int)ceil_div(N, kThreads);
  int nb_s = (int)ceil_div(max(N, S + 1), kThreads);
  // spread the j range so that the pair count fills the machine: about 4 CTAs per SM
  int want = 148 * 4;
  int ychunks = max(1, min((int)ceil_div(N, kThreads), want / max(nb, 1)));
  int jchunk = (int)round_up(ceil_div(N, ychunks), kThreads);
  ychunks = (int)ceil_div(N, jchunk);
  keys_kernel<<<nb, kThreads, 0, L.stream>>>(layer_seed, N, keys, rank, pos);
  rank_kernel<<<dim3(nb, ychunks), kThreads, 0, L.stream>>>(N, jchunk, keys, rank);
  group_kernel<<<nb_s, kThreads, 0, L.stream>>>(N, S, rank, grp, off);
  pos_kernel<<<dim3(nb, ychunks), kThreads, 0, L.stream>>>(N, jchunk, grp, pos);
  emit_kernel<<<nb, kThreads, 0, L.stream>>>(N, S, grp, pos, idx, st);
  L.count(5);
}

}  // namespace ist
