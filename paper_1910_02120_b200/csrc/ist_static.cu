// ist_partition_layer_static: the partition of one hidden layer, drawn with scratch memory that
// is part of the library image instead of a caller-provided workspace.
//
// Who this is for: code that is not allowed to obtain device memory when it needs a partition.
// Typical cases are a plugin running inside a host application that hands out its whole
// device-memory budget at start-up and forbids cudaMalloc afterwards, or a service whose arena is
// already carved up and which only wants the index lists (to plan which weight slices to
// fetch or ship) without creating a full ist_ctx and its workspace.  Such a caller passes only
// its own output buffers; everything the kernels need in between lives in `g_scratch` below.
//
// Cost: every GPU that loads this library holds kStaticScratchBytes (2 MB) of device
// memory for that array until the process exits, whether or not this entry point is ever used.
#include "../../include/ist.h"

#include <mutex>

#include "kernels.h"

using namespace ist;

namespace {

constexpr int kMaxDevices = 64;

// Largest scratch any allowed call can need: partition_scratch_bytes(IST_STATIC_MAX_NEURONS,
// IST_STATIC_MAX_SUBNETS) plus one status word; checked again at run time before every launch.
constexpr size_t kStaticScratchBytes = 2048 * 1024;

// File-scope device array.  In host code this name is only a handle for the symbol, not a
// device address: the address each device gives it is looked up with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_scratch[kStaticScratchBytes];

std::mutex g_mutex;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of g_scratch on the current device (looked up once per device), or null if no
// call has looked it up yet.
void* scratch_address_if_known() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lk(g_mutex);
  return g_scratch_addr[dev];
}

ist_status scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return IST_ERR_CUDA;
  std::lock_guard<std::mutex> lk(g_mutex);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_scratch) != cudaSuccess || !p) return IST_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return IST_OK;
}

uint64_t splitmix64_next(uint64_t* state) {
  uint64_t z = (*state += 0x9E3779B97F4A7C15ull);
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

}  // namespace

extern "C" ist_status ist_partition_layer_static(uint64_t seed, int hidden_layer, int64_t n_neurons, int S,
                                                 int32_t* idx_out_dev, int32_t* off_out_dev,
                                                 void* cuda_stream) {
  if (!idx_out_dev || !off_out_dev) return IST_ERR_ARG;
  if (hidden_layer < 1 || hidden_layer > 62) return IST_ERR_ARG;
  if (n_neurons < 1 || S < 1 || S > n_neurons) return IST_ERR_ARG;
  if (n_neurons > IST_STATIC_MAX_NEURONS || S > IST_STATIC_MAX_SUBNETS) return IST_ERR_UNSUPPORTED;
  const int N = (int)n_neurons;
  const size_t status_bytes = 256;
  if (status_bytes + partition_scratch_bytes(N, S) > kStaticScratchBytes) return IST_ERR_UNSUPPORTED;

  void* base = nullptr;
  ist_status s = scratch_address(&base);   // first call on a device: symbol look-up
  if (s != IST_OK) return s;

  cudaStream_t stream = (cudaStream_t)cuda_stream;
  // The array still holds whatever the previous call left: the status word is cleared here, the
  // bucket histogram and cursors are cleared by the partition kernels themselves; every other
  // scratch array is fully overwritten before it is read.
  if (cudaMemsetAsync(base, 0, status_bytes, stream) != cudaSuccess) return IST_ERR_CUDA;
  PartitionScratch sc{};
  partition_scratch_carve((char*)base + status_bytes, N, S, &sc);

  uint64_t state = seed, layer_seed = 0;
  for (int l = 1; l <= hidden_layer; ++l) layer_seed = splitmix64_next(&state);

  Launch L{stream, nullptr};
  if (!partition_layer(L, layer_seed, N, S, sc, idx_out_dev, off_out_dev, reinterpret_cast<DeviceStatus*>(base)))
    return IST_ERR_UNSUPPORTED;
  return cudaGetLastError() == cudaSuccess ? IST_OK : IST_ERR_CUDA;
}


extern "C" ist_status ist_static_partition_status(void* cuda_stream) {
  void* base = scratch_address_if_known();
  if (!base) return IST_OK;   // the entry point has not run on this device: nothing to report
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  DeviceStatus h{};
  if (cudaMemcpyAsync(&h, base, sizeof h, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return IST_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return IST_ERR_CUDA;
  return h.code == 0 ? IST_OK : (ist_status)h.code;
}
