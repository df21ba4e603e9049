// pbt_energy_fitness_static: the energy-distance scorer with its scratch memory built
// into the library image instead of taken from a caller-provided workspace.
//
// Who needs this: an embedding application that has handed the whole device to its own
// arena and forbids plug-ins to call cudaMalloc, or a scoring loop that must not pay for
// (or synchronise on) a driver allocation just to get a few kilobytes of partial sums.
// Such a caller has device buffers for its samples and for the result, but nowhere to put
// the per-block partial sums the reduction needs.  Here those live in a fixed array that
// every GPU loading this library keeps until the process exits.
//
// Consequences the caller has to know:
//   * the array has a fixed size (kScratchDoubles doubles = 1 MiB): larger problems are refused;
//   * all calls share it, and it keeps whatever the previous call left there.  Nothing in
//     it has to start at zero: every slot that the final pass reads is overwritten first by
//     the partial pass of the same call;
//   * two calls whose kernels overlap on the GPU (different streams, or different host
//     threads) would write the same slots and race.  Issue calls on one stream, or order them;
//   * the first call on each device looks up the array's device address; make that first
//     call outside any stream capture.
#include <stdio.h>

#include <mutex>

#include "pbt_common.cuh"

namespace pbt {
void set_last_error(const char* msg);
}

namespace {

constexpr int kScratchDoubles = 131072;  // 1 MiB
constexpr int kMaxDevices = 64;

// In host code this name is only a handle for the runtime, not a device pointer: its device
// address must be asked for with cudaGetSymbolAddress, once per device.
static __device__ __align__(256) double g_energy_scratch[kScratchDoubles];

std::mutex g_mu;
double* g_scratch_addr[kMaxDevices] = {nullptr};

int scratch_for_current_device(double** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) {
    pbt::set_last_error(cudaGetErrorString(e));
    return PBT_ERR_CUDA;
  }
  if (dev < 0 || dev >= kMaxDevices) {
    pbt::set_last_error("device ordinal beyond the supported range of the static scratch table");
    return PBT_ERR_UNSUPPORTED;
  }
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_energy_scratch);
    if (e != cudaSuccess || !p) {
      pbt::set_last_error(e != cudaSuccess ? cudaGetErrorString(e) : "cudaGetSymbolAddress returned NULL");
      return PBT_ERR_CUDA;
    }
    g_scratch_addr[dev] = static_cast<double*>(p);
  }
  *out = g_scratch_addr[dev];
  return PBT_OK;
}

}  // namespace

extern "C" int pbt_energy_fitness_static(const float* x_device, int n, int n_members, float* fitness_out_device,
                                         void* stream) {
  if (!x_device || !fitness_out_device) {
    pbt::set_last_error("x_device and fitness_out_device must not be NULL");
    return PBT_ERR_INVALID_ARG;
  }
  if (n < 1 || n_members < 1) {
    pbt::set_last_error("n and n_members must be positive");
    return PBT_ERR_INVALID_ARG;
  }
  // sizes are checked in 64-bit arithmetic before anything derived from them is used: 2 * ceil(n / 256) partial sums
  // per member (the layout of launch_energy_distance), at most 65535 members (the grid's second dimension)
  const long long need = (long long)n_members * (2ll * (((long long)n + 255) / 256));
  if (need > kScratchDoubles || n_members > 65535) {
    char msg[256];
    snprintf(msg, sizeof(msg),
             "problem too large for the built-in scratch: n_members * 2 * ceil(n / 256) = %lld doubles, limit %d "
             "(use pbt_eval with a caller-provided workspace instead)", need, kScratchDoubles);
    pbt::set_last_error(msg);
    return PBT_ERR_WORKSPACE;
  }
  // The scratch address that is looked up belongs to the CURRENT device, and the kernels run there: both buffers
  // must live on it too (a buffer of another GPU would be dereferenced as peer memory).
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    pbt::set_last_error("no current CUDA device");
    return PBT_ERR_CUDA;
  }
  const void* bufs[2] = {x_device, fitness_out_device};
  for (const void* b : bufs) {
    cudaPointerAttributes attr;
    const cudaError_t pe = cudaPointerGetAttributes(&attr, b);
    if (pe != cudaSuccess || (attr.type != cudaMemoryTypeDevice && attr.type != cudaMemoryTypeManaged) ||
        (attr.type == cudaMemoryTypeDevice && attr.device != dev)) {
      if (pe != cudaSuccess) cudaGetLastError();
      pbt::set_last_error("x_device and fitness_out_device must be device memory of the current device");
      return PBT_ERR_INVALID_ARG;
    }
  }
  double* scratch = nullptr;
  int rc = scratch_for_current_device(&scratch);
  if (rc != PBT_OK) return rc;
  cudaError_t e = pbt::launch_energy_distance(x_device, (long long)n * 2, n, n_members, scratch, fitness_out_device,
                                              (cudaStream_t)stream);
  if (e != cudaSuccess) {
    pbt::set_last_error(cudaGetErrorString(e));
    return PBT_ERR_CUDA;
  }
  return PBT_OK;
}
