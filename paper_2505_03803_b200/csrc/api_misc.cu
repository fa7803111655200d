// Device status word and CUDA error text.
#include <cuda_runtime.h>
#include <string.h>

#include <atomic>

#include "../../include/rwkvq.h"
#include "host_util.h"

namespace rwkvq {
__device__ int g_device_status = 0;
static thread_local char t_last_error[256] = "";
static std::atomic<unsigned> g_abort_epoch{0};
unsigned abort_epoch() { return g_abort_epoch.load(); }
void set_last_cuda_error(cudaError_t e) {
  strncpy(t_last_error, cudaGetErrorString(e), sizeof(t_last_error) - 1);
  t_last_error[sizeof(t_last_error) - 1] = 0;
}
// Device address of the status word for the current device (kernels in other translation units
// receive it as an argument).
int* device_status_ptr() {
  void* p = nullptr;
  if (cudaGetSymbolAddress(&p, g_device_status) != cudaSuccess) return nullptr;
  return static_cast<int*>(p);
}
}  // namespace rwkvq

extern "C" {
const char* rwkvq_last_cuda_error(void) { return rwkvq::t_last_error; }

rwkvq_status rwkvq_device_status(void* stream) {
  int v = 0, zero = 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemcpyFromSymbolAsync(&v, rwkvq::g_device_status, sizeof(int), 0, cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaMemcpyToSymbolAsync(rwkvq::g_device_status, &zero, sizeof(int), 0, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return rwkvq::cuda_status(e);
  if (v != 0) rwkvq::g_abort_epoch.fetch_add(1);
  return v == 0 ? RWKVQ_OK : (rwkvq_status)v;
}
}
