// Small host-side entry points of libdai8: status strings, defaults, device check, counters.
#include "dai8_common.cuh"

namespace dai8 {

std::atomic<uint64_t> g_launch_count{0};

dai8_status check_device_arch() {
  static std::atomic<int> cached[64];  // 0 = unknown, 1 = ok, 2 = wrong architecture
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return DAI8_ERR_CUDA;
  if (dev >= 0 && dev < 64) {
    const int c = cached[dev].load(std::memory_order_relaxed);
    if (c == 1) return DAI8_OK;
    if (c == 2) return DAI8_ERR_ARCH;
  }
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return DAI8_ERR_CUDA;
  const bool ok = major == 10;
  if (dev >= 0 && dev < 64) cached[dev].store(ok ? 1 : 2, std::memory_order_relaxed);
  return ok ? DAI8_OK : DAI8_ERR_ARCH;
}

}  // namespace dai8

extern "C" const char* dai8_status_string(dai8_status s) {
  switch (s) {
    case DAI8_OK: return "ok";
    case DAI8_ERR_INVALID_ARG: return "invalid argument";
    case DAI8_ERR_UNSUPPORTED: return "unsupported geometry or option";
    case DAI8_ERR_WORKSPACE: return "workspace too small";
    case DAI8_ERR_ARCH: return "device is not compute capability 10.x";
    case DAI8_ERR_CUDA: return "CUDA call failed";
    case DAI8_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

extern "C" void dai8_mcs_defaults(dai8_mcs_params* p) {
  if (!p) return;
  p->lambda = 0.3f;  // Eq. 15
  p->k = 1.0f;       // Sec. 4.1
  p->A = 0.8f;       // Sec. 4.1
  p->std_unbiased = 0;
  p->center_mean = 1;
  p->mode = DAI8_GRAD_FULL;
}

extern "C" int dai8_padded_channels(int C) { return C > 0 ? dai8::round_up(C, 16) : 0; }

extern "C" uint64_t dai8_launch_count(void) {
  return dai8::g_launch_count.load(std::memory_order_relaxed);
}

extern "C" dai8_status dai8_get_device_status(int* host_status, void* stream) {
  if (!host_status) return DAI8_ERR_INVALID_ARG;
  return dai8::read_clear_device_status(host_status, static_cast<cudaStream_t>(stream));
}

extern "C" const char* dai8_debug_last_kernel(void) { return dai8::last_kernel_slot(); }

extern "C" dai8_status dai8_debug_expire_waits(uint64_t limit_cycles, int* report, void* ws, size_t ws_bytes,
                                               void* stream) {
  if (!report || !ws || ws_bytes < 32 || !dai8::aligned16(ws)) return DAI8_ERR_INVALID_ARG;
  if (limit_cycles == 0 || limit_cycles > 100000000ull) return DAI8_ERR_INVALID_ARG;   // at most ~50 ms
  dai8_status a = dai8::check_device_arch();
  if (a != DAI8_OK) return a;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int* rep = reinterpret_cast<int*>(static_cast<char*>(ws) + 16);
  if (cudaMemsetAsync(rep, 0, 12, st) != cudaSuccess) return DAI8_ERR_CUDA;
  a = dai8::expire_gvq_waits((long long)limit_cycles, ws, rep, st);
  if (a == DAI8_OK) a = dai8::expire_conv_wait((long long)limit_cycles, rep, st);
  if (a != DAI8_OK) return a;
  if (cudaMemcpyAsync(report, rep, 12, cudaMemcpyDeviceToHost, st) != cudaSuccess) return DAI8_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return DAI8_ERR_CUDA;
  return DAI8_OK;
}
