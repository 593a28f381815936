// Shared host/device helpers of libdai8 (CUDA side only; the CPU oracle shares nothing with this).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>

#include "../../include/dai8.h"

namespace dai8 {

// bfloat16 values travel as their 16-bit patterns; widening to binary32 is exact.
struct bf16_t {
  uint16_t bits;
};

extern std::atomic<uint64_t> g_launch_count;
inline void note_launch(int n = 1) { g_launch_count.fetch_add((uint64_t)n, std::memory_order_relaxed); }

// Reads and clears the device status word kept beside the tensor-core kernels (conv_umma.cu).
dai8_status read_clear_device_status(int* host_status, cudaStream_t stream);
// Device address of that status word on the current device (nullptr on failure).
unsigned int* device_status_address();

// Self-tests of the bounded device-side waits (gvq.cu, conv_umma.cu): each runs the file's own wait
// helpers on barriers nobody completes, with `limit` cycles; report_dev[0..2] get 1 where the wait
// gave up as it must.  ws: 16 bytes of scratch.
dai8_status expire_gvq_waits(long long limit, void* ws, int* report_dev, cudaStream_t st);
dai8_status expire_conv_wait(long long limit, int* report_dev, cudaStream_t st);

// Programmatic dependent launch.  A kernel launched with launch_dependent() may start while the
// kernel before it on the stream is still running: its CTAs take the SM resources that become free
// and run their set-up (barrier initialisation, tensor-memory allocation, descriptor prefetch), then
// stop in grid_dependency_wait() until the earlier kernel has completed and its writes are visible.
// Nothing that reads or writes global memory may come before that wait.  grid_dependency_release()
// lets the NEXT kernel on the stream begin launching; it says nothing about memory.  Both are no-ops
// in a kernel launched the ordinary way.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// DAI8_LOG=1 in the environment: one line on stderr per call, naming the kernel chosen and its tiling.
inline bool log_enabled() {
  static const bool on = [] { const char* e = std::getenv("DAI8_LOG"); return e && e[0] && e[0] != '0'; }();
  return on;
}
inline void log_choice(const char* fmt, ...) {
  if (!log_enabled()) return;
  va_list ap;
  va_start(ap, fmt);
  std::fputs("[dai8] ", stderr);
  std::vfprintf(stderr, fmt, ap);
  std::fputc('\n', stderr);
  va_end(ap);
}

// The kernel (family) the calling thread's last entry-point call ran on: what dai8_debug_last_kernel
// reports, so that a timing harness can attribute device time to kernels by name.
inline const char*& last_kernel_slot() {
  static thread_local const char* name = "";
  return name;
}
inline void note_kernel(const char* name) { last_kernel_slot() = name; }

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int round_up(int x, int m) { return (x + m - 1) / m * m; }
inline int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }

#define DAI8_RETURN_IF_CUDA(expr)                 \
  do {                                            \
    cudaError_t e__ = (expr);                     \
    if (e__ != cudaSuccess) return DAI8_ERR_CUDA; \
  } while (0)

// DAI8_OK if the current device is compute capability 10.x, else DAI8_ERR_ARCH / DAI8_ERR_CUDA.
dai8_status check_device_arch();

// Multiprocessors of the current device (looked up once per device).
inline int sm_count() {
  static std::atomic<int> cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  int sms = cached[dev].load(std::memory_order_relaxed);
  if (sms == 0) {
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return 148;
    cached[dev].store(sms, std::memory_order_relaxed);
  }
  return sms;
}

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per device for one kernel: `slot` is a
// per-kernel array of 64 flags.
template <typename K>
inline cudaError_t set_max_smem_once(std::atomic<int>* slot, K kernel, int bytes) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (slot[dev].load(std::memory_order_acquire) == 1) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) slot[dev].store(1, std::memory_order_release);
  return e;
}


__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(bf16_t v) { return __uint_as_float((uint32_t)v.bits << 16); }

// Loads VE consecutive elements (VE*sizeof(T) is 16 bytes, or VE == 1) and widens them to fp32.
template <typename T, int VE>
__device__ __forceinline__ void load_vec(const T* p, float (&v)[VE]);

template <>
__device__ __forceinline__ void load_vec<float, 4>(const float* p, float (&v)[4]) {
  const float4 t = *reinterpret_cast<const float4*>(p);
  v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
template <>
__device__ __forceinline__ void load_vec<float, 1>(const float* p, float (&v)[1]) { v[0] = *p; }
template <>
__device__ __forceinline__ void load_vec<bf16_t, 8>(const bf16_t* p, float (&v)[8]) {
  const uint4 t = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}
template <>
__device__ __forceinline__ void load_vec<bf16_t, 1>(const bf16_t* p, float (&v)[1]) {
  v[0] = to_f32(*p);
}

// ------------------------------------------------------------------------------------------------
// Counter-based uniform numbers for stochastic rounding (the paper names the rounding mode in
// Sec. 3 but no generator).  key = avalanche32(seed xor 0x9E3779B9 * (high half of the element's NCHW
// index + 1)), once per 2^32 elements; x = low half * 0x9E3779B1 + key; f = high half xor low half of
// the 64-bit product x * 0x85EBCA6B; stream 0 uses f * 0xC2B2AE35, stream 1 f * 0x2C1B3C6D;
// u = (top 23 bits) * 2^-23.  Per element that is four multiplies and ONE instruction of the
// half-rate integer/logic pipe, which is what bounds the code sweep.
// ------------------------------------------------------------------------------------------------
__host__ __device__ __forceinline__ uint32_t avalanche32(uint32_t h) {
  h ^= h >> 16;
  h *= 0x85EBCA6Bu;
  h ^= h >> 13;
  h *= 0xC2B2AE35u;
  h ^= h >> 16;
  return h;
}
__host__ __device__ __forceinline__ uint32_t sr_key(uint32_t seed, uint32_t index_hi) {
  return avalanche32(seed ^ (0x9E3779B9u * (index_hi + 1u)));
}
__device__ __forceinline__ float sr_uniform(uint32_t h) {
  return __uint_as_float(0x3F800000u | (h >> 9)) - 1.0f;  // exact: (h >> 9) * 2^-23
}

// Eq. 1 on one element, given inv = 127/s (0 when s <= 0).  The operation order (multiply, clamp,
// then round) and the absence of fused multiply-add are part of the definition: codes must be
// reproducible bit for bit.
__device__ __forceinline__ int quant_nearest(float x, float inv) {
  float v = __fmul_rn(x, inv);
  v = fminf(fmaxf(v, -127.0f), 127.0f);
  return __float2int_rn(v);
}
__device__ __forceinline__ int quant_stochastic(float x, float inv, float u) {
  float v = __fmul_rn(x, inv);
  v = fminf(fmaxf(v, -127.0f), 127.0f);
  const int q = __float2int_rd(__fadd_rn(v, u));
  return min(q, 127);
}

// The same two quantizers without a float-to-int conversion: adding 1.5*2^23 to a value in
// [-127, 127] leaves its rounded integer in the low mantissa bits (two's complement), so the LOW
// BYTE of the returned bit pattern is the int8 code.  Round-to-nearest-even of the sum is Eq. 1's
// nearest rounding; round-down of the sum is the floor of stochastic rounding.  For the stochastic
// form the upper clamp moves behind the addition of u: floor(min(v + u, 127)) equals
// min(floor(min(v, 127) + u), 127) for every v and every u in [0, 1).
constexpr float kRoundMagic = 12582912.0f;  // 1.5 * 2^23
__device__ __forceinline__ uint32_t quant_nearest_bits(float x, float inv) {
  float v = __fmul_rn(x, inv);
  v = fminf(fmaxf(v, -127.0f), 127.0f);
  return __float_as_uint(__fadd_rn(v, kRoundMagic));
}
__device__ __forceinline__ uint32_t quant_stochastic_bits(float x, float inv, float u) {
  const float v = fmaxf(__fmul_rn(x, inv), -127.0f);
  const float t = fminf(__fadd_rn(v, u), 127.0f);
  return __float_as_uint(__fadd_rd(t, kRoundMagic));
}
// Low bytes of four such bit patterns -> one word of four consecutive int8 codes.
__device__ __forceinline__ uint32_t pack_codes4(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  return __byte_perm(__byte_perm(a, b, 0x0040), __byte_perm(c, d, 0x0040), 0x5410);
}
// u in [0,1) from a hash: one funnel shift builds the bits of 1.0 + (h >> 9) * 2^-23.
__device__ __forceinline__ float sr_uniform_fast(uint32_t h) {
  return __uint_as_float(__funnelshift_r(h, 0x7Fu, 9)) - 1.0f;
}
// The folded multiply f of an element (see above); sr_bits0 / sr_bits1 turn it into the two streams' bits.
__device__ __forceinline__ uint32_t sr_fold(uint32_t index_lo, uint32_t key) {
  const uint32_t x = index_lo * 0x9E3779B1u + key;
  const uint64_t p = (uint64_t)x * 0x85EBCA6Bull;
  return (uint32_t)(p >> 32) ^ (uint32_t)p;
}
__device__ __forceinline__ uint32_t sr_bits0(uint32_t f) { return f * 0xC2B2AE35u; }
__device__ __forceinline__ uint32_t sr_bits1(uint32_t f) { return f * 0x2C1B3C6Du; }
__device__ __forceinline__ float inv_scale(float s) { return s > 0.0f ? __fdiv_rn(127.0f, s) : 0.0f; }

}  // namespace dai8
