// PTX wrappers shared by the tensor-core convolution kernels: mbarriers with bounded waits, TMA loads
// and stores, tcgen05 allocation / MMA / commit / load, shared-memory matrix descriptors.
#pragma once

#include <cuda.h>

#include <mutex>
#include <string>
#include <unordered_map>

#include "conv_internal.cuh"

namespace dai8 {
namespace umma {

constexpr int kBM = 128;                            // MMA M: rows of an accumulator tile
constexpr long long kTimeoutCycles = 2000000000LL;  // about one second

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false if the CTA is aborting (this wait or another one expired).
// `status`: the device status word that receives DAI8_ERR_TIMEOUT.
// `limit`: cycles after which the wait gives up (the default everywhere but in the self-test of this path).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          unsigned int* status, long long limit = kTimeoutCycles) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > limit) {
      *abort_flag = 1u;
      atomicExch(status, (unsigned int)DAI8_ERR_TIMEOUT);
      return false;
    }
  }
}

// True in exactly one lane of a converged warp.  The single-thread roles (copy-engine issue, MMA
// issue) are written as loops that the WHOLE warp runs with warp-uniform control flow and values, in
// which only the elected lane executes the issuing instructions: tcgen05.mma, tcgen05.commit and the
// bulk-tensor copies take their operands from uniform registers, and only in uniform code can the
// compiler compute addresses and descriptors there.  Under `if (lane == 0)` every operand of every
// issue is moved from a vector register first, which costs far more than the instruction itself
// (measured: 154 cycles per tcgen05.mma whatever its shape, against 128 / 74 / 55 cycles for N = 256 /
// 128 / <= 64 from a uniform loop).
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xFFFFFFFF;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
  return pred != 0;
}

__device__ __forceinline__ void tma_load_im2col_4d(const CUtensorMap* map, uint64_t* bar, void* dst, int c,
                                                   int w, int h, int n, uint16_t off_w, uint16_t off_h) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c), "r"(w), "r"(h),
        "r"(n), "h"(off_w), "h"(off_h)
      : "memory");
}
__device__ __forceinline__ void tma_load_tile_3d(const CUtensorMap* map, uint64_t* bar, void* dst, int c0,
                                                 int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
// Shared -> global tile store (2D), tracked by the issuing thread's bulk async-group.
__device__ __forceinline__ void tma_store_tile_2d(const CUtensorMap* map, const void* src, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(src)), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

// Variants for the single-thread issue loops: shared-memory addresses are passed as 32-bit values
// computed once, so that no generic-to-shared conversion or 64-bit arithmetic sits between two
// issues (these loops are latency chains of one thread).
__device__ __forceinline__ void mbar_expect_tx_a(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tma_load_im2col_4d_a(uint64_t map, uint32_t bar, uint32_t dst, int c, int w, int h,
                                                     int n, uint16_t off_w, uint16_t off_h) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h)
      : "memory");
}
__device__ __forceinline__ void tma_load_tile_3d_a(uint64_t map, uint32_t bar, uint32_t dst, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tc_commit_a(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// The 64-bit matrix descriptor of a K-major tile is a constant high word and a low word that holds
// the 16-byte-granular address: stepping through chunks and K slices is a 32-bit addition.
__device__ __forceinline__ uint32_t kmajor_desc_hi(int kc_bytes) {
  const uint32_t layout = kc_bytes == 128 ? 2u : (kc_bytes == 64 ? 4u : 6u);
  const uint32_t sbo = (uint32_t)(8 * kc_bytes) >> 4;
  return sbo | (1u << 14) | (layout << 29);
}
__device__ __forceinline__ uint32_t kmajor_desc_lo(uint32_t saddr) { return ((saddr & 0x3FFFFu) >> 4) | (1u << 16); }
__device__ __forceinline__ void mma_i8_parts(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc,
                                             uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The same with separate high words for A and B (B in another layout than A).
__device__ __forceinline__ void mma_i8_parts2(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi,
                                              uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "mov.b64 da, {%1, %2};\n\t"
      "mov.b64 db, {%3, %4};\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], da, db, %5, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)),
               "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
// D[tmem] (+)= A[smem] * B[smem], int8 x int8 -> int32, one instruction covers K = 32.
__device__ __forceinline__ void mma_i8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
      : "memory");
}
// 32 lanes x 16 consecutive 32-bit columns: thread i of the warp gets lane (base lane + i).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, int (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr) : "memory");
}
// 32 lanes x 32 consecutive 32-bit columns.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, int (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor for a K-major operand tile [rows][kc_bytes] written by TMA with
// the matching swizzle (rows of 32/64/128 bytes; groups of 8 rows are `8*kc_bytes` apart).
__device__ __forceinline__ uint64_t kmajor_desc(uint32_t saddr, int kc_bytes) {
  const uint64_t layout = kc_bytes == 128 ? 2ull : (kc_bytes == 64 ? 4ull : 6ull);
  const uint64_t sbo = (uint64_t)(8 * kc_bytes) >> 4;
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | (sbo << 32) | (1ull << 46) | (layout << 61);
}
// Instruction descriptor: int32 accumulator, signed 8-bit A and B, both K-major, M = 128, N = bn.
__device__ __forceinline__ uint32_t idesc_i8_kmajor(int bn) {
  return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
}


// ---------------------------------------------------------------------------------------------
// Host side: tensor-map encoders of the driver (looked up once per process), device properties
// ---------------------------------------------------------------------------------------------
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
using EncodeIm2colFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const int*, const int*, cuuint32_t, cuuint32_t,
                                    const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
struct DriverApi {
  EncodeTiledFn tiled = nullptr;
  EncodeIm2colFn im2col = nullptr;
  bool ok() const { return tiled && im2col; }
};
inline const DriverApi& driver_api() {
  static const DriverApi api = [] {
    DriverApi a;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      a.tiled = reinterpret_cast<EncodeTiledFn>(fn);
    fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      a.im2col = reinterpret_cast<EncodeIm2colFn>(fn);
    return a;
  }();
  return api;
}

// Tensor maps are a function of the call's arguments only (pointer, extents, box), and a training
// loop repeats the same layer calls every step: encoded maps are kept in a small table keyed by the
// encoder's arguments, so that a repeated call encodes nothing.
struct MapCache {
  std::mutex mu;
  std::unordered_map<std::string, CUtensorMap> table;
  CUresult get(const std::string& key, CUtensorMap* out, CUresult (*encode)(CUtensorMap*, const void*), const void* args) {
    {
      std::lock_guard<std::mutex> lock(mu);
      auto it = table.find(key);
      if (it != table.end()) { *out = it->second; return CUDA_SUCCESS; }
    }
    const CUresult r = encode(out, args);
    if (r == CUDA_SUCCESS) {
      std::lock_guard<std::mutex> lock(mu);
      if (table.size() >= 4096) table.clear();
      table.emplace(key, *out);
    }
    return r;
  }
};
inline MapCache& map_cache() { static MapCache c; return c; }

template <typename T>
inline void key_add(std::string& k, const T* p, size_t n) { k.append(reinterpret_cast<const char*>(p), n * sizeof(T)); }

struct TiledArgs {
  CUtensorMapDataType dt; cuuint32_t rank; void* ptr; const cuuint64_t* dims; const cuuint64_t* strides;
  const cuuint32_t* box; const cuuint32_t* estr; CUtensorMapSwizzle sw; CUtensorMapL2promotion l2;
};
inline CUresult encode_tiled_cached(CUtensorMap* out, CUtensorMapDataType dt, cuuint32_t rank, void* ptr,
                                    const cuuint64_t* dims, const cuuint64_t* strides, const cuuint32_t* box,
                                    const cuuint32_t* estr, CUtensorMapSwizzle sw, CUtensorMapL2promotion l2) {
  int dev = 0;
  cudaGetDevice(&dev);
  std::string key;
  key.reserve(160);
  const int tag[5] = {0, dev, (int)dt, (int)sw, (int)l2};
  key_add(key, tag, 5); key_add(key, &rank, 1); key_add(key, &ptr, 1);
  key_add(key, dims, rank); key_add(key, strides, rank - 1); key_add(key, box, rank); key_add(key, estr, rank);
  TiledArgs a{dt, rank, ptr, dims, strides, box, estr, sw, l2};
  return map_cache().get(key, out, [](CUtensorMap* m, const void* p) {
    const TiledArgs& t = *static_cast<const TiledArgs*>(p);
    return driver_api().tiled(m, t.dt, t.rank, t.ptr, t.dims, t.strides, t.box, t.estr, CU_TENSOR_MAP_INTERLEAVE_NONE, t.sw,
                              t.l2, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }, &a);
}
struct Im2colArgs {
  void* ptr; const cuuint64_t* dims; const cuuint64_t* strides; const int* lower; const int* upper;
  cuuint32_t channels, pixels; const cuuint32_t* estr; CUtensorMapSwizzle sw;
};
// 4-D uint8 im2col map (the only form the library uses).
inline CUresult encode_im2col_cached(CUtensorMap* out, void* ptr, const cuuint64_t* dims, const cuuint64_t* strides,
                                     const int* lower, const int* upper, cuuint32_t channels, cuuint32_t pixels,
                                     const cuuint32_t* estr, CUtensorMapSwizzle sw) {
  int dev = 0;
  cudaGetDevice(&dev);
  std::string key;
  key.reserve(160);
  const int tag[3] = {1, dev, (int)sw};
  key_add(key, tag, 3); key_add(key, &ptr, 1); key_add(key, dims, 4); key_add(key, strides, 3);
  key_add(key, lower, 2); key_add(key, upper, 2); key_add(key, &channels, 1); key_add(key, &pixels, 1); key_add(key, estr, 4);
  Im2colArgs a{ptr, dims, strides, lower, upper, channels, pixels, estr, sw};
  return map_cache().get(key, out, [](CUtensorMap* m, const void* p) {
    const Im2colArgs& t = *static_cast<const Im2colArgs*>(p);
    return driver_api().im2col(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, t.ptr, t.dims, t.strides, t.lower, t.upper, t.channels,
                               t.pixels, t.estr, CU_TENSOR_MAP_INTERLEAVE_NONE, t.sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }, &a);
}

inline CUtensorMapSwizzle swizzle_for(int kc_bytes) {
  return kc_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                         : (kc_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
}

}  // namespace umma
}  // namespace dai8
