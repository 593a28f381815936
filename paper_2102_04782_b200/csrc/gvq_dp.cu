// Batch-sharded gradient quantization: the stages of Algorithm 1 as separate calls, for data-parallel
// training in which every rank holds some of the images of dY.  Per-channel statistics (Algorithm 1,
// first step), the density count (Eq. 15) and hence the classes and clip values (Eq. 11 / 14) are
// properties of the WHOLE batch, so the ranks exchange per-channel scalars between the stages:
//
//   dai8_dp_grad_pivot     the channel values of the shard's first pixel (exchange: broadcast from rank 0)
//   dai8_dp_grad_moments   local |g|max, sum (g - pivot), sum (g - pivot)^2 per channel, pivot common
//        exchange:         maximum of |g|max, sum of the two sums
//   dai8_dp_grad_sigma     mean, sigma, layer |g|max of the whole batch (every rank, identical)
//   dai8_dp_grad_count     local #{|g| > sigma_c}
//        exchange:         sum of the counts
//   dai8_dp_grad_solve     class and clip value per channel (every rank, identical)
//   dai8_dp_grad_codes     both code tensors of the rank's own images; the generator's counter is the
//                          element's index in the whole batch (first_image), so the codes are the ones
//                          dai8_quantize_grad writes for these images on the unsharded tensor
//
// plus two helpers of the sharded layer step: dai8_absmax (layer scale of X before its exchange) and
// dai8_dequant_filter (Eq. 7 after the int32 weight-gradient partials of the ranks have been added).
// NHWC only.  Correctness first: plain grid-stride kernels with per-block partials combined in a
// fixed order; they are not tuned like the one-launch kernel of the unsharded path.
#include "dai8_common.cuh"

namespace dai8 {
namespace {

constexpr int kDpThreads = 256;
constexpr int kDpMaxBlocks = 296;       // pixel blocks: two per SM

struct DpGrid {
  int cols, rows_per_iter, pixel_blocks, col_blocks;
};
DpGrid dp_grid(int64_t npix, int C) {
  DpGrid g;
  g.cols = C < kDpThreads ? C : kDpThreads;
  g.rows_per_iter = kDpThreads / g.cols;
  g.col_blocks = (C + g.cols - 1) / g.cols;
  int64_t pb = (npix + (int64_t)g.rows_per_iter * 8 - 1) / ((int64_t)g.rows_per_iter * 8);
  if (pb > kDpMaxBlocks) pb = kDpMaxBlocks;
  if (pb < 1) pb = 1;
  g.pixel_blocks = (int)pb;
  return g;
}

// workspace: [pixel_blocks][C] x (float max, double s1, double s2), or uint32 counts in the same place
size_t dp_ws_bytes(int C) { return (size_t)kDpMaxBlocks * C * (8 + 8 + 4) + 64; }

struct DpPartials {
  double* s1;
  double* s2;
  float* mx;
};
DpPartials dp_carve(void* ws, int C) {
  DpPartials p;
  p.s1 = static_cast<double*>(ws);
  p.s2 = p.s1 + (size_t)kDpMaxBlocks * C;
  p.mx = reinterpret_cast<float*>(p.s2 + (size_t)kDpMaxBlocks * C);
  return p;
}

// Partial moments of this block's pixels, per channel.  Thread (r, c) walks rows r, r + rows_per_iter, ...
template <typename T>
__global__ void __launch_bounds__(kDpThreads)
dp_moments_kernel(const T* __restrict__ x, int64_t npix, int C, int cols, int rows_per_iter,
                  const float* __restrict__ pivot, DpPartials out) {
  __shared__ double sh1[kDpThreads], sh2[kDpThreads];
  __shared__ float shm[kDpThreads];
  const int tid = threadIdx.x;
  const int r = tid / cols, c = blockIdx.y * cols + (tid - r * cols);
  const bool live = r < rows_per_iter && c < C;
  const int64_t chunk = (npix + gridDim.x - 1) / gridDim.x;
  const int64_t p0 = (int64_t)blockIdx.x * chunk, p1 = p0 + chunk < npix ? p0 + chunk : npix;
  float m = 0.f, f1 = 0.f, f2 = 0.f;
  double d1 = 0.0, d2 = 0.0;
  if (live) {
    const float piv = pivot[c];
    int run = 0;
    for (int64_t p = p0 + r; p < p1; p += rows_per_iter) {
      const float v = to_f32(x[p * C + c]);
      m = fmaxf(m, fabsf(v));
      const float d = __fsub_rn(v, piv);
      f1 = __fadd_rn(f1, d);
      f2 = __fmaf_rn(d, d, f2);
      if (++run == 32) { run = 0; d1 += (double)f1; d2 += (double)f2; f1 = 0.f; f2 = 0.f; }   // short fp32 runs, combined in binary64
    }
    d1 += (double)f1; d2 += (double)f2;
  }
  sh1[tid] = d1; sh2[tid] = d2; shm[tid] = m;
  __syncthreads();
  if (r == 0 && c < C) {          // fixed order over the rows of the block
    for (int k = 1; k < rows_per_iter; ++k) {
      const int o = tid + k * cols;
      d1 += sh1[o]; d2 += sh2[o]; m = fmaxf(m, shm[o]);
    }
    const size_t o = (size_t)blockIdx.x * C + c;
    out.s1[o] = d1; out.s2[o] = d2; out.mx[o] = m;
  }
}

// Sums the blocks' partials in block order.  sums: [2][C].
__global__ void __launch_bounds__(kDpThreads)
dp_moments_reduce_kernel(DpPartials in, int blocks, int C, float* __restrict__ absmax, double* __restrict__ sums) {
  const int c = blockIdx.x * kDpThreads + threadIdx.x;
  if (c >= C) return;
  double d1 = 0.0, d2 = 0.0;
  float m = 0.f;
  for (int b = 0; b < blocks; ++b) {
    const size_t o = (size_t)b * C + c;
    d1 += in.s1[o]; d2 += in.s2[o]; m = fmaxf(m, in.mx[o]);
  }
  absmax[c] = m; sums[c] = d1; sums[C + c] = d2;
}

// Whole-batch mean and sigma from the exchanged moments of d = g - pivot (binary64), and the layer |g|max.
__global__ void __launch_bounds__(kDpThreads)
dp_sigma_kernel(const float* __restrict__ absmax, const double* __restrict__ sums, const float* __restrict__ pivot,
                int C, double M, int std_unbiased, int center_mean, float* __restrict__ mean,
                float* __restrict__ sigma, unsigned int* __restrict__ gmax_bits) {
  const int c = blockIdx.x * kDpThreads + threadIdx.x;
  if (c >= C) return;
  const double s1 = sums[c], s2 = sums[C + c], piv = (double)pivot[c];
  const double md = s1 / M;
  double var = center_mean ? (s2 - s1 * md) : (s2 + 2.0 * piv * s1 + M * piv * piv);
  if (var < 0.0) var = 0.0;
  const double denom = std_unbiased ? M - 1.0 : M;
  mean[c] = (float)(piv + md);
  sigma[c] = denom > 0.0 ? (float)sqrt(var / denom) : 0.0f;
  const float mx = absmax[c];
  if (mx > 0.f) atomicMax(gmax_bits, __float_as_uint(mx));     // non-negative floats order like their bits
}

// Local density count #{|g| > sigma_c} (binary32 compare, strict), per-block partials in block order.
template <typename T>
__global__ void __launch_bounds__(kDpThreads)
dp_count_kernel(const T* __restrict__ x, int64_t npix, int C, int cols, int rows_per_iter,
                const float* __restrict__ sigma, unsigned int* __restrict__ partial) {
  __shared__ unsigned int shc[kDpThreads];
  const int tid = threadIdx.x;
  const int r = tid / cols, c = blockIdx.y * cols + (tid - r * cols);
  const bool live = r < rows_per_iter && c < C;
  const int64_t chunk = (npix + gridDim.x - 1) / gridDim.x;
  const int64_t p0 = (int64_t)blockIdx.x * chunk, p1 = p0 + chunk < npix ? p0 + chunk : npix;
  unsigned int n = 0u;
  if (live) {
    const float sg = sigma[c];
    for (int64_t p = p0 + r; p < p1; p += rows_per_iter) n += fabsf(to_f32(x[p * C + c])) > sg ? 1u : 0u;
  }
  shc[tid] = n;
  __syncthreads();
  if (r == 0 && c < C) {
    for (int k = 1; k < rows_per_iter; ++k) n += shc[tid + k * cols];
    partial[(size_t)blockIdx.x * C + c] = n;
  }
}
__global__ void __launch_bounds__(kDpThreads)
dp_count_reduce_kernel(const unsigned int* __restrict__ partial, int blocks, int C, long long* __restrict__ cnt) {
  const int c = blockIdx.x * kDpThreads + threadIdx.x;
  if (c >= C) return;
  long long n = 0;
  for (int b = 0; b < blocks; ++b) n += (long long)partial[(size_t)b * C + c];
  cnt[c] = n;
}

// Discriminator (Eq. 15) and clip value (Eq. 11: |g|max for a bell-shaped channel; Eq. 14 otherwise),
// from the whole batch's count and |g|max.  The state is written in both branches.
__global__ void __launch_bounds__(kDpThreads)
dp_solve_kernel(const long long* __restrict__ cnt, const float* __restrict__ absmax, int C, double M, float lambda,
                float k, float A, float* __restrict__ s_state, int has_prev, uint8_t* __restrict__ cls) {
  const int c = blockIdx.x * kDpThreads + threadIdx.x;
  if (c >= C) return;
  const float gmax = absmax[c];
  const bool bell = (double)cnt[c] > (double)lambda * M;
  float s = gmax;
  if (!bell) {
    const float t = __fsub_rn(1.0f, __fmul_rn(k, A));
    s = __fadd_rn(__fmul_rn(t, has_prev ? s_state[c] : gmax), __fmul_rn(A, gmax));
  }
  s_state[c] = s;
  if (cls) cls[c] = bell ? 1 : 0;
}

// Both code tensors of the rank's images.  One thread = four consecutive channels of one pixel (one
// 32-bit word of each code tensor).  The generator's counter is the element's NCHW index in the WHOLE
// batch: image n of this rank is image first_image + n there.
template <typename T>
__global__ void __launch_bounds__(kDpThreads)
dp_codes_kernel(const T* __restrict__ x, int64_t npix, int64_t HW, int C, int Cp, int64_t first_image,
                const float* __restrict__ s, const float* __restrict__ gmax_layer, uint32_t seed,
                int8_t* __restrict__ vq, int8_t* __restrict__ gq) {
  const int cw = Cp >> 2;
  const int64_t words = npix * cw;
  const float inv2 = inv_scale(*gmax_layer);
  const uint32_t key0 = sr_key(seed, 0u);
  for (int64_t o = (int64_t)blockIdx.x * kDpThreads + threadIdx.x; o < words; o += (int64_t)gridDim.x * kDpThreads) {
    const int64_t pix = o / cw;
    const int c0 = (int)(o - pix * cw) << 2;
    const int64_t n = pix / HW, hw = pix - n * HW;
    uint32_t a[4], b[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = c0 + j;
      a[j] = 0u; b[j] = 0u;
      if (c < C) {
        const float v = to_f32(x[pix * C + c]);
        const uint64_t idx = ((uint64_t)(first_image + n) * (uint64_t)C + (uint64_t)c) * (uint64_t)HW + (uint64_t)hw;
        const uint32_t hi = (uint32_t)(idx >> 32);
        const uint32_t key = hi == 0u ? key0 : sr_key(seed, hi);
        const uint32_t f = sr_fold((uint32_t)idx, key);
        a[j] = quant_stochastic_bits(v, inv_scale(s[c]), sr_uniform(sr_bits0(f)));
        if (gq) b[j] = quant_stochastic_bits(v, inv2, sr_uniform(sr_bits1(f)));
      }
    }
    reinterpret_cast<uint32_t*>(vq)[o] = pack_codes4(a[0], a[1], a[2], a[3]);
    if (gq) reinterpret_cast<uint32_t*>(gq)[o] = pack_codes4(b[0], b[1], b[2], b[3]);
  }
}

template <typename T>
__global__ void __launch_bounds__(kDpThreads)
dp_absmax_kernel(const T* __restrict__ x, int64_t count, unsigned int* __restrict__ out_bits) {
  float m = 0.f;
  for (int64_t i = (int64_t)blockIdx.x * kDpThreads + threadIdx.x; i < count; i += (int64_t)gridDim.x * kDpThreads)
    m = fmaxf(m, fabsf(to_f32(x[i])));
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  if ((threadIdx.x & 31) == 0 && m > 0.f) atomicMax(out_bits, __float_as_uint(m));
}

// Eq. 7 for the weight gradient: dW = acc * (sX / 127) * (s_co / 127), each step rounded in binary32.
__global__ void __launch_bounds__(kDpThreads)
dp_dequant_filter_kernel(const int* __restrict__ acc, const float* __restrict__ sX, const float* __restrict__ s,
                         int64_t total, int64_t per_cout, float* __restrict__ dW) {
  const float ax = __fdiv_rn(*sX, 127.0f);
  for (int64_t i = (int64_t)blockIdx.x * kDpThreads + threadIdx.x; i < total; i += (int64_t)gridDim.x * kDpThreads) {
    const float scale = __fmul_rn(ax, __fdiv_rn(s[i / per_cout], 127.0f));
    dW[i] = __fmul_rn(__int2float_rn(acc[i]), scale);
  }
}

template <typename T>
__global__ void __launch_bounds__(kDpThreads)
dp_pivot_kernel(const T* __restrict__ x, int C, float* __restrict__ pivot) {
  const int c = blockIdx.x * kDpThreads + threadIdx.x;
  if (c < C) pivot[c] = to_f32(x[c]);     // pixel 0 of the shard
}

bool dp_bad_shape(int N, int C, int H, int W) { return N <= 0 || C <= 0 || H <= 0 || W <= 0; }
int dp_blocks_1d(int64_t n) {
  int64_t b = (n + kDpThreads - 1) / kDpThreads;
  const int64_t cap = (int64_t)sm_count() * 8;
  return (int)(b < 1 ? 1 : (b > cap ? cap : b));
}

}  // namespace
}  // namespace dai8

using namespace dai8;

extern "C" size_t dai8_dp_grad_workspace_bytes(int C) { return C > 0 ? dp_ws_bytes(C) : 0; }

extern "C" dai8_status dai8_dp_grad_moments(const void* dY, dai8_dtype dtype, dai8_layout layout, int N_local,
                                            int C, int H, int W, const float* pivot, float* absmax,
                                            double* sums, void* ws, size_t ws_bytes, void* stream) {
  if (!dY || !pivot || !absmax || !sums || !ws) return DAI8_ERR_INVALID_ARG;
  if (dp_bad_shape(N_local, C, H, W)) return DAI8_ERR_INVALID_ARG;
  if (dtype != DAI8_F32 && dtype != DAI8_BF16) return DAI8_ERR_INVALID_ARG;
  if (layout != DAI8_NHWC) return DAI8_ERR_UNSUPPORTED;
  if (!aligned16(ws)) return DAI8_ERR_INVALID_ARG;
  if (ws_bytes < dp_ws_bytes(C)) return DAI8_ERR_WORKSPACE;
  dai8_status a = check_device_arch();
  if (a != DAI8_OK) return a;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t npix = (int64_t)N_local * H * W;
  const DpGrid g = dp_grid(npix, C);
  const DpPartials p = dp_carve(ws, C);
  const dim3 grid((unsigned)g.pixel_blocks, (unsigned)g.col_blocks);
  if (dtype == DAI8_F32)
    dp_moments_kernel<float><<<grid, kDpThreads, 0, st>>>(static_cast<const float*>(dY), npix, C, g.cols, g.rows_per_iter, pivot, p);
  else
    dp_moments_kernel<bf16_t><<<grid, kDpThreads, 0, st>>>(static_cast<const bf16_t*>(dY), npix, C, g.cols, g.rows_per_iter, pivot, p);
  dp_moments_reduce_kernel<<<(C + kDpThreads - 1) / kDpThreads, kDpThreads, 0, st>>>(p, g.pixel_blocks, C, absmax, sums);
  note_launch(2);
  note_kernel("dp_moments_kernel");
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}

extern "C" dai8_status dai8_dp_grad_pivot(const void* dY, dai8_dtype dtype, dai8_layout layout, int C, float* pivot,
                                          void* stream) {
  if (!dY || !pivot || C <= 0) return DAI8_ERR_INVALID_ARG;
  if (dtype != DAI8_F32 && dtype != DAI8_BF16) return DAI8_ERR_INVALID_ARG;
  if (layout != DAI8_NHWC) return DAI8_ERR_UNSUPPORTED;
  dai8_status a = check_device_arch();
  if (a != DAI8_OK) return a;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int blocks = (C + kDpThreads - 1) / kDpThreads;
  if (dtype == DAI8_F32) dp_pivot_kernel<float><<<blocks, kDpThreads, 0, st>>>(static_cast<const float*>(dY), C, pivot);
  else dp_pivot_kernel<bf16_t><<<blocks, kDpThreads, 0, st>>>(static_cast<const bf16_t*>(dY), C, pivot);
  note_launch(1);
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}

extern "C" dai8_status dai8_dp_grad_sigma(const float* absmax, const double* sums, const float* pivot, int C,
                                          int64_t M_global, const dai8_mcs_params* params, float* mean,
                                          float* sigma, float* gmax_layer, void* stream) {
  if (!absmax || !sums || !pivot || !mean || !sigma || !gmax_layer || C <= 0 || M_global <= 0) return DAI8_ERR_INVALID_ARG;
  dai8_status a = check_device_arch();
  if (a != DAI8_OK) return a;
  dai8_mcs_params p;
  if (params) p = *params; else dai8_mcs_defaults(&p);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  DAI8_RETURN_IF_CUDA(cudaMemsetAsync(gmax_layer, 0, sizeof(float), st));
  dp_sigma_kernel<<<(C + kDpThreads - 1) / kDpThreads, kDpThreads, 0, st>>>(
      absmax, sums, pivot, C, (double)M_global, p.std_unbiased, p.center_mean, mean, sigma,
      reinterpret_cast<unsigned int*>(gmax_layer));
  note_launch(1);
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}

extern "C" dai8_status dai8_dp_grad_count(const void* dY, dai8_dtype dtype, dai8_layout layout, int N_local, int C,
                                          int H, int W, const float* sigma, long long* cnt, void* ws,
                                          size_t ws_bytes, void* stream) {
  if (!dY || !sigma || !cnt || !ws) return DAI8_ERR_INVALID_ARG;
  if (dp_bad_shape(N_local, C, H, W)) return DAI8_ERR_INVALID_ARG;
  if (dtype != DAI8_F32 && dtype != DAI8_BF16) return DAI8_ERR_INVALID_ARG;
  if (layout != DAI8_NHWC) return DAI8_ERR_UNSUPPORTED;
  if (!aligned16(ws)) return DAI8_ERR_INVALID_ARG;
  if (ws_bytes < dp_ws_bytes(C)) return DAI8_ERR_WORKSPACE;
  const int64_t npix = (int64_t)N_local * H * W;
  if (npix >= (int64_t)1 << 32) return DAI8_ERR_UNSUPPORTED;       // per-block counts are 32-bit
  dai8_status a = check_device_arch();
  if (a != DAI8_OK) return a;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const DpGrid g = dp_grid(npix, C);
  unsigned int* partial = static_cast<unsigned int*>(ws);
  const dim3 grid((unsigned)g.pixel_blocks, (unsigned)g.col_blocks);
  if (dtype == DAI8_F32)
    dp_count_kernel<float><<<grid, kDpThreads, 0, st>>>(static_cast<const float*>(dY), npix, C, g.cols, g.rows_per_iter, sigma, partial);
  else
    dp_count_kernel<bf16_t><<<grid, kDpThreads, 0, st>>>(static_cast<const bf16_t*>(dY), npix, C, g.cols, g.rows_per_iter, sigma, partial);
  dp_count_reduce_kernel<<<(C + kDpThreads - 1) / kDpThreads, kDpThreads, 0, st>>>(partial, g.pixel_blocks, C, cnt);
  note_launch(2);
  note_kernel("dp_count_kernel");
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}

extern "C" dai8_status dai8_dp_grad_solve(const long long* cnt, const float* absmax, int C, int64_t M_global,
                                          const dai8_mcs_params* params, float* s_state, int has_prev,
                                          uint8_t* cls, void* stream) {
  if (!cnt || !absmax || !s_state || C <= 0 || M_global <= 0) return DAI8_ERR_INVALID_ARG;
  dai8_mcs_params p;
  if (params) p = *params; else dai8_mcs_defaults(&p);
  if (p.mode != DAI8_GRAD_FULL) return DAI8_ERR_UNSUPPORTED;
  dai8_status a = check_device_arch();
  if (a != DAI8_OK) return a;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  dp_solve_kernel<<<(C + kDpThreads - 1) / kDpThreads, kDpThreads, 0, st>>>(cnt, absmax, C, (double)M_global, p.lambda, p.k,
                                                                           p.A, s_state, has_prev, cls);
  note_launch(1);
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}

extern "C" dai8_status dai8_dp_grad_codes(const void* dY, dai8_dtype dtype, dai8_layout layout, int N_local, int C,
                                          int H, int W, int64_t first_image, const float* s,
                                          const float* gmax_layer, uint32_t seed, int8_t* vq, int8_t* gq,
                                          void* stream) {
  if (!dY || !s || !gmax_layer || !vq || first_image < 0) return DAI8_ERR_INVALID_ARG;
  if (dp_bad_shape(N_local, C, H, W)) return DAI8_ERR_INVALID_ARG;
  if (dtype != DAI8_F32 && dtype != DAI8_BF16) return DAI8_ERR_INVALID_ARG;
  if (layout != DAI8_NHWC) return DAI8_ERR_UNSUPPORTED;
  if (!aligned16(vq) || (gq && !aligned16(gq))) return DAI8_ERR_INVALID_ARG;
  dai8_status a = check_device_arch();
  if (a != DAI8_OK) return a;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t HW = (int64_t)H * W, npix = (int64_t)N_local * HW;
  const int Cp = round_up(C, 16);
  const int blocks = dp_blocks_1d(npix * (Cp / 4));
  if (dtype == DAI8_F32)
    dp_codes_kernel<float><<<blocks, kDpThreads, 0, st>>>(static_cast<const float*>(dY), npix, HW, C, Cp, first_image, s, gmax_layer, seed, vq, gq);
  else
    dp_codes_kernel<bf16_t><<<blocks, kDpThreads, 0, st>>>(static_cast<const bf16_t*>(dY), npix, HW, C, Cp, first_image, s, gmax_layer, seed, vq, gq);
  note_launch(1);
  note_kernel("dp_codes_kernel");
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}

extern "C" dai8_status dai8_absmax(const void* x, dai8_dtype dtype, int64_t count, float* out, void* stream) {
  if (!x || !out || count <= 0) return DAI8_ERR_INVALID_ARG;
  if (dtype != DAI8_F32 && dtype != DAI8_BF16) return DAI8_ERR_INVALID_ARG;
  dai8_status a = check_device_arch();
  if (a != DAI8_OK) return a;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  DAI8_RETURN_IF_CUDA(cudaMemsetAsync(out, 0, sizeof(float), st));
  const int blocks = dp_blocks_1d(count);
  if (dtype == DAI8_F32)
    dp_absmax_kernel<float><<<blocks, kDpThreads, 0, st>>>(static_cast<const float*>(x), count, reinterpret_cast<unsigned int*>(out));
  else
    dp_absmax_kernel<bf16_t><<<blocks, kDpThreads, 0, st>>>(static_cast<const bf16_t*>(x), count, reinterpret_cast<unsigned int*>(out));
  note_launch(1);
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}

extern "C" dai8_status dai8_dequant_filter(const int32_t* acc, const float* sX, const float* s, int Cout,
                                           int64_t per_cout, float* dW, void* stream) {
  if (!acc || !sX || !s || !dW || Cout <= 0 || per_cout <= 0) return DAI8_ERR_INVALID_ARG;
  dai8_status a = check_device_arch();
  if (a != DAI8_OK) return a;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t total = (int64_t)Cout * per_cout;
  dp_dequant_filter_kernel<<<dp_blocks_1d(total), kDpThreads, 0, st>>>(acc, sX, s, total, per_cout, dW);
  note_launch(1);
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}
