// Gradient Vectorized Quantization with the Magnitude-aware Clipping Strategy (Algorithm 1 up to
// the two quantizations) and the layer-wide quantizer of the forward pass (Eq. 1), as HBM-bound kernels.
//
// Each step of Algorithm 1 needs a per-channel scalar the previous one produces: |g|max,c and sigma_c
// (statistics), then #{|g| > sigma_c} (density), then the class and the clip value s_c (Eq. 14/15), then
// the codes.  The kernels that run, by input:
//   * NHWC, C a multiple of the 16-byte vector (the layout of the benchmarks): ONE persistent
//     cooperative launch.  gvq_fused_nhwc_kernel partitions the pixels over the SMs, keeps as much of
//     a CTA's range as fits resident in shared memory (bulk asynchronous copies on an mbarrier ring)
//     and makes two sweeps: statistics, then density count fused with both code tensors, written with
//     the clip value of a PREDICTED class; channels whose count contradicts the prediction are redone.
//     gvq_columns_kernel serves many channels x few pixels: a CTA owns whole channel vectors, so
//     everything but the layer-wide |g|max is CTA-local.
//   * anything else (NCHW, ragged C, no cooperative launch): three launches -- stats_*, count_*,
//     quantize_* -- whose last block (ticket counter) finishes the per-channel scalars.
// Floating-point sums are combined in a fixed order (per-block partials, then a fixed tree), so results
// do not depend on scheduling; maxima and counts are order-independent.
// dai8_quantize_tensor: one launch for small tensors (every CTA finds the maximum itself) and for
// tensors that fit the GPU's shared memory (quantize_flat_fused_kernel); else max, then codes.
//
// Layouts.  The native layout is NHWC: a thread owns one 16-byte vector of channels
// (4 fp32 / 8 bf16) of one pixel and walks down the pixels, so per-channel scalars stay in
// registers and every load/store instruction of a warp covers contiguous memory.  NCHW inputs are
// read along H*W per (n, c) row and transposed through shared memory when codes are written.
#include <cmath>
#include <mutex>
#include <type_traits>

#include "dai8_common.cuh"

namespace dai8 {
namespace {

constexpr int kThreads = 256;
constexpr int kMaxPixelBlocks = 592;  // 4 blocks on each of 148 SMs

struct GvqWs {
  uint32_t* tickets;    // [C] arrival counters of the stats sweep (per column block / channel)
  uint32_t* ticket2;    // [1] arrival counter of the count sweep
  uint32_t* cnt;        // [C] density counts
  uint32_t* gmax_bits;  // [1] layer |g|max as the bit pattern of a non-negative float
  uint32_t* gridbar;    // [1] arrival counter of the fused kernel's grid barriers
  float* absmax;        // [C]
  float* mean;          // [C]
  float* sigma;         // [C]
  float* pmax;          // [PB][C] per-block partial max
  double* psum;         // [PB][C]
  double* pss;          // [PB][C]
  float* layer_scale;   // [1] the single clip value of the layer-wide modes
};

size_t control_words(int C) { return (size_t)2 * C + 4; }

size_t ws_bytes_for(int C) {
  size_t b = control_words(C) * 4;
  b = (b + 15) / 16 * 16;
  b += (size_t)3 * C * 4;
  b = (b + 15) / 16 * 16;
  b += (size_t)kMaxPixelBlocks * C * (4 + 8 + 8);
  return b + 64;
}

GvqWs carve(void* ws, int C) {
  GvqWs w;
  char* p = static_cast<char*>(ws);
  w.tickets = reinterpret_cast<uint32_t*>(p);
  w.ticket2 = w.tickets + C;
  w.cnt = w.ticket2 + 1;
  w.gmax_bits = w.cnt + C;
  w.gridbar = w.gmax_bits + 1;
  size_t off = (control_words(C) * 4 + 15) / 16 * 16;
  w.absmax = reinterpret_cast<float*>(p + off);
  w.mean = w.absmax + C;
  w.sigma = w.mean + C;
  off += (size_t)3 * C * 4;
  off = (off + 15) / 16 * 16;
  w.psum = reinterpret_cast<double*>(p + off);
  w.pss = w.psum + (size_t)kMaxPixelBlocks * C;
  w.pmax = reinterpret_cast<float*>(w.pss + (size_t)kMaxPixelBlocks * C);
  w.layer_scale = w.pmax + (size_t)kMaxPixelBlocks * C;     // inside the 64 bytes of slack at the end
  return w;
}

struct McsDev {
  float lambda, k, A;
  int std_unbiased, center_mean;
  int mode;   // dai8_grad_mode
};

// mean and sigma of one channel from the moments of d = g - pivot (binary64).  The pivot (the
// channel's first element) keeps sum d^2 - (sum d)^2/M free of cancellation when |mean| >> sigma.
__device__ __forceinline__ void finish_moments(double pivot, double s1, double s2, int64_t M,
                                               const McsDev& mp, float* mean, float* sigma) {
  const double md = s1 / (double)M;
  double var = mp.center_mean ? (s2 - s1 * md)                                  // sum (g-mu)^2
                              : (s2 + 2.0 * pivot * s1 + (double)M * pivot * pivot);  // sum g^2
  if (var < 0.0) var = 0.0;
  const double denom = mp.std_unbiased ? (double)(M - 1) : (double)M;
  *mean = (float)(pivot + md);
  *sigma = denom > 0.0 ? (float)sqrt(var / denom) : 0.0f;
}

// Returns true in every thread of the one block that arrives last at `ticket`.
__device__ __forceinline__ bool last_block_arrives(uint32_t* ticket, uint32_t expected) {
  __shared__ uint32_t s_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = (atomicAdd(ticket, 1u) == expected - 1u) ? 1u : 0u;
  __syncthreads();
  const bool last = s_last != 0u;
  if (last) __threadfence();
  return last;
}

// ------------------------------------------------------------------------------------------------
// Sweep 1, NHWC.  grid = (pixel blocks, column blocks of up to 256 vectors).
// ------------------------------------------------------------------------------------------------
template <typename T, int VE>
__global__ void __launch_bounds__(kThreads)
stats_nhwc_kernel(const T* __restrict__ x, int64_t npix, int C, int G, GvqWs ws, McsDev mp,
                  float* __restrict__ stats_out) {
  __shared__ double sred[kThreads * VE];
  const int tid = threadIdx.x;
  const int colv0 = blockIdx.y * kThreads;
  const int gcols = min(G - colv0, kThreads);
  const int rpi = kThreads / gcols;
  const int col = tid % gcols, rl = tid / gcols;
  const int64_t chunk = (npix + gridDim.x - 1) / gridDim.x;
  const int64_t p0 = (int64_t)blockIdx.x * chunk;
  const int64_t p1 = min(npix, p0 + chunk);

  float amax[VE], fs[VE], fss[VE];
  double ds[VE], dss[VE];
#pragma unroll
  for (int e = 0; e < VE; ++e) { amax[e] = 0.f; fs[e] = 0.f; fss[e] = 0.f; ds[e] = 0.0; dss[e] = 0.0; }

  if (rl < rpi) {
    const T* base = x + (int64_t)(colv0 + col) * VE;
    float piv[VE];
    load_vec<T, VE>(base, piv);  // pixel 0 of these channels
    int it = 0;
    for (int64_t p = p0 + rl; p < p1; p += rpi) {
      float v[VE];
      load_vec<T, VE>(base + p * C, v);
#pragma unroll
      for (int e = 0; e < VE; ++e) {
        amax[e] = fmaxf(amax[e], fabsf(v[e]));
        const float d = v[e] - piv[e];
        fs[e] += d;
        fss[e] = fmaf(d, d, fss[e]);
      }
      if (++it == 32) {  // short fp32 runs, combined in binary64
        it = 0;
#pragma unroll
        for (int e = 0; e < VE; ++e) { ds[e] += (double)fs[e]; dss[e] += (double)fss[e]; fs[e] = 0.f; fss[e] = 0.f; }
      }
    }
#pragma unroll
    for (int e = 0; e < VE; ++e) { ds[e] += (double)fs[e]; dss[e] += (double)fss[e]; }
  }

  const int nch = gcols * VE;             // channels of this column block
  const int c0 = colv0 * VE;
  const size_t prow = (size_t)blockIdx.x * C + c0;
  // three fixed-order reductions over the rpi row lanes
  for (int pass = 0; pass < 3; ++pass) {
    __syncthreads();
#pragma unroll
    for (int e = 0; e < VE; ++e)
      sred[tid * VE + e] = pass == 0 ? (double)amax[e] : (pass == 1 ? ds[e] : dss[e]);
    __syncthreads();
    for (int j = tid; j < nch; j += kThreads) {
      const int cc = j / VE, e = j % VE;
      double acc = 0.0;
      if (pass == 0) {
        for (int r = 0; r < rpi; ++r) acc = fmax(acc, sred[(r * gcols + cc) * VE + e]);
        ws.pmax[prow + j] = (float)acc;
      } else {
        for (int r = 0; r < rpi; ++r) acc += sred[(r * gcols + cc) * VE + e];
        (pass == 1 ? ws.psum : ws.pss)[prow + j] = acc;
      }
    }
  }

  if (!last_block_arrives(ws.tickets + blockIdx.y, gridDim.x)) return;

  // Last block of this column block: combine the per-block partials, channel by channel.
  const int PB = gridDim.x;
  const int nparts = nch >= kThreads ? 1 : kThreads / nch;
  const int64_t M = npix;
  float* smax = reinterpret_cast<float*>(sred);  // reuse: [kThreads] floats + 2*[kThreads] doubles
  __shared__ double ssum[kThreads], sss[kThreads];
  float block_max = 0.f;
  for (int cbase = 0; cbase < nch; cbase += kThreads) {
    const int j = (nparts == 1) ? cbase + tid : tid % nch;
    const int part = (nparts == 1) ? 0 : tid / nch;
    float m = 0.f;
    double s = 0.0, q = 0.0;
    if (j < nch && part < nparts) {
      for (int pb = part; pb < PB; pb += nparts) {
        const size_t idx = (size_t)pb * C + c0 + j;
        m = fmaxf(m, __ldcg(ws.pmax + idx));
        s += __ldcg(ws.psum + idx);
        q += __ldcg(ws.pss + idx);
      }
    }
    __syncthreads();
    smax[tid] = m; ssum[tid] = s; sss[tid] = q;
    __syncthreads();
    if (j < nch && part == 0) {
      for (int r = 1; r < nparts; ++r) {
        m = fmaxf(m, smax[r * nch + j]);
        s += ssum[r * nch + j];
        q += sss[r * nch + j];
      }
      float mean, sigma;
      const int c = c0 + j;
      finish_moments((double)to_f32(x[c]), s, q, M, mp, &mean, &sigma);
      ws.absmax[c] = m; ws.mean[c] = mean; ws.sigma[c] = sigma;
      if (stats_out) {
        stats_out[c * 4 + DAI8_STAT_ABSMAX] = m;
        stats_out[c * 4 + DAI8_STAT_MEAN] = mean;
        stats_out[c * 4 + DAI8_STAT_SIGMA] = sigma;
      }
      block_max = fmaxf(block_max, m);
    }
  }
  // layer |g|max: non-negative floats order like their bit patterns
  for (int o = 16; o > 0; o >>= 1) block_max = fmaxf(block_max, __shfl_xor_sync(0xFFFFFFFFu, block_max, o));
  if ((tid & 31) == 0 && block_max > 0.f) atomicMax(ws.gmax_bits, __float_as_uint(block_max));
}

// ------------------------------------------------------------------------------------------------
// Sweep 1, NCHW.  grid = (C, slices over n).  Each block reduces rows (n, c, :) of one channel.
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kThreads)
stats_nchw_kernel(const T* __restrict__ x, int N, int C, int64_t HW, GvqWs ws, McsDev mp,
                  float* __restrict__ stats_out) {
  const int c = blockIdx.x, tid = threadIdx.x;
  const int NS = gridDim.y;
  const int nper = (N + NS - 1) / NS;
  const int n0 = blockIdx.y * nper, n1 = min(N, n0 + nper);
  float amax = 0.f;
  double ds = 0.0, dss = 0.0;
  const float piv = to_f32(x[(int64_t)c * HW]);  // element (0, c, 0, 0)
  for (int n = n0; n < n1; ++n) {
    const T* row = x + ((int64_t)n * C + c) * HW;
    float fs = 0.f, fss = 0.f;
    int it = 0;
    for (int64_t i = tid; i < HW; i += kThreads) {
      const float v = to_f32(row[i]);
      amax = fmaxf(amax, fabsf(v));
      const float d = v - piv;
      fs += d;
      fss = fmaf(d, d, fss);
      if (++it == 32) { it = 0; ds += (double)fs; dss += (double)fss; fs = 0.f; fss = 0.f; }
    }
    ds += (double)fs; dss += (double)fss;
  }
  __shared__ float smax[kThreads];
  __shared__ double ssum[kThreads], sss[kThreads];
  smax[tid] = amax; ssum[tid] = ds; sss[tid] = dss;
  __syncthreads();
  for (int o = kThreads / 2; o > 0; o >>= 1) {  // fixed tree
    if (tid < o) {
      smax[tid] = fmaxf(smax[tid], smax[tid + o]);
      ssum[tid] += ssum[tid + o];
      sss[tid] += sss[tid + o];
    }
    __syncthreads();
  }
  if (tid == 0) {
    const size_t idx = (size_t)blockIdx.y * C + c;
    ws.pmax[idx] = smax[0]; ws.psum[idx] = ssum[0]; ws.pss[idx] = sss[0];
  }
  if (!last_block_arrives(ws.tickets + c, NS)) return;
  if (tid == 0) {
    float m = 0.f;
    double s = 0.0, q = 0.0;
    for (int pb = 0; pb < NS; ++pb) {
      const size_t idx = (size_t)pb * C + c;
      m = fmaxf(m, __ldcg(ws.pmax + idx));
      s += __ldcg(ws.psum + idx);
      q += __ldcg(ws.pss + idx);
    }
    float mean, sigma;
    finish_moments((double)piv, s, q, (int64_t)N * HW, mp, &mean, &sigma);
    ws.absmax[c] = m; ws.mean[c] = mean; ws.sigma[c] = sigma;
    if (stats_out) {
      stats_out[c * 4 + DAI8_STAT_ABSMAX] = m;
      stats_out[c * 4 + DAI8_STAT_MEAN] = mean;
      stats_out[c * 4 + DAI8_STAT_SIGMA] = sigma;
    }
    if (m > 0.f) atomicMax(ws.gmax_bits, __float_as_uint(m));
  }
}

// ------------------------------------------------------------------------------------------------
// Discriminator and clip update of Algorithm 1 for every channel, by the last block of the count sweep.
//   P > lambda (cnt > lambda*M in binary64): s = |g|max,c                       (Eq. 11)
//   otherwise: s = (1 - k*A)*s_prev + A*|g|max,c, each operation rounded to fp32  (Eq. 14)
// ------------------------------------------------------------------------------------------------
__device__ void solve_channels(const GvqWs& ws, int C, int64_t M, const McsDev& mp,
                               float* __restrict__ s_state, int has_prev,
                               float* __restrict__ gmax_layer, float* __restrict__ stats_out,
                               uint8_t* __restrict__ cls) {
  const float t = __fsub_rn(1.0f, __fmul_rn(mp.k, mp.A));
  const float gmax_l = __uint_as_float(__ldcg(ws.gmax_bits));
  if (mp.mode == DAI8_GRAD_GQ || mp.mode == DAI8_GRAD_LAYER_MCS) {
    // One scale for the whole layer (the ablation baselines of Sec. 4.1).  GQ: s = |g|max of the layer.
    // Layer-wise MCS: Eq. 15 and Eq. 14 on the statistics of the whole layer -- the count sweep ran with
    // the layer's sigma for every channel, so the layer's density is the sum of the channel counts.
    __shared__ unsigned long long s_total;
    __shared__ float s_layer;
    __shared__ int s_bell;
    if (threadIdx.x == 0) s_total = 0ull;
    __syncthreads();
    unsigned long long part = 0ull;
    for (int c = threadIdx.x; c < C; c += blockDim.x) part += (unsigned long long)__ldcg(ws.cnt + c);
    if (part) atomicAdd(&s_total, part);
    __syncthreads();
    if (threadIdx.x == 0) {
      float s = gmax_l;
      bool bell = true;                   // GQ: no clipping
      if (mp.mode == DAI8_GRAD_LAYER_MCS) {
        bell = (double)s_total > (double)mp.lambda * ((double)M * (double)C);
        if (!bell) s = __fadd_rn(__fmul_rn(t, has_prev ? s_state[0] : gmax_l), __fmul_rn(mp.A, gmax_l));
      }
      s_layer = s;
      s_bell = bell ? 1 : 0;
    }
    __syncthreads();
    const bool bell = s_bell != 0;
    const float s = s_layer;
    const double P_layer = (double)s_total / ((double)M * (double)C);
    for (int c = threadIdx.x; c < C; c += blockDim.x) {
      s_state[c] = s;
      if (cls) cls[c] = bell ? 1 : 0;
      if (stats_out)
        stats_out[c * 4 + DAI8_STAT_P] = mp.mode == DAI8_GRAD_LAYER_MCS ? (float)P_layer
                                                                         : (float)((double)__ldcg(ws.cnt + c) / (double)M);
    }
    if (threadIdx.x == 0) { *gmax_layer = gmax_l; *ws.layer_scale = s; }   // the layer scale, for the code kernels
    return;
  }
  for (int c = threadIdx.x; c < C; c += blockDim.x) {
    const uint32_t cnt = __ldcg(ws.cnt + c);
    const float gmax = __ldcg(ws.absmax + c);
    const bool bell = mp.mode == DAI8_GRAD_GVQ_MAX || (double)cnt > (double)mp.lambda * (double)M;
    float s;
    if (bell) {
      s = gmax;
    } else {
      const float s_prev = has_prev ? s_state[c] : gmax;
      s = __fadd_rn(__fmul_rn(t, s_prev), __fmul_rn(mp.A, gmax));
    }
    s_state[c] = s;
    if (cls) cls[c] = bell ? 1 : 0;
    if (stats_out) stats_out[c * 4 + DAI8_STAT_P] = (float)((double)cnt / (double)M);
  }
  if (threadIdx.x == 0) *gmax_layer = gmax_l;
}

// Layer-wise MCS: sigma of the whole layer from the per-channel means and sigmas (every channel has the
// same number of elements), written over every channel's sigma for the count sweep.
//   mean_l = sum_c mean_c / C;   var_l = sum_c (var_c + mean_c^2) / C - mean_l^2   (population form;
//   the sample form rescales by M/(M-1) per channel and back by CM/(CM-1))
__global__ void __launch_bounds__(kThreads)
layer_sigma_kernel(GvqWs ws, int C, int64_t M, McsDev mp, float* __restrict__ stats_out) {
  __shared__ double s_a[kThreads], s_b[kThreads];
  double a = 0.0, b = 0.0;
  const double unb = mp.std_unbiased && M > 1 ? (double)(M - 1) / (double)M : 1.0;   // back to sum of squares / M
  for (int c = threadIdx.x; c < C; c += kThreads) {
    const double m = (double)ws.mean[c], sg = (double)ws.sigma[c];
    a += m;
    b += sg * sg * unb + (mp.center_mean ? m * m : 0.0);
  }
  s_a[threadIdx.x] = a; s_b[threadIdx.x] = b;
  __syncthreads();
  for (int o = kThreads / 2; o > 0; o >>= 1) {
    if (threadIdx.x < o) { s_a[threadIdx.x] += s_a[threadIdx.x + o]; s_b[threadIdx.x] += s_b[threadIdx.x + o]; }
    __syncthreads();
  }
  const double mean_l = s_a[0] / (double)C;
  double var = s_b[0] / (double)C - (mp.center_mean ? mean_l * mean_l : 0.0);
  if (var < 0.0) var = 0.0;
  const double total = (double)M * (double)C;
  if (mp.std_unbiased && total > 1.0) var *= total / (total - 1.0);
  const float sigma_l = (float)sqrt(var);
  for (int c = threadIdx.x; c < C; c += kThreads) {
    ws.sigma[c] = sigma_l;
    if (stats_out) {      // in this mode the rows report the layer's mean and sigma
      stats_out[c * 4 + DAI8_STAT_MEAN] = (float)mean_l;
      stats_out[c * 4 + DAI8_STAT_SIGMA] = sigma_l;
    }
  }
}

// Sweep 2, NHWC.  grid = (pixel blocks, column blocks).
template <typename T, int VE>
__global__ void __launch_bounds__(kThreads)
count_nhwc_kernel(const T* __restrict__ x, int64_t npix, int C, int G, GvqWs ws,
                  const float* __restrict__ sigma, McsDev mp, float* __restrict__ s_state,
                  int has_prev, float* __restrict__ gmax_layer, float* __restrict__ stats_out,
                  uint8_t* __restrict__ cls) {
  __shared__ uint32_t scnt[kThreads * VE];
  const int tid = threadIdx.x;
  const int colv0 = blockIdx.y * kThreads;
  const int gcols = min(G - colv0, kThreads);
  const int rpi = kThreads / gcols;
  const int col = tid % gcols, rl = tid / gcols;
  const int64_t chunk = (npix + gridDim.x - 1) / gridDim.x;
  const int64_t p0 = (int64_t)blockIdx.x * chunk;
  const int64_t p1 = min(npix, p0 + chunk);
  uint32_t k[VE];
#pragma unroll
  for (int e = 0; e < VE; ++e) k[e] = 0;
  if (rl < rpi) {
    float sg[VE];
#pragma unroll
    for (int e = 0; e < VE; ++e) sg[e] = sigma[(colv0 + col) * VE + e];
    const T* base = x + (int64_t)(colv0 + col) * VE;
    for (int64_t p = p0 + rl; p < p1; p += rpi) {
      float v[VE];
      load_vec<T, VE>(base + p * C, v);
#pragma unroll
      for (int e = 0; e < VE; ++e) k[e] += (fabsf(v[e]) > sg[e]) ? 1u : 0u;
    }
  }
#pragma unroll
  for (int e = 0; e < VE; ++e) scnt[tid * VE + e] = k[e];
  __syncthreads();
  const int nch = gcols * VE;
  for (int j = tid; j < nch; j += kThreads) {
    const int cc = j / VE, e = j % VE;
    uint32_t acc = 0;
    for (int r = 0; r < rpi; ++r) acc += scnt[(r * gcols + cc) * VE + e];
    if (acc) atomicAdd(ws.cnt + colv0 * VE + j, acc);
  }
  if (!last_block_arrives(ws.ticket2, gridDim.x * gridDim.y)) return;
  solve_channels(ws, C, npix, mp, s_state, has_prev, gmax_layer, stats_out, cls);
}

// Sweep 2, NCHW.  grid = (C, slices over n).
template <typename T>
__global__ void __launch_bounds__(kThreads)
count_nchw_kernel(const T* __restrict__ x, int N, int C, int64_t HW, GvqWs ws,
                  const float* __restrict__ sigma, McsDev mp, float* __restrict__ s_state,
                  int has_prev, float* __restrict__ gmax_layer, float* __restrict__ stats_out,
                  uint8_t* __restrict__ cls) {
  const int c = blockIdx.x, tid = threadIdx.x;
  const int NS = gridDim.y;
  const int nper = (N + NS - 1) / NS;
  const int n0 = blockIdx.y * nper, n1 = min(N, n0 + nper);
  const float sg = sigma[c];
  uint32_t k = 0;
  for (int n = n0; n < n1; ++n) {
    const T* row = x + ((int64_t)n * C + c) * HW;
    for (int64_t i = tid; i < HW; i += kThreads) k += (fabsf(to_f32(row[i])) > sg) ? 1u : 0u;
  }
  for (int o = 16; o > 0; o >>= 1) k += __shfl_xor_sync(0xFFFFFFFFu, k, o);
  if ((tid & 31) == 0 && k) atomicAdd(ws.cnt + c, k);
  if (!last_block_arrives(ws.ticket2, gridDim.x * gridDim.y)) return;
  solve_channels(ws, C, (int64_t)N * HW, mp, s_state, has_prev, gmax_layer, stats_out, cls);
}

// ------------------------------------------------------------------------------------------------
// Sweep 3: Eq. 1 on every element.  Output 1 uses `scale1` (per channel if PER_CHANNEL, else one
// value) and generator stream 0; the optional output 2 uses the single value `scale2` and
// stream 1 (the two quantizations of Algorithm 1 fused, as Sec. 3.4 suggests).  STOCH selects the rounding.
// Codes are written as [pixel][Cp] with zero padding channels.
// ------------------------------------------------------------------------------------------------
template <int VE>
__device__ __forceinline__ void store_codes(int8_t* dst, const int (&q)[VE]);
template <>
__device__ __forceinline__ void store_codes<1>(int8_t* dst, const int (&q)[1]) { *dst = (int8_t)q[0]; }
template <>
__device__ __forceinline__ void store_codes<4>(int8_t* dst, const int (&q)[4]) {
  const uint32_t w = (q[0] & 0xFF) | ((q[1] & 0xFF) << 8) | ((q[2] & 0xFF) << 16) | ((uint32_t)q[3] << 24);
  *reinterpret_cast<uint32_t*>(dst) = w;
}
template <>
__device__ __forceinline__ void store_codes<8>(int8_t* dst, const int (&q)[8]) {
  uint2 w;
  w.x = (q[0] & 0xFF) | ((q[1] & 0xFF) << 8) | ((q[2] & 0xFF) << 16) | ((uint32_t)q[3] << 24);
  w.y = (q[4] & 0xFF) | ((q[5] & 0xFF) << 8) | ((q[6] & 0xFF) << 16) | ((uint32_t)q[7] << 24);
  *reinterpret_cast<uint2*>(dst) = w;
}

template <typename T, int VE, bool PER_CHANNEL, bool STOCH, bool DUAL>
__global__ void __launch_bounds__(kThreads)
quantize_nhwc_kernel(const T* __restrict__ x, int64_t npix, int64_t HW, int C, int Cp, int Gp,
                     const float* __restrict__ scale1, const float* __restrict__ scale2,
                     uint32_t seed, int8_t* __restrict__ q1, int8_t* __restrict__ q2) {
  const int tid = threadIdx.x;
  const int colv0 = blockIdx.y * kThreads;
  const int gcols = min(Gp - colv0, kThreads);
  const int rpi = kThreads / gcols;
  const int col = tid % gcols, rl = tid / gcols;
  if (rl >= rpi) return;
  const int64_t chunk = (npix + gridDim.x - 1) / gridDim.x;
  const int64_t p0 = (int64_t)blockIdx.x * chunk;
  const int64_t p1 = min(npix, p0 + chunk);
  const int c0 = (colv0 + col) * VE;  // first channel of this thread's vector
  const bool real = c0 < C;           // else: padding channels, write zeros (C % VE == 0)
  float inv1[VE];
  float inv2 = 0.f;
#pragma unroll
  for (int e = 0; e < VE; ++e) inv1[e] = real ? inv_scale(PER_CHANNEL ? scale1[c0 + e] : scale1[0]) : 0.f;
  if (DUAL) inv2 = inv_scale(scale2[0]);
  const uint32_t key0 = sr_key(seed, 0u);

  int64_t p = p0 + rl;
  if (p >= p1) return;
  int64_t n = p / HW;
  int64_t hw = p - n * HW;
  for (; p < p1; p += rpi) {
    int qa[VE], qb[VE];
    if (real) {
      float v[VE];
      load_vec<T, VE>(x + p * C + c0, v);
      // NCHW index of element (n, c0+e, hw): (n*C + c0 + e)*HW + hw
      const uint64_t idx0 = ((uint64_t)n * C + c0) * HW + hw;
#pragma unroll
      for (int e = 0; e < VE; ++e) {
        if (STOCH) {
          const uint64_t idx = idx0 + (uint64_t)e * HW;
          const uint32_t hi = (uint32_t)(idx >> 32);
          const uint32_t key = hi == 0u ? key0 : sr_key(seed, hi);
          const uint32_t f = sr_fold((uint32_t)idx, key), h = sr_bits0(f);
          qa[e] = quant_stochastic(v[e], inv1[e], sr_uniform(h));
          qb[e] = DUAL ? quant_stochastic(v[e], inv2, sr_uniform(sr_bits1(f))) : 0;
        } else {
          qa[e] = quant_nearest(v[e], inv1[e]);
          qb[e] = DUAL ? quant_nearest(v[e], inv2) : 0;
        }
      }
    } else {
#pragma unroll
      for (int e = 0; e < VE; ++e) { qa[e] = 0; qb[e] = 0; }
    }
    store_codes<VE>(q1 + p * Cp + c0, qa);
    if (DUAL) store_codes<VE>(q2 + p * Cp + c0, qb);
    hw += rpi;
    while (hw >= HW) { hw -= HW; ++n; }
  }
}

// NCHW input, NHWC codes: a block transposes a tile of 32 channels x 128 positions of one image
// through shared memory.  grid = (hw tiles, channel tiles over Cp, N).
constexpr int kTileC = 32, kTileHW = 128, kTileRow = 36;  // 36-byte rows: conflict-free byte writes

template <typename T, bool PER_CHANNEL, bool STOCH, bool DUAL>
__global__ void __launch_bounds__(kThreads)
quantize_nchw_kernel(const T* __restrict__ x, int C, int Cp, int64_t HW,
                     const float* __restrict__ scale1, const float* __restrict__ scale2,
                     uint32_t seed, int8_t* __restrict__ q1, int8_t* __restrict__ q2) {
  __shared__ __align__(16) int8_t t1[kTileHW * kTileRow];
  __shared__ __align__(16) int8_t t2[kTileHW * kTileRow];
  __shared__ float sinv[kTileC];
  const int tid = threadIdx.x;
  const int64_t hw0 = (int64_t)blockIdx.x * kTileHW;
  const int c0 = blockIdx.y * kTileC;
  const int n = blockIdx.z;
  if (tid < kTileC) {
    const int c = c0 + tid;
    sinv[tid] = c < C ? inv_scale(PER_CHANNEL ? scale1[c] : scale1[0]) : 0.f;
  }
  const float inv2 = DUAL ? inv_scale(scale2[0]) : 0.f;
  const uint32_t key0 = sr_key(seed, 0u);
  __syncthreads();
  for (int i = tid; i < kTileC * kTileHW; i += kThreads) {
    const int cl = i / kTileHW, hl = i % kTileHW;
    const int c = c0 + cl;
    const int64_t hw = hw0 + hl;
    int a = 0, b = 0;
    if (c < C && hw < HW) {
      const uint64_t idx = ((uint64_t)n * C + c) * HW + hw;
      const float v = to_f32(x[idx]);
      if (STOCH) {
        const uint32_t hi = (uint32_t)(idx >> 32);
        const uint32_t key = hi == 0u ? key0 : sr_key(seed, hi);
        const uint32_t f = sr_fold((uint32_t)idx, key), h = sr_bits0(f);
        a = quant_stochastic(v, sinv[cl], sr_uniform(h));
        if (DUAL) b = quant_stochastic(v, inv2, sr_uniform(sr_bits1(f)));
      } else {
        a = quant_nearest(v, sinv[cl]);
        if (DUAL) b = quant_nearest(v, inv2);
      }
    }
    t1[hl * kTileRow + cl] = (int8_t)a;
    if (DUAL) t2[hl * kTileRow + cl] = (int8_t)b;
  }
  __syncthreads();
  // 8 threads write the 32 bytes of one position; Cp is a multiple of 16, so a tile is 16 or 32 wide
  const int cw = min(kTileC, Cp - c0);
  for (int i = tid; i < kTileHW * (kTileC / 4); i += kThreads) {
    const int hl = i / (kTileC / 4), w4 = i % (kTileC / 4);
    const int64_t hw = hw0 + hl;
    if (hw < HW && w4 * 4 < cw) {
      const size_t o = ((size_t)n * HW + hw) * Cp + c0 + w4 * 4;
      *reinterpret_cast<uint32_t*>(q1 + o) = *reinterpret_cast<const uint32_t*>(t1 + hl * kTileRow + w4 * 4);
      if (DUAL) *reinterpret_cast<uint32_t*>(q2 + o) = *reinterpret_cast<const uint32_t*>(t2 + hl * kTileRow + w4 * 4);
    }
  }
}

// NCHW input with few positions per (n, c) row -- weights, (Cout, Cin, R, S) with H*W = R*S -- to
// [N][H*W][Cp] codes: the tile transpose above would leave most of its 128-position tiles empty.
// A block takes whole images n: their C*HW values are contiguous, are read coalesced, quantized
// into a [HW][Cp] image in shared memory and written out as 16-byte vectors.
template <typename T, bool STOCH>
__global__ void __launch_bounds__(kThreads)
quantize_nchw_rows_kernel(const T* __restrict__ x, int N, int C, int Cp, int HW, const float* __restrict__ scale,
                          uint32_t seed, int8_t* __restrict__ q) {
  extern __shared__ __align__(16) int8_t rows_sm[];      // [HW][Cp]
  grid_dependency_release();
  grid_dependency_wait();
  const int tid = threadIdx.x;
  const int per_n = C * HW, codes = HW * Cp;
  const float inv = inv_scale(*scale);
  const uint32_t key0 = sr_key(seed, 0u);
  for (int i = tid; i < codes / 4; i += kThreads) reinterpret_cast<uint32_t*>(rows_sm)[i] = 0u;   // padding channels stay 0
  __syncthreads();
  for (int n = blockIdx.x; n < N; n += gridDim.x) {
    const T* src = x + (size_t)n * per_n;
    for (int i = tid; i < per_n; i += kThreads) {
      const int c = i / HW, hw = i - c * HW;
      const float v = to_f32(src[i]);
      int code;
      if (STOCH) {
        const uint64_t idx = (uint64_t)n * per_n + (uint64_t)i;       // the NCHW index
        const uint32_t hi = (uint32_t)(idx >> 32);
        const uint32_t key = hi == 0u ? key0 : sr_key(seed, hi);
        code = quant_stochastic(v, inv, sr_uniform(sr_bits0(sr_fold((uint32_t)idx, key))));
      } else {
        code = quant_nearest(v, inv);
      }
      rows_sm[hw * Cp + c] = (int8_t)code;
    }
    __syncthreads();
    uint4* dst = reinterpret_cast<uint4*>(q + (size_t)n * codes);
    for (int i = tid; i < codes / 16; i += kThreads) dst[i] = reinterpret_cast<const uint4*>(rows_sm)[i];
    __syncthreads();
  }
}

// Eq. 1 for an NHWC tensor of at most 16 channels (the images a network's first layer reads): a thread
// owns one pixel and writes its padded code row as one 16-byte vector.
template <typename T, bool STOCH>
__global__ void __launch_bounds__(kThreads)
quantize_nhwc_c16_kernel(const T* __restrict__ x, int64_t npix, int64_t HW, int C, const float* __restrict__ scale,
                         uint32_t seed, int8_t* __restrict__ q) {
  const float inv = inv_scale(*scale);
  const uint32_t key0 = sr_key(seed, 0u);
  for (int64_t pix = (int64_t)blockIdx.x * kThreads + threadIdx.x; pix < npix; pix += (int64_t)gridDim.x * kThreads) {
    const T* src = x + pix * C;
    uint32_t b[16];
    uint64_t idx = 0;
    if (STOCH) {
      const int64_t n = pix / HW;
      idx = (uint64_t)n * (uint64_t)C * (uint64_t)HW + (uint64_t)(pix - n * HW);   // NCHW index of channel 0
    }
#pragma unroll
    for (int c = 0; c < 16; ++c) {
      b[c] = 0u;
      if (c < C) {
        const float v = to_f32(src[c]);
        if (STOCH) {
          const uint32_t hi = (uint32_t)(idx >> 32);
          const uint32_t key = hi == 0u ? key0 : sr_key(seed, hi);
          b[c] = quant_stochastic_bits(v, inv, sr_uniform(sr_bits0(sr_fold((uint32_t)idx, key))));
          idx += (uint64_t)HW;
        } else {
          b[c] = quant_nearest_bits(v, inv);
        }
      }
    }
    *reinterpret_cast<uint4*>(q + pix * 16) = make_uint4(pack_codes4(b[0], b[1], b[2], b[3]), pack_codes4(b[4], b[5], b[6], b[7]),
                                                         pack_codes4(b[8], b[9], b[10], b[11]), pack_codes4(b[12], b[13], b[14], b[15]));
  }
}

// max|x| over a whole tensor (layout-free), into the bit pattern at out_bits (zeroed before).
template <typename T, int VE>
__global__ void __launch_bounds__(kThreads)
absmax_kernel(const T* __restrict__ x, int64_t nvec, uint32_t* __restrict__ out_bits) {
  float m = 0.f;
  for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < nvec; i += (int64_t)gridDim.x * kThreads) {
    float v[VE];
    load_vec<T, VE>(x + i * VE, v);
#pragma unroll
    for (int e = 0; e < VE; ++e) m = fmaxf(m, fabsf(v[e]));
  }
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  if ((threadIdx.x & 31) == 0 && m > 0.f) atomicMax(out_bits, __float_as_uint(m));
}

// Eq. 1 with one scale and nearest rounding over a tensor whose codes have the layout of its values
// (NHWC with C a multiple of 16, or any layout-free use): no index arithmetic at all.  The vectors are
// visited from the END of the tensor downwards: absmax_kernel, which runs just before, has left the
// tail of the tensor in L2, so most of this second read never reaches DRAM.
template <typename T, int VE>
__global__ void __launch_bounds__(kThreads)
quantize_flat_nearest_kernel(const T* __restrict__ x, int64_t nvec, const float* __restrict__ scale,
                             int8_t* __restrict__ q) {
  grid_dependency_release();
  grid_dependency_wait();
  const float inv = inv_scale(*scale);
  const int64_t stride = (int64_t)gridDim.x * kThreads;
#pragma unroll 4
  for (int64_t i = nvec - 1 - ((int64_t)blockIdx.x * kThreads + threadIdx.x); i >= 0; i -= stride) {
    float v[VE];
    load_vec<T, VE>(x + i * VE, v);
    uint32_t r[VE];
#pragma unroll
    for (int e = 0; e < VE; ++e) r[e] = quant_nearest_bits(v[e], inv);
    if constexpr (VE == 8)
      *reinterpret_cast<uint2*>(q + i * VE) = make_uint2(pack_codes4(r[0], r[1], r[2], r[3]), pack_codes4(r[4], r[5], r[6], r[7]));
    else
      *reinterpret_cast<uint32_t*>(q + i * VE) = pack_codes4(r[0], r[1], r[2], r[3]);
  }
}

// ------------------------------------------------------------------------------------------------
// Fused NHWC path: statistics, density count, clip update and both code tensors in ONE persistent
// cooperative kernel, one CTA per SM, in two sweeps over dY (plus a rare partial third).
//
// A CTA owns a contiguous range of pixels, i.e. a contiguous byte range of dY.  One producer warp
// streams that range into shared memory with bulk asynchronous copies (cp.async.bulk, completion on
// mbarriers) in pieces of up to 32 KB; sixteen consumer warps work on the pieces.  As many pieces as
// fit stay resident for all sweeps, the rest cycles through a small ring and is fetched again in the
// later sweeps (L2 hits for tensors of up to ~100 MB).  The producer runs ahead across sweep
// boundaries, so the first pieces of the next sweep are already in flight while the CTAs meet at a
// grid barrier.
//
// Sweep 1 takes the statistics.  The per-CTA partial moments are combined once: channel c is
// finished by one warp of CTA c mod gridDim.x (fixed order, hence deterministic), and after a second
// barrier every CTA reads the finished |g|max and sigma.  Sweep 2 takes the density count AND writes
// the codes, with the clip value of the class it predicts for each channel.  The per-CTA partial
// counts are summed the same distributed way after a third barrier; the class that the count yields
// is the one reported and the one the codes must match, so the warp that classifies a channel flags
// a wrong prediction, and after a fourth barrier the flagged channels are re-quantized in a fix-up
// sweep that only their threads take part in.
//
// Two things bound this kernel, and neither is HBM.  (1) The integer/logic pipe in sweep 2, which
// issues at half the rate of the floating-point pipes: every element needs a 32-bit hash, two
// uniforms and two stochastic roundings.  So bf16 inputs take |g|max and the density count two
// elements at a time in packed bf16 arithmetic (both are exact there), codes come out of a
// magic-number addition instead of a float-to-int conversion, rows without large elements skip the
// clamps and add in pairs, and tensors of fewer than 2^32 elements use 32-bit index arithmetic.
// (2) Everything outside the loops runs exactly once per CTA, straight from a cold instruction
// cache, at roughly ten cycles per instruction: the code between the loops is therefore kept SMALL
// rather than fast -- out-of-line reduction routines with run-time loops, no binary64 division or
// square root (reciprocals come from the host), spin loops out of line.
// ------------------------------------------------------------------------------------------------
constexpr int kFT = 512;             // consumer threads per CTA (one CTA per SM)
constexpr int kFusedThreads = kFT + 32;  // plus the producer warp
constexpr int kFusedMaxC = 2048;     // per-channel scalars kept in shared memory
constexpr int kMaxSlots = 28;        // shared-memory pieces per CTA
constexpr int kMaxRing = 8;          // of which at most this many cycle when not all pieces fit
constexpr int kPieceBytes = 32768;
constexpr long long kWaitTimeoutCycles = 2000000000LL;  // about one second

// reduction scratch at the start of the dynamic shared memory: per consumer thread and vector
// element one float (max) and two doubles (sum, sum of squares)
__host__ __device__ constexpr size_t fused_red_bytes(int ve) { return (size_t)ve * kFT * 20; }

__device__ __forceinline__ void unpack_raw(const uint4& r, float (&v)[4], const float*) {
  v[0] = __uint_as_float(r.x); v[1] = __uint_as_float(r.y); v[2] = __uint_as_float(r.z); v[3] = __uint_as_float(r.w);
}
__device__ __forceinline__ void unpack_raw(const uint4& r, float (&v)[8], const bf16_t*) {
  const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) { v[2 * i] = __uint_as_float(w[i] << 16); v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u); }
}

// Packed bf16 helpers (two values per 32-bit word).  max and compare are exact in bf16.
__device__ __forceinline__ uint32_t bf16x2_max(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
// 1.0 (0x3F80) in every half where a > b, else 0.
__device__ __forceinline__ uint32_t bf16x2_gt_one(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("set.gt.bf16x2.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t bf16x2_add(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}

// Two binary32 additions per instruction on a register pair (lower word = first element).  Each
// half is rounded exactly like the scalar addition of the same rounding mode.  There is no packed
// multiply here on purpose: the assembler contracts a packed multiply with a packed addition that
// consumes it into one fused operation (observed: codes that differ from the two-rounding
// definition about once in 2^21 elements), which it never does with the scalar __fmul_rn.
__device__ __forceinline__ uint64_t f32x2_pack(uint32_t lo, uint32_t hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
  return r;
}
__device__ __forceinline__ void f32x2_unpack(uint64_t p, uint32_t& lo, uint32_t& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(p));
}
__device__ __forceinline__ uint64_t f32x2_add_rn(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t f32x2_add_rd(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rm.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}

// ---- mbarrier / bulk-copy wrappers ---------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false if the CTA is giving up (this wait or another one ran out).
__device__ __noinline__ bool mbar_wait_slow(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                            unsigned int* status, long long limit) {
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > limit) {
      *abort_flag = 1u;
      atomicExch(status, (unsigned int)DAI8_ERR_TIMEOUT);
      return false;
    }
  }
}
// `limit`: cycles after which the wait gives up (the default, about a second, everywhere but in the
// self-test of the give-up path).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          unsigned int* status, long long limit = kWaitTimeoutCycles) {
  if (mbar_try_wait(bar, parity)) return true;
  return mbar_wait_slow(bar, parity, abort_flag, status, limit);
}
// Contiguous global -> shared copy of `bytes` (multiple of 16, both addresses 16-byte aligned).
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kFT) : "memory"); }

struct FusedArgs {
  int64_t npix, HW;
  double inv_M, inv_denom; // 1/M and 1/(M or M-1), from the host
  float pred_ratio;        // a channel is predicted bell-shaped when |g|max < pred_ratio * sigma
  int C, Cp, G, Gp;        // G input vector columns, Gp output vector columns (>= G, zero padding)
  int rows_per_warp, rpi;  // thread tiling, see fused_map
  int rp;                  // pixel rows per piece (a multiple of rpi)
  int adv_q, adv_rem;      // rpi / HW and rpi % HW: how the (image, pixel) position advances per iteration
  int slots, ring_log2;    // shared-memory pieces per CTA; log2 of how many of them cycle when not all fit
  GvqWs ws;
  uint32_t* gridbar;
  const float* sigma_override;
  McsDev mp;
  float* s_state;
  int has_prev;
  float* gmax_layer;
  float* stats_out;
  uint8_t* cls;
  uint32_t seed;
  int8_t* q1;
  int8_t* q2;
  unsigned int* status;
};

// All consumer threads of all CTAs of a cooperative launch meet here.  Bounded: returns false (in
// every consumer thread of the CTA) if the others do not arrive in time, after recording
// DAI8_ERR_TIMEOUT.
__device__ __noinline__ bool grid_barrier(uint32_t* counter, uint32_t target, unsigned int* status,
                                          volatile uint32_t* abort_flag, uint32_t* s_ok,
                                          long long limit = kWaitTimeoutCycles) {
  consumer_sync();
  if (threadIdx.x == 0) {
    // release: the CTA's writes (ordered before this thread by the barrier above) become visible
    // to whoever acquires the counter; acquire: the other CTAs' writes are visible after the loop
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(counter) : "memory");
    uint32_t ok = *abort_flag ? 0u : 1u;
    const long long t0 = clock64();
    for (;;) {
      uint32_t seen;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
      if (!ok || seen >= target) break;
      if (clock64() - t0 > limit) {
        atomicExch(status, (unsigned int)DAI8_ERR_TIMEOUT);
        *abort_flag = 1u;
        ok = 0u;
      }
    }
    *s_ok = ok;
  }
  consumer_sync();
  return *reinterpret_cast<volatile uint32_t*>(s_ok) != 0u;
}

// How the 512 consumer threads of a CTA tile (pixel row, vector column) pairs: with Gp <= 32 vector
// columns, Gp a divisor of 32, a warp holds rows_per_warp = 32/Gp whole rows; otherwise the CTA holds
// rpi = 512/Gp rows that run across warp boundaries (only 512 mod Gp threads idle).
__host__ __device__ inline int fused_rows_per_iteration(int Gp) { return (Gp <= 32 && 32 % Gp == 0) ? (kFT / 32) * (32 / Gp) : kFT / Gp; }

// Combines, in a fixed order, what the consumer threads have stored per (vector element e, pixel
// row lane, vector column) at index e*kFT + row*Gp + col over the row lanes, and writes the result for
// channel c = col*VE + e (c < C).  First `parts` interleaved subsets of the rows are combined in
// place by all threads, then the subsets.  Ends with a consumer barrier, after which the scratch may
// be rewritten.  Out of line, with run-time loops: it runs once per call and is kept small.
struct RedIndex { int total0, parts, NV; };
__device__ __forceinline__ RedIndex red_index(int rows, int Gp, int VE) {
  RedIndex r;
  r.NV = VE * Gp;
  r.parts = r.NV >= kFT ? 1 : kFT / r.NV;
  if (r.parts > rows) r.parts = rows;
  r.total0 = r.NV * r.parts;
  return r;
}

// max (float) and two sums (double) at once: the statistics of phase 1
__device__ __noinline__ void column_reduce_stats(float* smax, double* ssum, double* sss, int rows, int Gp, int VE,
                                                 int C, float* out_max, double* out_sum, double* out_ss) {
  const int tid = threadIdx.x;
  const RedIndex ri = red_index(rows, Gp, VE);
  consumer_sync();
#pragma unroll 1
  for (int idx = tid; idx < ri.total0; idx += kFT) {
    const int p = idx / ri.NV, j = idx - p * ri.NV;
    const int e = j / Gp, col = j - e * Gp;
    const int cell = e * kFT + p * Gp + col;
    float m = smax[cell];
    double s1 = ssum[cell], s2 = sss[cell];
#pragma unroll 4
    for (int r = p + ri.parts; r < rows; r += ri.parts) {
      const int o = cell + (r - p) * Gp;
      m = fmaxf(m, smax[o]); s1 += ssum[o]; s2 += sss[o];
    }
    smax[cell] = m; ssum[cell] = s1; sss[cell] = s2;
  }
  consumer_sync();
#pragma unroll 1
  for (int j = tid; j < ri.NV; j += kFT) {
    const int e = j / Gp, col = j - e * Gp;
    const int cell = e * kFT + col;
    float m = smax[cell];
    double s1 = ssum[cell], s2 = sss[cell];
#pragma unroll 4
    for (int p = 1; p < ri.parts; ++p) {
      const int o = cell + p * Gp;
      m = fmaxf(m, smax[o]); s1 += ssum[o]; s2 += sss[o];
    }
    const int c = col * VE + e;
    if (c < C) { out_max[c] = m; out_sum[c] = s1; out_ss[c] = s2; }
  }
  consumer_sync();
}

// counts of phase 2, written to this CTA's row of partial counts
__device__ __noinline__ void column_reduce_counts(uint32_t* scnt, int rows, int Gp, int VE, int C, uint32_t* out) {
  const int tid = threadIdx.x;
  const RedIndex ri = red_index(rows, Gp, VE);
  consumer_sync();
#pragma unroll 1
  for (int idx = tid; idx < ri.total0; idx += kFT) {
    const int p = idx / ri.NV, j = idx - p * ri.NV;
    const int e = j / Gp, col = j - e * Gp;
    const int cell = e * kFT + p * Gp + col;
    uint32_t n = scnt[cell];
#pragma unroll 4
    for (int r = p + ri.parts; r < rows; r += ri.parts) n += scnt[cell + (r - p) * Gp];
    scnt[cell] = n;
  }
  consumer_sync();
#pragma unroll 1
  for (int j = tid; j < ri.NV; j += kFT) {
    const int e = j / Gp, col = j - e * Gp;
    const int cell = e * kFT + col;
    uint32_t n = scnt[cell];
#pragma unroll 4
    for (int p = 1; p < ri.parts; ++p) n += scnt[cell + p * Gp];
    const int c = col * VE + e;
    if (c < C) out[c] = n;
  }
  consumer_sync();
}

// The rare sigma whose square leaves the binary32 range.
__device__ __noinline__ float sigma_wide(double var_over_denom) { return (float)sqrt(var_over_denom); }

template <typename T, int VE, bool DUAL, bool IDX32>
__global__ void __launch_bounds__(kFusedThreads, 1)
gvq_fused_nhwc_kernel(const T* __restrict__ x, const FusedArgs a) {
  constexpr bool kPacked = VE == 8;  // bf16 vectors: packed max / compare
  extern __shared__ __align__(128) uint8_t fsmem[];
  __shared__ uint64_t full_bar[kMaxSlots], empty_bar[kMaxRing];
  __shared__ volatile uint32_t s_abort;
  __shared__ uint32_t s_ok;
  __shared__ volatile uint32_t s_fix;        // 0 undecided, 1 no fix-up pass, 2 fix-up pass
  __shared__ uint32_t s_any_mis;

  double* red_sum = reinterpret_cast<double*>(fsmem);                    // [VE][kFT]
  double* red_ss = red_sum + (size_t)VE * kFT;                           // [VE][kFT]
  float* red_max = reinterpret_cast<float*>(red_ss + (size_t)VE * kFT);  // [VE][kFT]
  uint32_t* red_cnt = reinterpret_cast<uint32_t*>(fsmem);                // [VE][kFT]
  float* ch_absmax = reinterpret_cast<float*>(fsmem + fused_red_bytes(VE));  // [C + 1], last = layer |g|max
  float* ch_sigma = ch_absmax + a.C + 1;                                 // [C]
  float* ch_sprev = ch_sigma + a.C;                                      // [C]
  float* ch_inv = ch_sprev + a.C;                                        // [C + 1], last = layer scale
  uint8_t* ch_pred = reinterpret_cast<uint8_t*>(ch_inv + a.C + 1);       // [C] predicted class; 2 = mispredicted
  uint8_t* pieces = fsmem + ((fused_red_bytes(VE) + (size_t)a.C * 17 + 8 + 127) / 128) * 128;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int C = a.C, Gp = a.Gp, G = a.G;
  const int rb = C * (int)sizeof(T);                 // bytes per pixel row
  const int rp = a.rp;
  const uint32_t piece_stride = (uint32_t)rp * (uint32_t)rb;   // bytes per shared-memory piece
  const int64_t chunk = (a.npix + gridDim.x - 1) / gridDim.x;
  const int64_t p0 = (int64_t)blockIdx.x * chunk;
  const int64_t p1 = min(a.npix, p0 + chunk);
  const int rows_total = p1 > p0 ? (int)(p1 - p0) : 0;
  const int K = (rows_total + rp - 1) / rp;          // pieces of this CTA
  const int ring = 1 << a.ring_log2;
  const int R = K <= a.slots ? K : a.slots - ring;   // pieces that stay resident
  const int NS = K - R;                              // pieces streamed again in every phase

  if (tid == 0) {
    s_abort = 0u; s_fix = 0u; s_any_mis = 0u;
#pragma unroll 1
    for (int s = 0; s < kMaxSlots; ++s) mbar_init(&full_bar[s], 1);
#pragma unroll 1
    for (int r = 0; r < kMaxRing; ++r) mbar_init(&empty_bar[r], kFT / 32);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  // ---------------- producer warp ------------------------------------------------------------------
  if (warp == kFT / 32) {
    if (lane == 0) {
      const uint8_t* src = reinterpret_cast<const uint8_t*>(x) + (size_t)p0 * rb;
      // resident pieces once, then one pass over the streamed ones per sweep: statistics, the
      // count + quantize sweep, and -- only if a channel's class was mispredicted -- the fix-up sweep
      int k = 0;
      auto issue = [&](int begin, int end) {
#pragma unroll 1
        for (int i = begin; i < end; ++i) {
          int slot = i;
          if (i >= R) {
            const int t = i - R, r = t & (ring - 1);
            slot = R + r;
            if (t >= ring && !mbar_wait(&empty_bar[r], (uint32_t)((t >> a.ring_log2) - 1) & 1u, &s_abort, a.status)) return false;
          }
          const uint32_t bytes = (uint32_t)min(rp, rows_total - k * rp) * (uint32_t)rb;
          mbar_expect_tx(&full_bar[slot], bytes);
          bulk_load(pieces + (size_t)slot * piece_stride, src + (size_t)k * piece_stride, bytes, &full_bar[slot]);
          if (++k == K) k = R;
        }
        return true;
      };
      if (issue(0, R + 2 * NS) && NS > 0) {
        const long long t0 = clock64();
        while (s_fix == 0u && !s_abort) {          // the consumers decide after the last grid barrier
          if (clock64() - t0 > kWaitTimeoutCycles) { s_abort = 1u; atomicExch(a.status, (unsigned int)DAI8_ERR_TIMEOUT); }
          __nanosleep(200);
        }
        if (s_fix == 2u && !s_abort) issue(R + 2 * NS, R + 3 * NS);
      }
    }
    return;
  }

  // ---------------- consumers ----------------------------------------------------------------------
  int col, rl;
  bool active;
  if (a.rows_per_warp > 0) {       // Gp divides 32: a warp holds rows_per_warp whole rows
    const int r = lane / Gp;
    col = lane - r * Gp;
    rl = warp * a.rows_per_warp + r;
    active = r < a.rows_per_warp;
  } else {
    rl = tid / Gp;
    col = tid - rl * Gp;
    active = rl < a.rpi;
  }
  const int rpi = a.rpi;
  const bool real = active && col < G;       // has input; columns >= G are code padding
  const int c0 = col * VE;
  const int pos = rl * Gp + col;             // this thread's cell in the reduction scratch
  int t_cons = 0;                            // streamed pieces consumed so far (all phases)
  bool ok = true;

  // Runs f(shared-memory piece, rows in it) over the CTA's pieces from `first_piece` on, in order:
  // the resident ones wait for their one and only fill, the others for the current fill of their
  // ring slot.  After phase 1 the resident pieces are one contiguous run of rows_res rows.
  auto for_each_piece = [&](int first_piece, auto&& f) {
#pragma unroll 1
    for (int j = first_piece; j < K && ok; ++j) {
      int slot = j, r = 0;
      uint32_t parity = 0u;
      if (j >= R) {
        const int t = t_cons + (j - R);
        r = t & (ring - 1);
        slot = R + r;
        parity = (uint32_t)(t >> a.ring_log2) & 1u;
      }
      ok = mbar_wait(&full_bar[slot], parity, &s_abort, a.status);
      if (ok) f(pieces + (size_t)slot * piece_stride, min(rp, rows_total - j * rp));
      if (j >= R) {
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[r]);
      }
    }
    t_cons += NS;
  };
  const int rows_res = min(rows_total, R * rp);
  auto vec_at = [&](const uint8_t* piece, int row) {
    return *reinterpret_cast<const uint4*>(piece + ((uint32_t)row * (uint32_t)G + (uint32_t)col) * 16u);
  };

  // ---------------- phase 1: statistics -----------------------------------------------------------
  {
    float amax[VE], fs[VE], fss[VE], piv[VE];
    uint32_t amax2[4] = {0u, 0u, 0u, 0u};
    double ds[VE], dss[VE];
#pragma unroll
    for (int e = 0; e < VE; ++e) { amax[e] = 0.f; fs[e] = 0.f; fss[e] = 0.f; ds[e] = 0.0; dss[e] = 0.0; piv[e] = 0.f; }
    if (real) load_vec<T, VE>(x + c0, piv);  // pixel 0 of these channels
    int run = 0;
    for_each_piece(0, [&](const uint8_t* piece, int rows) {
      if (!real) return;
#pragma unroll 1
      for (int row = rl; row < rows; row += rpi) {
        const uint4 raw = vec_at(piece, row);
        float v[VE];
        unpack_raw(raw, v, (const T*)nullptr);
        if constexpr (kPacked) {
          const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) amax2[j] = bf16x2_max(amax2[j], w[j] & 0x7FFF7FFFu);
        }
#pragma unroll
        for (int e = 0; e < VE; ++e) {
          if constexpr (!kPacked) amax[e] = fmaxf(amax[e], fabsf(v[e]));
          const float d = v[e] - piv[e];
          fs[e] += d;
          fss[e] = fmaf(d, d, fss[e]);
        }
        if (++run == 32) {  // short fp32 runs, combined in binary64
          run = 0;
#pragma unroll
          for (int e = 0; e < VE; ++e) { ds[e] += (double)fs[e]; dss[e] += (double)fss[e]; fs[e] = 0.f; fss[e] = 0.f; }
        }
      }
    });
    if constexpr (kPacked) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        amax[2 * j] = __uint_as_float(amax2[j] << 16);
        amax[2 * j + 1] = __uint_as_float(amax2[j] & 0xFFFF0000u);
      }
    }
    // per-CTA partials of every channel: [blockIdx][C] rows of the workspace
    const size_t prow = (size_t)blockIdx.x * C;
    if (active) {
#pragma unroll
      for (int e = 0; e < VE; ++e) {
        red_max[e * kFT + pos] = amax[e];
        red_sum[e * kFT + pos] = ds[e] + (double)fs[e];
        red_ss[e * kFT + pos] = dss[e] + (double)fss[e];
      }
    }
    column_reduce_stats(red_max, red_sum, red_ss, rpi, Gp, VE, C, a.ws.pmax + prow, a.ws.psum + prow, a.ws.pss + prow);
  }
  // previous clip values are read before the barriers after which CTA 0 overwrites them
#pragma unroll 1
  for (int c = tid; c < C; c += kFT) ch_sprev[c] = a.has_prev ? a.s_state[c] : 0.f;
  ok = grid_barrier(a.gridbar, gridDim.x, a.status, &s_abort, &s_ok) && ok;

  // channel c is finished by one warp of CTA (c mod gridDim.x): fixed order over the CTAs' partials
  if (ok) {
    const int nblk = gridDim.x;
#pragma unroll 1
    for (int c = blockIdx.x + nblk * warp; c < C; c += nblk * (kFT / 32)) {
      float mx = 0.f;
      double s1 = 0.0, s2 = 0.0;
      const double pivot = (double)to_f32(x[c]);
#pragma unroll 1
      for (int b0 = lane; b0 < nblk; b0 += 32 * 5) {   // five independent partials per round trip
        float pm[5];
        double p1[5], p2[5];
#pragma unroll
        for (int u = 0; u < 5; ++u) {
          const int b = b0 + 32 * u;
          const size_t idx = (size_t)(b < nblk ? b : b0) * C + c;
          pm[u] = __ldcg(a.ws.pmax + idx); p1[u] = __ldcg(a.ws.psum + idx); p2[u] = __ldcg(a.ws.pss + idx);
        }
#pragma unroll
        for (int u = 0; u < 5; ++u)
          if (b0 + 32 * u < nblk) { mx = fmaxf(mx, pm[u]); s1 += p1[u]; s2 += p2[u]; }
      }
#pragma unroll 1
      for (int o = 16; o > 0; o >>= 1) {
        mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
        s1 += __shfl_xor_sync(0xFFFFFFFFu, s1, o);
        s2 += __shfl_xor_sync(0xFFFFFFFFu, s2, o);
      }
      if (lane == 0) {
        // mean and sigma from the moments of d = g - pivot; the pivot (the channel's first element)
        // keeps sum d^2 - (sum d)^2/M free of cancellation when |mean| >> sigma
        const double md = s1 * a.inv_M;
        double var = a.mp.center_mean ? (s2 - s1 * md)
                                      : (s2 + 2.0 * pivot * s1 + pivot * pivot * (double)a.npix);
        var = fmax(var, 0.0) * a.inv_denom;
        const float vf = (float)var;
        const float sigma = (vf > 1e-30f || var == 0.0) ? sqrtf(vf) : sigma_wide(var);
        const float mean = (float)(pivot + md);
        a.ws.absmax[c] = mx; a.ws.mean[c] = mean; a.ws.sigma[c] = sigma;
        if (a.stats_out) {
          a.stats_out[c * 4 + DAI8_STAT_ABSMAX] = mx;
          a.stats_out[c * 4 + DAI8_STAT_MEAN] = mean;
          a.stats_out[c * 4 + DAI8_STAT_SIGMA] = sigma;
        }
        if (mx > 0.f) atomicMax(a.ws.gmax_bits, __float_as_uint(mx));  // non-negative floats order like their bits
      }
    }
  }
  ok = grid_barrier(a.gridbar, 2u * gridDim.x, a.status, &s_abort, &s_ok) && ok;

  // Every CTA now holds |g|max and sigma of every channel.  The class (Eq. 15) needs one more
  // sweep for the density count, the codes another one; to save a sweep the class is PREDICTED --
  // from the caller's classes of the previous iteration if given, else from |g|max / sigma, which
  // is about sqrt(2 ln M) for a bell-shaped and ln(M)/sqrt(2) for a long-tailed channel -- and the
  // codes are written with the clip value of the predicted class while the count is taken.  After
  // the count the true class is known; channels whose prediction was wrong (rare) get their
  // per-channel codes rewritten in a fix-up sweep, so the result never depends on the prediction.
  const float tcoef = __fsub_rn(1.0f, __fmul_rn(a.mp.k, a.mp.A));
  if (ok) {
    const bool hinted = a.has_prev && a.cls != nullptr;
#pragma unroll 1
    for (int c = tid; c <= C; c += kFT) {     // entry C: the layer-wide scale
      float gmax, s;
      if (c < C) {
        gmax = __ldcg(a.ws.absmax + c);
        const float sigma = __ldcg(a.ws.sigma + c);
        ch_sigma[c] = a.sigma_override ? a.sigma_override[c] : sigma;
        const bool pred = hinted ? a.cls[c] != 0 : gmax < a.pred_ratio * sigma;
        ch_pred[c] = pred ? 1 : 0;
        s = gmax;
        if (!pred) s = __fadd_rn(__fmul_rn(tcoef, a.has_prev ? ch_sprev[c] : gmax), __fmul_rn(a.mp.A, gmax));
      } else {
        gmax = __uint_as_float(__ldcg(a.ws.gmax_bits));
        s = gmax;
      }
      ch_absmax[c] = gmax;
      ch_inv[c] = inv_scale(s);
    }
    consumer_sync();
  }

  // ---------------- sweep 2: density count + both sets of codes --------------------------------------
  using Idx = typename std::conditional<IDX32, uint32_t, uint64_t>::type;
  const uint32_t key0 = sr_key(a.seed, 0u);
  const Idx HWi = (Idx)a.HW;
  const Idx wrap = (Idx)(C - 1) * HWi;           // added to the NCHW index when n advances
  const int64_t first = p0 + rl;                 // this thread's first pixel
  int64_t n0;
  if constexpr (IDX32) n0 = (int64_t)((uint32_t)first / (uint32_t)a.HW);   // fewer than 2^32 elements
  else n0 = first / a.HW;
  const Idx hw_first = (Idx)(first - n0 * a.HW);
  const Idx idx_first = ((Idx)n0 * (Idx)C + (Idx)c0) * HWi + hw_first;   // NCHW index of (n, c0, hw)
  const size_t o_stride = (size_t)rpi * a.Cp;
  const Idx adv_rem = (Idx)a.adv_rem, adv_idx = (Idx)rpi + (Idx)a.adv_q * wrap;
  Idx hw = hw_first, idx0 = idx_first;
  int8_t* o1 = a.q1 + first * a.Cp + c0;
  int8_t* o2 = DUAL ? a.q2 + first * a.Cp + c0 : nullptr;
  float inv1[VE];
  auto hash_at = [&](Idx idx) -> uint32_t {     // the element's folded multiply (sr_fold)
    if constexpr (IDX32) {
      return sr_fold(idx, key0);
    } else {
      const uint32_t hi = (uint32_t)(idx >> 32);
      const uint32_t key = hi == 0u ? key0 : sr_key(a.seed, hi);
      return sr_fold((uint32_t)idx, key);
    }
  };
  // One pixel's vector of this thread: codes with inv1 (and, if with_gq, the layer-wide ones).
  // `unclipped` promises |g * inv| <= 126.75 for every element and both scales: then neither clamp of
  // the stochastic quantizer can act (v + u stays inside (-127.75, 127.75)), so the codes are
  // floor(fl(fl(g * inv) + u)) and the additions run two elements at a time.
  auto quantize_row = [&](const uint4& raw, bool with_gq, float inv2, bool unclipped, auto has_input) {
    uint32_t ra[VE], rb2[VE];
    if constexpr (decltype(has_input)::value) {
      Idx idx = idx0;
      bool done = false;
      if constexpr (kPacked) {
        if (unclipped) {
          done = true;
          const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
          const uint32_t one_bits = 0xBF800000u, magic_bits = 0x4B400000u;   // -1.0f, 1.5 * 2^23
          const uint64_t minus1 = f32x2_pack(one_bits, one_bits), magic = f32x2_pack(magic_bits, magic_bits);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint32_t h0 = hash_at(idx);
            idx += HWi;
            const uint32_t h1 = hash_at(idx);
            idx += HWi;
            const float g0 = __uint_as_float(w[j] << 16), g1 = __uint_as_float(w[j] & 0xFFFF0000u);
            const uint64_t v1 = f32x2_pack(__float_as_uint(__fmul_rn(g0, inv1[2 * j])), __float_as_uint(__fmul_rn(g1, inv1[2 * j + 1])));
            const uint64_t u1 = f32x2_add_rn(f32x2_pack(__funnelshift_r(sr_bits0(h0), 0x7Fu, 9), __funnelshift_r(sr_bits0(h1), 0x7Fu, 9)), minus1);
            f32x2_unpack(f32x2_add_rd(f32x2_add_rn(v1, u1), magic), ra[2 * j], ra[2 * j + 1]);
            if constexpr (DUAL) {
              if (with_gq) {
                const uint64_t u2 = f32x2_add_rn(f32x2_pack(__funnelshift_r(sr_bits1(h0), 0x7Fu, 9),
                                                            __funnelshift_r(sr_bits1(h1), 0x7Fu, 9)), minus1);
                const uint64_t v2 = f32x2_pack(__float_as_uint(__fmul_rn(g0, inv2)), __float_as_uint(__fmul_rn(g1, inv2)));
                f32x2_unpack(f32x2_add_rd(f32x2_add_rn(v2, u2), magic), rb2[2 * j], rb2[2 * j + 1]);
              }
            }
          }
        }
      }
      if (!done) {
        float v[VE];
        unpack_raw(raw, v, (const T*)nullptr);
#pragma unroll
        for (int e = 0; e < VE; ++e) {
          const uint32_t f = hash_at(idx), h = sr_bits0(f);
          ra[e] = quant_stochastic_bits(v[e], inv1[e], sr_uniform_fast(h));
          if constexpr (DUAL) {
            if (with_gq) rb2[e] = quant_stochastic_bits(v[e], inv2, sr_uniform_fast(sr_bits1(f)));
          }
          idx += HWi;
        }
      }
    } else {
#pragma unroll
      for (int e = 0; e < VE; ++e) { ra[e] = 0u; rb2[e] = 0u; }
    }
    if constexpr (VE == 8) {
      *reinterpret_cast<uint2*>(o1) = make_uint2(pack_codes4(ra[0], ra[1], ra[2], ra[3]), pack_codes4(ra[4], ra[5], ra[6], ra[7]));
      if constexpr (DUAL)
        if (with_gq)
          *reinterpret_cast<uint2*>(o2) = make_uint2(pack_codes4(rb2[0], rb2[1], rb2[2], rb2[3]), pack_codes4(rb2[4], rb2[5], rb2[6], rb2[7]));
    } else {
      *reinterpret_cast<uint32_t*>(o1) = pack_codes4(ra[0], ra[1], ra[2], ra[3]);
      if constexpr (DUAL)
        if (with_gq) *reinterpret_cast<uint32_t*>(o2) = pack_codes4(rb2[0], rb2[1], rb2[2], rb2[3]);
    }
    o1 += o_stride;
    if constexpr (DUAL) o2 += o_stride;
    hw += adv_rem;                      // rpi pixels further: rpi = adv_q * HW + adv_rem
    idx0 += adv_idx;
    if (hw >= HWi) { hw -= HWi; idx0 += wrap; }
  };

  if (ok) {
    uint32_t k[VE];
#pragma unroll
    for (int e = 0; e < VE; ++e) { k[e] = 0u; inv1[e] = real ? ch_inv[c0 + e] : 0.f; }
    const float inv2 = ch_inv[C];
    // density count.  bf16: |g| > sigma in binary32 is |g| > (sigma truncated to bf16) for a bf16 g,
    // two elements per instruction; counts of up to 128 ones are exact in a bf16 accumulator
    uint32_t thr[4] = {0u, 0u, 0u, 0u}, acc2[4] = {0u, 0u, 0u, 0u};
    float sg[VE];
#pragma unroll
    for (int e = 0; e < VE; ++e) sg[e] = real ? ch_sigma[c0 + e] : 0.f;
    if constexpr (kPacked) {
#pragma unroll
      for (int j = 0; j < 4; ++j) thr[j] = (__float_as_uint(sg[2 * j]) >> 16) | (__float_as_uint(sg[2 * j + 1]) & 0xFFFF0000u);
    }
    // packed bf16 bounds below which no clamp of either quantizer can act: 126.6/inv = 0.9969 * scale,
    // rounded toward zero to bf16, the smaller of the channel's and the layer's
    uint32_t cthr[4] = {0u, 0u, 0u, 0u};
    if constexpr (kPacked) {
      const float lim2 = inv2 > 0.f ? __fdiv_rn(126.6f, inv2) : 3.0e38f;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float l0 = fminf(inv1[2 * j] > 0.f ? __fdiv_rn(126.6f, inv1[2 * j]) : 3.0e38f, lim2);
        const float l1 = fminf(inv1[2 * j + 1] > 0.f ? __fdiv_rn(126.6f, inv1[2 * j + 1]) : 3.0e38f, lim2);
        cthr[j] = (__float_as_uint(l0) >> 16) | (__float_as_uint(l1) & 0xFFFF0000u);
      }
    }
    int run = 0;
    auto flush = [&]() {   // move the packed counts into the 32-bit counters
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        k[2 * j < VE ? 2 * j : 0] += (uint32_t)__uint_as_float(acc2[j] << 16);
        k[2 * j + 1 < VE ? 2 * j + 1 : 0] += (uint32_t)__uint_as_float(acc2[j] & 0xFFFF0000u);
        acc2[j] = 0u;
      }
    };
    // the rows of this thread in one contiguous run of `rows` pixel rows starting at `base`
    const uint32_t pstep = (uint32_t)rpi * (uint32_t)G * 16u;
    auto sweep_rows = [&](const uint8_t* base, int rows) {
      if (real) {
        const uint8_t* p = base + ((uint32_t)rl * (uint32_t)G + (uint32_t)col) * 16u;
#pragma unroll 1
        for (int row = rl; row < rows; row += rpi, p += pstep) {
          const uint4 raw = *reinterpret_cast<const uint4*>(p);
          uint32_t over = 0u;     // nonzero if an element is large enough for a clamp to matter
          if constexpr (kPacked) {
            const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const uint32_t mag = w[j] & 0x7FFF7FFFu;
              acc2[j] = bf16x2_add(acc2[j], bf16x2_gt_one(mag, thr[j]));
              over |= bf16x2_gt_one(mag, cthr[j]);
            }
            if (++run == 128) { run = 0; flush(); }
          } else {
            float v[VE];
            unpack_raw(raw, v, (const T*)nullptr);
#pragma unroll
            for (int e = 0; e < VE; ++e) k[e] += (fabsf(v[e]) > sg[e]) ? 1u : 0u;
          }
          quantize_row(raw, true, inv2, over == 0u, std::true_type{});
        }
      } else if (active) {        // zero padding of the code rows
#pragma unroll 1
        for (int row = rl; row < rows; row += rpi) quantize_row(make_uint4(0u, 0u, 0u, 0u), true, 0.f, false, std::false_type{});
      }
    };
    sweep_rows(pieces, rows_res);
    for_each_piece(R, sweep_rows);
    if constexpr (kPacked) flush();
    if (active) {
#pragma unroll
      for (int e = 0; e < VE; ++e) red_cnt[e * kFT + pos] = k[e];
    }
    // the partial maxima are no longer needed: their rows now take the partial counts
    column_reduce_counts(red_cnt, rpi, Gp, VE, C, reinterpret_cast<uint32_t*>(a.ws.pmax) + (size_t)blockIdx.x * C);
  }
  ok = grid_barrier(a.gridbar, 3u * gridDim.x, a.status, &s_abort, &s_ok) && ok;

  // ---------------- classify + clip (Algorithm 1, Eq. 14/15) ---------------------------------------
  // Channel c is classified by one warp of CTA (c mod gridDim.x), which adds the CTAs' partial counts,
  // writes the channel's outputs and flags the channel if its class was mispredicted.
  if (ok) {
    const double thr = (double)a.mp.lambda * (double)a.npix;
    const uint32_t* pcnt = reinterpret_cast<const uint32_t*>(a.ws.pmax);
    const int nblk = gridDim.x;
#pragma unroll 1
    for (int c = blockIdx.x + nblk * warp; c < C; c += nblk * (kFT / 32)) {
      uint32_t cnt = 0u;
#pragma unroll 1
      for (int b0 = lane; b0 < nblk; b0 += 32 * 5) {   // five independent partials per round trip
        uint32_t pc[5];
#pragma unroll
        for (int u = 0; u < 5; ++u) {
          const int b = b0 + 32 * u;
          pc[u] = b < nblk ? __ldcg(pcnt + (size_t)b * C + c) : 0u;
        }
#pragma unroll
        for (int u = 0; u < 5; ++u) cnt += pc[u];
      }
#pragma unroll 1
      for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xFFFFFFFFu, cnt, o);
      if (lane == 0) {
        const float gmax = ch_absmax[c];
        const bool bell = (double)cnt > thr;
        float s = gmax;
        if (!bell) s = __fadd_rn(__fmul_rn(tcoef, a.has_prev ? ch_sprev[c] : gmax), __fmul_rn(a.mp.A, gmax));
        a.s_state[c] = s;
        if (a.cls) a.cls[c] = bell ? 1 : 0;
        if (a.stats_out) a.stats_out[c * 4 + DAI8_STAT_P] = (float)((double)cnt * a.inv_M);
        const bool mis = bell != (ch_pred[c] != 0);
        a.ws.tickets[c] = mis ? 1u : 0u;
        if (mis) *reinterpret_cast<volatile uint32_t*>(a.ws.ticket2) = 1u;
      }
    }
    if (blockIdx.x == 0 && tid == 0) *a.gmax_layer = ch_absmax[C];
  }
  ok = grid_barrier(a.gridbar, 4u * gridDim.x, a.status, &s_abort, &s_ok) && ok;

  // mispredicted channels (rare): their per-channel codes are redone with the right clip value
  bool fix_mine = false;
  if (ok && __ldcg(a.ws.ticket2) != 0u) {
#pragma unroll 1
    for (int c = tid; c < C; c += kFT) {
      if (__ldcg(a.ws.tickets + c) != 0u) {
        ch_pred[c] = 2;
        ch_inv[c] = inv_scale(__ldcg(a.s_state + c));
        s_any_mis = 1u;
      }
    }
    consumer_sync();
    if (real) {
#pragma unroll
      for (int e = 0; e < VE; ++e) fix_mine = fix_mine || ch_pred[c0 + e] == 2;
    }
  }
  const bool fix_pass = ok && s_any_mis != 0u;
  if (tid == 0) s_fix = fix_pass ? 2u : 1u;    // tells the producer whether a third sweep is streamed

  // ---------------- fix-up sweep: per-channel codes of the vector columns with a wrong prediction ----
  if (fix_pass) {
    hw = hw_first; idx0 = idx_first;
    o1 = a.q1 + first * a.Cp + c0;
#pragma unroll
    for (int e = 0; e < VE; ++e) inv1[e] = real ? ch_inv[c0 + e] : 0.f;
    auto fix_rows = [&](const uint8_t* base, int rows) {
      if (!fix_mine) return;
#pragma unroll 1
      for (int row = rl; row < rows; row += rpi) quantize_row(vec_at(base, row), false, 0.f, false, std::true_type{});
    };
    fix_rows(pieces, rows_res);
    for_each_piece(R, fix_rows);
  }

  if (s_abort) {
    // a wait ran out: give copies that may still be in flight time to land before the CTA ends
#pragma unroll 1
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
}

// ------------------------------------------------------------------------------------------------
// Column-owner variant of the fused path, for gradients with many channels and few pixels (the deep
// stages of ResNet-50 / MobileNetV2 at 14x14 and 7x7).  There the pixel-partitioned kernel above is
// bound by its cross-CTA reductions: 148 CTAs each hold a partial for every channel.  Here a CTA owns
// whole vector columns (8 bf16 / 4 fp32 channels) with ALL their pixels, held in shared memory, so
// |g|max, mean, sigma, the density count, the class and the clip value are CTA-local and exact
// before a single code is written: no prediction, no fix-up.  Only the layer-wide |g|max needs the
// grid: one atomic max per CTA and one grid barrier, which the density count overlaps.
// ------------------------------------------------------------------------------------------------
constexpr int kColMaxLocal = 4;      // vector columns per CTA

struct ColArgs {
  int64_t npix, HW;
  double inv_M, inv_denom;
  int C, Cp, G, Gp;
  int cols_per_cta;
  uint32_t* gmax_bits;
  uint32_t* gridbar;
  const float* sigma_override;
  McsDev mp;
  float* s_state;
  int has_prev;
  float* gmax_layer;
  float* stats_out;
  uint8_t* cls;
  uint32_t seed;
  int8_t* q1;
  int8_t* q2;
  unsigned int* status;
};

// Eight bf16 elements (one vector) with 32-bit element indices, none of them large enough for a clamp
// to act: the clamp-free form of the stochastic quantizer with paired additions (see the sweep of
// the pixel-partitioned kernel for the argument).
template <bool DUAL>
__device__ __forceinline__ void quantize_vec8_unclipped(const uint4& raw, const float (&inv1)[8], float inv2, uint32_t idx,
                                                        uint32_t HW, uint32_t key0, uint32_t (&ra)[8], uint32_t (&rb)[8]) {
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
  const uint64_t minus1 = f32x2_pack(0xBF800000u, 0xBF800000u), magic = f32x2_pack(0x4B400000u, 0x4B400000u);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const uint32_t h0 = sr_fold(idx, key0);
    idx += HW;
    const uint32_t h1 = sr_fold(idx, key0);
    idx += HW;
    const float g0 = __uint_as_float(w[j] << 16), g1 = __uint_as_float(w[j] & 0xFFFF0000u);
    const uint64_t v1 = f32x2_pack(__float_as_uint(__fmul_rn(g0, inv1[2 * j])), __float_as_uint(__fmul_rn(g1, inv1[2 * j + 1])));
    const uint64_t u1 = f32x2_add_rn(f32x2_pack(__funnelshift_r(sr_bits0(h0), 0x7Fu, 9), __funnelshift_r(sr_bits0(h1), 0x7Fu, 9)), minus1);
    f32x2_unpack(f32x2_add_rd(f32x2_add_rn(v1, u1), magic), ra[2 * j], ra[2 * j + 1]);
    if (DUAL) {
      const uint64_t u2 = f32x2_add_rn(f32x2_pack(__funnelshift_r(sr_bits1(h0), 0x7Fu, 9),
                                                  __funnelshift_r(sr_bits1(h1), 0x7Fu, 9)), minus1);
      const uint64_t v2 = f32x2_pack(__float_as_uint(__fmul_rn(g0, inv2)), __float_as_uint(__fmul_rn(g1, inv2)));
      f32x2_unpack(f32x2_add_rd(f32x2_add_rn(v2, u2), magic), rb[2 * j], rb[2 * j + 1]);
    }
  }
}

template <typename T, int VE, bool DUAL>
__global__ void __launch_bounds__(kFT, 1)
gvq_columns_kernel(const T* __restrict__ x, const ColArgs a) {
  extern __shared__ __align__(16) uint8_t csmem[];
  __shared__ double red_d[kFT / 32][2 * VE];     // per warp: sum and sum of squares of every channel
  __shared__ float red_f[kFT / 32][VE];          // per warp: |g|max
  __shared__ uint32_t red_u[kFT / 32][VE];       // per warp: density count
  __shared__ float ch_inv[kColMaxLocal][VE], ch_sig[kColMaxLocal][VE];
  __shared__ volatile uint32_t s_abort;
  __shared__ uint32_t s_ok;
  using Idx = uint64_t;
  const int tid = threadIdx.x;
  const int C = a.C, G = a.G;
  const int npix = (int)a.npix;                       // at most a few ten thousand (host check)
  uint4* cols = reinterpret_cast<uint4*>(csmem);      // [local column][pixel]
  if (tid == 0) s_abort = 0u;
  const float tcoef = __fsub_rn(1.0f, __fmul_rn(a.mp.k, a.mp.A));
  const double thr = (double)a.mp.lambda * (double)a.npix;

  // ---- load the columns, statistics, density count, class and clip: all local -------------------
#pragma unroll 1
  for (int lc = 0; lc < a.cols_per_cta; ++lc) {
    const int col = blockIdx.x + lc * gridDim.x;
    if (col >= G) break;                              // padding columns hold no input
    const int c0 = col * VE;
    uint4* mine = cols + (size_t)lc * npix;
    float piv[VE], amax[VE], fs[VE], fss[VE];
    load_vec<T, VE>(x + c0, piv);
#pragma unroll
    for (int e = 0; e < VE; ++e) { amax[e] = 0.f; fs[e] = 0.f; fss[e] = 0.f; }
    double ds[VE], dss[VE];
#pragma unroll
    for (int e = 0; e < VE; ++e) { ds[e] = 0.0; dss[e] = 0.0; }
    int run = 0;
#pragma unroll 4
    for (int p = tid; p < npix; p += kFT) {
      const uint4 raw = *reinterpret_cast<const uint4*>(x + (size_t)p * C + c0);
      mine[p] = raw;
      float v[VE];
      unpack_raw(raw, v, (const T*)nullptr);
#pragma unroll
      for (int e = 0; e < VE; ++e) {
        amax[e] = fmaxf(amax[e], fabsf(v[e]));
        const float d = v[e] - piv[e];
        fs[e] += d;
        fss[e] = fmaf(d, d, fss[e]);
      }
      if (++run == 32) {
        run = 0;
#pragma unroll
        for (int e = 0; e < VE; ++e) { ds[e] += (double)fs[e]; dss[e] += (double)fss[e]; fs[e] = 0.f; fss[e] = 0.f; }
      }
    }
    // all channels of the vector at once: butterflies inside the warps, then thread e adds the sixteen
    // warp results of channel e in warp order (fixed order: deterministic)
#pragma unroll
    for (int e = 0; e < VE; ++e) {
      float m = amax[e];
      double s1 = ds[e] + (double)fs[e], s2 = dss[e] + (double)fss[e];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
        s1 += __shfl_xor_sync(0xFFFFFFFFu, s1, o);
        s2 += __shfl_xor_sync(0xFFFFFFFFu, s2, o);
      }
      if ((tid & 31) == 0) { red_f[tid >> 5][e] = m; red_d[tid >> 5][e] = s1; red_d[tid >> 5][VE + e] = s2; }
    }
    __syncthreads();
    if (tid < VE) {
      const int e = tid, c = c0 + e;
      float mx = red_f[0][e];
      double s1 = red_d[0][e], s2 = red_d[0][VE + e];
#pragma unroll
      for (int w = 1; w < kFT / 32; ++w) { mx = fmaxf(mx, red_f[w][e]); s1 += red_d[w][e]; s2 += red_d[w][VE + e]; }
      const double pivot = (double)to_f32(x[c]);
      const double md = s1 * a.inv_M;
      double var = a.mp.center_mean ? (s2 - s1 * md) : (s2 + 2.0 * pivot * s1 + pivot * pivot * (double)a.npix);
      var = fmax(var, 0.0) * a.inv_denom;
      const float vf = (float)var;
      const float sigma = (vf > 1e-30f || var == 0.0) ? sqrtf(vf) : sigma_wide(var);
      ch_sig[lc][e] = a.sigma_override ? a.sigma_override[c] : sigma;
      ch_inv[lc][e] = mx;                              // |g|max for now, the scale after the count
      if (a.stats_out) {
        a.stats_out[c * 4 + DAI8_STAT_ABSMAX] = mx;
        a.stats_out[c * 4 + DAI8_STAT_MEAN] = (float)(pivot + md);
        a.stats_out[c * 4 + DAI8_STAT_SIGMA] = sigma;
      }
      if (mx > 0.f) atomicMax(a.gmax_bits, __float_as_uint(mx));
    }
    __syncthreads();
  }

  // density count on the resident columns (overlaps the other CTAs' way to the barrier)
#pragma unroll 1
  for (int lc = 0; lc < a.cols_per_cta; ++lc) {
    const int col = blockIdx.x + lc * gridDim.x;
    if (col >= G) break;
    const int c0 = col * VE;
    const uint4* mine = cols + (size_t)lc * npix;
    float sg[VE];
    uint32_t k[VE];
#pragma unroll
    for (int e = 0; e < VE; ++e) { sg[e] = ch_sig[lc][e]; k[e] = 0u; }
#pragma unroll 4
    for (int p = tid; p < npix; p += kFT) {
      float v[VE];
      unpack_raw(mine[p], v, (const T*)nullptr);
#pragma unroll
      for (int e = 0; e < VE; ++e) k[e] += (fabsf(v[e]) > sg[e]) ? 1u : 0u;
    }
#pragma unroll
    for (int e = 0; e < VE; ++e) {
      uint32_t n = k[e];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) n += __shfl_xor_sync(0xFFFFFFFFu, n, o);
      if ((tid & 31) == 0) red_u[tid >> 5][e] = n;
    }
    __syncthreads();
    if (tid < VE) {
      const int e = tid, c = c0 + e;
      uint32_t cnt = 0u;
#pragma unroll
      for (int w = 0; w < kFT / 32; ++w) cnt += red_u[w][e];
      const float gmax = ch_inv[lc][e];
      const bool bell = (double)cnt > thr;
      float s = gmax;
      if (!bell) s = __fadd_rn(__fmul_rn(tcoef, a.has_prev ? a.s_state[c] : gmax), __fmul_rn(a.mp.A, gmax));
      a.s_state[c] = s;
      if (a.cls) a.cls[c] = bell ? 1 : 0;
      if (a.stats_out) a.stats_out[c * 4 + DAI8_STAT_P] = (float)((double)cnt * a.inv_M);
      ch_inv[lc][e] = inv_scale(s);
    }
    __syncthreads();
  }

  // ---- the layer-wide scale needs every CTA's maximum --------------------------------------------
  bool ok = true;
  {
    if (tid == 0) {
      asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(a.gridbar) : "memory");
      uint32_t good = 1u;
      const long long t0 = clock64();
      for (;;) {
        uint32_t seen;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(a.gridbar) : "memory");
        if (seen >= gridDim.x) break;
        if (clock64() - t0 > kWaitTimeoutCycles) {
          atomicExch(a.status, (unsigned int)DAI8_ERR_TIMEOUT);
          good = 0u;
          break;
        }
      }
      s_ok = good;
    }
    __syncthreads();
    ok = s_ok != 0u;
  }
  if (!ok) return;
  const float gmax_l = __uint_as_float(__ldcg(a.gmax_bits));
  const float inv2 = inv_scale(gmax_l);
  if (blockIdx.x == 0 && tid == 0) *a.gmax_layer = gmax_l;

  // ---- codes --------------------------------------------------------------------------------------
  const uint32_t key0 = sr_key(a.seed, 0u);
  const Idx HWi = (Idx)a.HW;
#pragma unroll 1
  for (int lc = 0; lc < a.cols_per_cta; ++lc) {
    const int col = blockIdx.x + lc * gridDim.x;
    if (col >= a.Gp) break;
    const int c0 = col * VE;
    int8_t* o1 = a.q1 + c0;
    int8_t* o2 = DUAL ? a.q2 + c0 : nullptr;
    if (col >= G) {                                   // zero padding of the code rows
      for (int p = tid; p < npix; p += kFT) {
        if (VE == 8) {
          *reinterpret_cast<uint2*>(o1 + (size_t)p * a.Cp) = make_uint2(0u, 0u);
          if (DUAL) *reinterpret_cast<uint2*>(o2 + (size_t)p * a.Cp) = make_uint2(0u, 0u);
        } else {
          *reinterpret_cast<uint32_t*>(o1 + (size_t)p * a.Cp) = 0u;
          if (DUAL) *reinterpret_cast<uint32_t*>(o2 + (size_t)p * a.Cp) = 0u;
        }
      }
      continue;
    }
    const uint4* mine = cols + (size_t)lc * npix;
    float inv1[VE];
#pragma unroll
    for (int e = 0; e < VE; ++e) inv1[e] = ch_inv[lc][e];
    // bf16, fewer than 2^32 elements: packed bounds below which no clamp can act (126.6/inv, the
    // smaller of the channel's and the layer's, rounded toward zero to bf16)
    const bool small_idx = (uint64_t)a.npix * (uint64_t)C < ((uint64_t)1 << 32);
    uint32_t cthr[4] = {0u, 0u, 0u, 0u};
    if (VE == 8) {
      const float lim2 = DUAL ? (inv2 > 0.f ? __fdiv_rn(126.6f, inv2) : 3.0e38f) : 3.0e38f;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float l0 = fminf(inv1[(2 * j) % VE] > 0.f ? __fdiv_rn(126.6f, inv1[(2 * j) % VE]) : 3.0e38f, lim2);
        const float l1 = fminf(inv1[(2 * j + 1) % VE] > 0.f ? __fdiv_rn(126.6f, inv1[(2 * j + 1) % VE]) : 3.0e38f, lim2);
        cthr[j] = (__float_as_uint(l0) >> 16) | (__float_as_uint(l1) & 0xFFFF0000u);
      }
    }
  #pragma unroll 2
    for (int p = tid; p < npix; p += kFT) {
      const uint4 raw = mine[p];
      float v[VE];
      unpack_raw(raw, v, (const T*)nullptr);
      const uint32_t n = (uint32_t)p / (uint32_t)a.HW;
      const uint32_t hw = (uint32_t)p - n * (uint32_t)a.HW;
      Idx idx = ((Idx)n * (Idx)C + (Idx)c0) * HWi + (Idx)hw;      // NCHW index of (n, c0, hw)
      uint32_t ra[VE], rb[VE];
      bool done = false;
      if constexpr (VE == 8) {
        if (small_idx) {
          const uint32_t over = bf16x2_gt_one(raw.x & 0x7FFF7FFFu, cthr[0]) | bf16x2_gt_one(raw.y & 0x7FFF7FFFu, cthr[1]) |
                                bf16x2_gt_one(raw.z & 0x7FFF7FFFu, cthr[2]) | bf16x2_gt_one(raw.w & 0x7FFF7FFFu, cthr[3]);
          if (over == 0u) {
            quantize_vec8_unclipped<DUAL>(raw, inv1, inv2, (uint32_t)idx, (uint32_t)a.HW, key0, ra, rb);
            done = true;
          }
        }
      }
      if (!done) {
#pragma unroll
      for (int e = 0; e < VE; ++e) {
        const uint32_t hi = (uint32_t)(idx >> 32);
        const uint32_t key = hi == 0u ? key0 : sr_key(a.seed, hi);
        const uint32_t f = sr_fold((uint32_t)idx, key), h = sr_bits0(f);
        ra[e] = quant_stochastic_bits(v[e], inv1[e], sr_uniform_fast(h));
        if (DUAL) rb[e] = quant_stochastic_bits(v[e], inv2, sr_uniform_fast(sr_bits1(f)));
        idx += HWi;
      }
      }
      if (VE == 8) {
        *reinterpret_cast<uint2*>(o1 + (size_t)p * a.Cp) = make_uint2(pack_codes4(ra[0], ra[1], ra[2], ra[3]), pack_codes4(ra[4 % VE], ra[5 % VE], ra[6 % VE], ra[7 % VE]));
        if (DUAL) *reinterpret_cast<uint2*>(o2 + (size_t)p * a.Cp) = make_uint2(pack_codes4(rb[0], rb[1], rb[2], rb[3]), pack_codes4(rb[4 % VE], rb[5 % VE], rb[6 % VE], rb[7 % VE]));
      } else {
        *reinterpret_cast<uint32_t*>(o1 + (size_t)p * a.Cp) = pack_codes4(ra[0], ra[1], ra[2], ra[3]);
        if (DUAL) *reinterpret_cast<uint32_t*>(o2 + (size_t)p * a.Cp) = pack_codes4(rb[0], rb[1], rb[2], rb[3]);
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// dai8_quantize_tensor in ONE launch for tensors whose codes have the layout of their values (NHWC
// with C a multiple of 16), layer scale = max|x|, nearest rounding: the forward quantization of the
// activations (Eq. 1, Fig. 2).  The scale needs the whole tensor before the first code can be
// written, so the tensor is swept twice; this kernel makes the second sweep as cheap as the chip
// allows.  A persistent cooperative launch, one CTA per SM, each owning a contiguous range of the
// tensor.  A producer warp streams the range through a ring of 13 KB shared-memory pieces with bulk
// asynchronous copies, one ring slot per consumer warp; sweep 1 takes max|x| (packed bf16
// arithmetic, exact).  After one atomic max
// per CTA and one grid barrier, sweep 2 writes the codes walking the range BACKWARDS: first the
// pieces that are still in shared memory from sweep 1 (no memory traffic at all), then the rest in
// reverse order, so that what it fetches is what sweep 1 touched last and L2 still holds.
//
// With scale = max|x| no clamp of Eq. 1 can change a code: |x * fl(127/s)| <= 127 (1 + 2^-23)^2,
// which rounds to 127 like the clamped value does.  Codes come out of the magic-number addition
// (quant_nearest_bits without the clamps).
// ------------------------------------------------------------------------------------------------
constexpr int kQtMaxSlots = 16;                // one shared-memory piece per consumer warp
constexpr int kQtPieceBytes = 13312;           // 16 pieces fill the shared memory of an SM
constexpr int kQtPieceVecs = kQtPieceBytes / 16;

struct QtArgs {
  const uint8_t* x;      // the tensor as bytes
  int8_t* q;
  float* scale;          // out: max|x|
  uint32_t* ctrl;        // [0] grid-barrier counter, [1] bit pattern of the running maximum; zeroed before the launch
  int64_t nvec;          // 16-byte vectors in the tensor
  int64_t vec_per_cta;
  int slots;             // shared-memory pieces per CTA
  unsigned int* status;
};

template <typename T>
__global__ void __launch_bounds__(kFusedThreads, 1)
quantize_flat_fused_kernel(const QtArgs a) {
  constexpr int VE = 16 / (int)sizeof(T);
  constexpr int NW = kFT / 32;                 // consumer warps
  extern __shared__ __align__(128) uint8_t qsmem[];
  __shared__ uint64_t full_bar[kQtMaxSlots], empty_bar[kQtMaxSlots];
  __shared__ volatile uint32_t s_abort;
  __shared__ uint32_t s_ok;
  __shared__ float s_wmax[NW];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t v0 = (int64_t)blockIdx.x * a.vec_per_cta;
  const int64_t v1 = min(a.nvec, v0 + a.vec_per_cta);
  const int nv = v1 > v0 ? (int)(v1 - v0) : 0;          // vectors of this CTA
  const int K = (nv + kQtPieceVecs - 1) / kQtPieceVecs;  // pieces of this CTA
  const int S = a.slots;
  // Piece u of sweep 1 goes to slot u mod S; afterwards the last min(K, S) pieces are resident.  Step v
  // of sweep 2 handles piece K-1-v in the slot of step v - S (the same slot for v < S: resident).
  // Slot w belongs to consumer warp w, which takes every fill of it in turn: a warp meets the producer
  // once per 13 KB, and it can never run a whole fill ahead of its slot's barrier (a parity wait
  // cannot tell the phase before last from the one awaited).
  auto slot2 = [&](int v) { int r = (K - 1 - (v % S)) % S; return r < 0 ? r + S : r; };
  auto fills1 = [&](int slot) { return slot < K ? (K - slot + S - 1) / S : 0; };   // sweep-1 fills of a slot

  if (tid == 0) {
    s_abort = 0u;
#pragma unroll 1
    for (int s = 0; s < kQtMaxSlots; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp == NW) {
    // ---- producer: every fill of a slot but its first waits for the consumer's hand-back of the fill before
    if (lane == 0 && K > 0) {
      const uint8_t* src = a.x + (size_t)v0 * 16;
      const int total = K + (K > S ? K - S : 0);
#pragma unroll 1
      for (int t = 0; t < total; ++t) {
        int piece, slot, fill;
        if (t < K) { piece = t; slot = t % S; fill = t / S; }
        else { const int v = t - K + S; piece = K - 1 - v; slot = slot2(v); fill = fills1(slot) - 1 + v / S; }
        if (fill > 0 && !mbar_wait(&empty_bar[slot], (uint32_t)(fill - 1) & 1u, &s_abort, a.status)) break;
        const uint32_t bytes = (uint32_t)min(kQtPieceVecs, nv - piece * kQtPieceVecs) * 16u;
        mbar_expect_tx(&full_bar[slot], bytes);
        bulk_load(qsmem + (size_t)slot * kQtPieceBytes, src + (size_t)piece * kQtPieceBytes, bytes, &full_bar[slot]);
      }
    }
    return;
  }

  // ---- sweep 1: max|x| -------------------------------------------------------------------------------
  bool ok = true;
  float m = 0.f;
  uint32_t m2[4] = {0u, 0u, 0u, 0u};
#pragma unroll 1
  for (int u = warp; u < K && ok && warp < S; u += S) {
    const int slot = warp;
    ok = mbar_wait(&full_bar[slot], (uint32_t)(u / S) & 1u, &s_abort, a.status);
    if (!ok) break;
    const uint4* pv = reinterpret_cast<const uint4*>(qsmem + (size_t)slot * kQtPieceBytes);
    const int cnt = min(kQtPieceVecs, nv - u * kQtPieceVecs);
#pragma unroll 4
    for (int i = lane; i < cnt; i += 32) {
      const uint4 r = pv[i];
      if constexpr (VE == 8) {
        m2[0] = bf16x2_max(m2[0], r.x & 0x7FFF7FFFu); m2[1] = bf16x2_max(m2[1], r.y & 0x7FFF7FFFu);
        m2[2] = bf16x2_max(m2[2], r.z & 0x7FFF7FFFu); m2[3] = bf16x2_max(m2[3], r.w & 0x7FFF7FFFu);
      } else {
        m = fmaxf(fmaxf(m, fabsf(__uint_as_float(r.x))), fmaxf(fabsf(__uint_as_float(r.y)),
            fmaxf(fabsf(__uint_as_float(r.z)), fabsf(__uint_as_float(r.w)))));
      }
    }
    if (u + S < K) {            // the slot is filled again in this sweep: hand it back
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty_bar[slot]);
    }
  }
  if constexpr (VE == 8) {
#pragma unroll
    for (int j = 0; j < 4; ++j)
      m = fmaxf(m, fmaxf(__uint_as_float(m2[j] << 16), __uint_as_float(m2[j] & 0xFFFF0000u)));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  if (lane == 0) s_wmax[warp] = m;
  consumer_sync();
  if (tid == 0) {
#pragma unroll 1
    for (int w = 1; w < NW; ++w) m = fmaxf(m, s_wmax[w]);
    if (m > 0.f) atomicMax(a.ctrl + 1, __float_as_uint(m));   // non-negative floats order like their bit patterns
  }
  ok = grid_barrier(a.ctrl, gridDim.x, a.status, &s_abort, &s_ok) && ok;

  // ---- sweep 2: codes, backwards -----------------------------------------------------------------------
  if (ok) {
    const float s = __uint_as_float(__ldcg(a.ctrl + 1));
    if (blockIdx.x == 0 && tid == 0) *a.scale = s;
    const float inv = inv_scale(s);
    int8_t* qbase = a.q + (size_t)v0 * VE;
    int v_first = (K - 1 - warp) % S;        // the first step of sweep 2 that uses this warp's slot
    if (v_first < 0) v_first += S;
#pragma unroll 1
    for (int v = v_first; v < K && ok && warp < S; v += S) {
      const int piece = K - 1 - v, slot = warp;
      ok = mbar_wait(&full_bar[slot], (uint32_t)(fills1(slot) - 1 + v / S) & 1u, &s_abort, a.status);
      if (!ok) break;
      const uint4* pv = reinterpret_cast<const uint4*>(qsmem + (size_t)slot * kQtPieceBytes);
      const int cnt = min(kQtPieceVecs, nv - piece * kQtPieceVecs);
      int8_t* qp = qbase + (size_t)piece * kQtPieceVecs * VE;
#pragma unroll 2
      for (int i = lane; i < cnt; i += 32) {
        const uint4 r = pv[i];
        if constexpr (VE == 8) {
          const uint32_t w[4] = {r.x, r.y, r.z, r.w};
          uint32_t c[8];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            c[2 * j] = __float_as_uint(__fadd_rn(__fmul_rn(__uint_as_float(w[j] << 16), inv), kRoundMagic));
            c[2 * j + 1] = __float_as_uint(__fadd_rn(__fmul_rn(__uint_as_float(w[j] & 0xFFFF0000u), inv), kRoundMagic));
          }
          *reinterpret_cast<uint2*>(qp + (size_t)i * 8) = make_uint2(pack_codes4(c[0], c[1], c[2], c[3]), pack_codes4(c[4], c[5], c[6], c[7]));
        } else {
          const uint32_t c0 = __float_as_uint(__fadd_rn(__fmul_rn(__uint_as_float(r.x), inv), kRoundMagic));
          const uint32_t c1 = __float_as_uint(__fadd_rn(__fmul_rn(__uint_as_float(r.y), inv), kRoundMagic));
          const uint32_t c2 = __float_as_uint(__fadd_rn(__fmul_rn(__uint_as_float(r.z), inv), kRoundMagic));
          const uint32_t c3 = __float_as_uint(__fadd_rn(__fmul_rn(__uint_as_float(r.w), inv), kRoundMagic));
          *reinterpret_cast<uint32_t*>(qp + (size_t)i * 4) = pack_codes4(c0, c1, c2, c3);
        }
      }
      if (v + S < K) {          // another piece is fetched into this slot
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[slot]);
      }
    }
  }
  if (s_abort) {
    // a wait ran out: give copies that may still be in flight time to land before the CTA ends
#pragma unroll 1
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
}

// ------------------------------------------------------------------------------------------------
// Host-side launch helpers
// ------------------------------------------------------------------------------------------------
struct FusedConfig {
  int sms = 0;
  size_t smem_max = 0;
  bool coop = false;
};

// Properties of the current device, looked up once per device.
const FusedConfig& fused_config() {
  static FusedConfig cfgs[64];
  static std::once_flag once[64];
  static const FusedConfig none;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return none;
  std::call_once(once[dev], [dev] {
    int coop = 0, sms = 0, smem = 0;
    cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    cfgs[dev].sms = sms;
    cfgs[dev].smem_max = (size_t)smem;
    cfgs[dev].coop = coop != 0 && sms > 0;
  });
  return cfgs[dev];
}

template <typename T, int VE, bool DUAL, bool IDX32>
dai8_status launch_fused(const T* dY, FusedArgs& a, cudaStream_t st) {
  const FusedConfig& cfg = fused_config();
  const size_t fixed = (fused_red_bytes(VE) + (size_t)a.C * 17 + 8 + 127) / 128 * 128;
  const size_t budget = cfg.smem_max - 1024;   // static shared memory of the kernel
  const int rb = a.C * (int)sizeof(T);
  const int rpi = fused_rows_per_iteration(a.Gp);
  a.rpi = rpi;
  a.adv_q = (int)(rpi / a.HW);
  a.adv_rem = (int)(rpi % a.HW);
  a.rows_per_warp = (a.Gp <= 32 && 32 % a.Gp == 0) ? 32 / a.Gp : 0;   // else rows run across warp boundaries
  int mult = kPieceBytes / (rpi * rb);
  if (mult < 1) mult = 1;
  a.rp = rpi * mult;
  const size_t piece_bytes = (size_t)a.rp * rb;
  int64_t ctas = ceil_div64(a.npix, rpi);
  if (ctas > cfg.sms) ctas = cfg.sms;
  const int64_t chunk = ceil_div64(a.npix, ctas);
  const int64_t pieces = ceil_div64(chunk, a.rp);       // of the largest CTA
  if (budget < fixed + 2 * piece_bytes) return DAI8_ERR_UNSUPPORTED;
  int64_t slots = (int64_t)((budget - fixed) / piece_bytes);
  if (slots > kMaxSlots) slots = kMaxSlots;
  if (slots > pieces) slots = pieces;
  a.slots = (int)slots;
  // 8, 4, 2 or 1 cycling pieces: for tensors far larger than shared memory what stays resident is a few
  // per cent, and the bytes in flight per SM matter more (four 32 KB pieces instead of two: 309 -> 299 us
  // on 822 MB)
  a.ring_log2 = slots >= 10 ? 3 : (slots >= 4 ? 2 : (slots >= 2 ? 1 : 0));
  {
    const double M = (double)a.npix;
    const double denom = a.mp.std_unbiased ? M - 1.0 : M;
    a.inv_M = 1.0 / M;
    a.inv_denom = denom > 0.0 ? 1.0 / denom : 0.0;
    // expected |g|max / sigma of M samples: sqrt(2 ln M) for a Gaussian, ln(M)/sqrt(2) for a Laplace
    // density; the midpoint separates the two channel shapes well for the M of real layers
    const double lnM = std::log(M > 2.0 ? M : 2.0);
    a.pred_ratio = (float)(0.5 * (std::sqrt(2.0 * lnM) + lnM / std::sqrt(2.0)));
  }
  const size_t smem = fixed + (size_t)slots * piece_bytes;
  auto kern = gvq_fused_nhwc_kernel<T, VE, DUAL, IDX32>;
  static std::atomic<int> attr_done[64];
  if (set_max_smem_once(attr_done, kern, (int)(cfg.smem_max - 1024)) != cudaSuccess) return DAI8_ERR_CUDA;
  void* args[] = {(void*)&dY, (void*)&a};
  DAI8_RETURN_IF_CUDA(cudaLaunchCooperativeKernel((void*)kern, dim3((unsigned)ctas), dim3(kFusedThreads), args, smem, st));
  note_launch(1);
  return DAI8_OK;
}

// Column-owner kernel: applicable when all pixels of a CTA's vector columns fit in shared memory.
template <typename T, int VE>
bool columns_plan(int64_t npix, int Gp, int* grid, int* cols_per_cta, size_t* smem) {
  const FusedConfig& cfg = fused_config();
  if (!cfg.coop || npix > 65536) return false;
  int per = (Gp + cfg.sms - 1) / cfg.sms;
  if (per > kColMaxLocal) return false;
  const size_t bytes = (size_t)per * (size_t)npix * 16;
  if (bytes + 8192 > cfg.smem_max) return false;      // static shared memory of the kernel: about 4 KB
  *grid = (Gp + per - 1) / per;
  *cols_per_cta = per;
  *smem = bytes;
  return true;
}

template <typename T, int VE>
dai8_status launch_columns(const T* dY, ColArgs& a, bool dual, int grid, size_t smem, cudaStream_t st) {
  const double M = (double)a.npix;
  const double denom = a.mp.std_unbiased ? M - 1.0 : M;
  a.inv_M = 1.0 / M;
  a.inv_denom = denom > 0.0 ? 1.0 / denom : 0.0;
  void* args[] = {(void*)&dY, (void*)&a};
  static std::atomic<int> attr_done[2][64];
  const int lim = (int)fused_config().smem_max - 8192;
  if (set_max_smem_once(attr_done[0], gvq_columns_kernel<T, VE, true>, lim) != cudaSuccess ||
      set_max_smem_once(attr_done[1], gvq_columns_kernel<T, VE, false>, lim) != cudaSuccess)
    return DAI8_ERR_CUDA;
  if (dual)
    DAI8_RETURN_IF_CUDA(cudaLaunchCooperativeKernel((void*)gvq_columns_kernel<T, VE, true>, dim3((unsigned)grid), dim3(kFT), args, smem, st));
  else
    DAI8_RETURN_IF_CUDA(cudaLaunchCooperativeKernel((void*)gvq_columns_kernel<T, VE, false>, dim3((unsigned)grid), dim3(kFT), args, smem, st));
  note_launch(1);
  return DAI8_OK;
}

template <typename T, int VE>
dai8_status launch_fused_select(const T* dY, FusedArgs& a, bool dual, bool idx32, cudaStream_t st) {
  if (dual) return idx32 ? launch_fused<T, VE, true, true>(dY, a, st) : launch_fused<T, VE, true, false>(dY, a, st);
  return idx32 ? launch_fused<T, VE, false, true>(dY, a, st) : launch_fused<T, VE, false, false>(dY, a, st);
}

struct NhwcGrid {
  dim3 grid;
  int G;   // vectors per pixel that are processed
};

// Pixel blocks x column blocks for the NHWC mapping: at most kMaxPixelBlocks blocks in total and
// at least ~8 iterations of work per block.
NhwcGrid nhwc_grid(int64_t npix, int vectors_per_pixel) {
  NhwcGrid g;
  g.G = vectors_per_pixel;
  const int colblocks = (vectors_per_pixel + kThreads - 1) / kThreads;
  const int gcols = vectors_per_pixel < kThreads ? vectors_per_pixel : kThreads;
  const int rpi = kThreads / gcols;
  int64_t pb = ceil_div64(npix, (int64_t)rpi * 8);
  int64_t cap = kMaxPixelBlocks / colblocks;
  if (cap < 1) cap = 1;
  if (pb > cap) pb = cap;
  if (pb < 1) pb = 1;
  g.grid = dim3((unsigned)pb, (unsigned)colblocks, 1);
  return g;
}

int nchw_slices(int N, int C) {
  int ns = (kMaxPixelBlocks + C - 1) / C;
  if (ns > N) ns = N;
  if (ns > kMaxPixelBlocks) ns = kMaxPixelBlocks;
  if (ns < 1) ns = 1;
  return ns;
}

template <typename T>
constexpr int vec_elems() { return 16 / (int)sizeof(T); }

McsDev make_mcs(const dai8_mcs_params& p) {
  McsDev mp{p.lambda, p.k, p.A, p.std_unbiased, p.center_mean, p.mode};
  return mp;
}

template <typename T>
dai8_status quantize_grad_typed(const T* dY, dai8_layout layout, int N, int C, int H, int W,
                                const McsDev& mp_in, float* s_state, int has_prev, float* gmax_layer,
                                float* stats, uint8_t* cls, int8_t* vq, int8_t* gq, uint32_t seed,
                                const float* sigma_override, const GvqWs& ws, cudaStream_t st) {
  const int64_t HW = (int64_t)H * W;
  const int64_t npix = (int64_t)N * HW;
  const int Cp = round_up(C, 16);
  constexpr int VEfull = vec_elems<T>();
  McsDev mp = mp_in;
  // The ablation modes of Sec. 4.1.  Per-channel |g|max without the discriminator is the full method
  // with a threshold no density can fall below; the two layer-wide modes (one clip value for all
  // channels) take the three-launch path, whose last count block solves for the layer.
  if (mp.mode == DAI8_GRAD_GVQ_MAX) mp.lambda = -1.0f;
  const bool layer_wide = mp.mode == DAI8_GRAD_GQ || mp.mode == DAI8_GRAD_LAYER_MCS;
  if (mp.mode == DAI8_GRAD_LAYER_MCS) sigma_override = nullptr;   // the layer's own sigma is the method here
  const float* sigma = sigma_override ? sigma_override : ws.sigma;
  if (!layer_wide && layout == DAI8_NHWC && C % VEfull == 0) {
    // many channels, few pixels: whole vector columns per CTA (no cross-CTA reductions)
    int grid = 0, per = 0;
    size_t smem = 0;
    const int Gp = Cp / VEfull;
    const bool fits = columns_plan<T, VEfull>(npix, Gp, &grid, &per, &smem);
    // Fits to measured times (microseconds, B200): the column kernel costs a fixed part plus its
    // longest CTA's rows; the pixel-partitioned kernel a larger fixed part (four barriers), its
    // cross-CTA reductions (per channel) and the elements.
    const double t_columns = 9.0 + 3.4e-3 * (double)npix * per;
    const double t_pixels = 18.0 + 0.019 * C + (double)npix * C / 1.2e6;
    const bool wanted = t_columns < t_pixels;
    if (fits && wanted) {
      ColArgs a;
      a.npix = npix; a.HW = HW; a.inv_M = 0.0; a.inv_denom = 0.0; a.C = C; a.Cp = Cp; a.G = C / VEfull; a.Gp = Gp;
      a.cols_per_cta = per; a.gmax_bits = ws.gmax_bits; a.gridbar = ws.gridbar; a.sigma_override = sigma_override;
      a.mp = mp; a.s_state = s_state; a.has_prev = has_prev; a.gmax_layer = gmax_layer; a.stats_out = stats;
      a.cls = cls; a.seed = seed; a.q1 = vq; a.q2 = gq; a.status = device_status_address();
      if (!a.status) return DAI8_ERR_CUDA;
      note_kernel("gvq_columns_kernel");
      log_choice("quantize_grad: gvq_columns_kernel, %d CTAs x %d vector columns, %lld pixels", grid, per, (long long)npix);
      return launch_columns<T, VEfull>(dY, a, gq != nullptr, grid, smem, st);
    }
  }
  if (!layer_wide && layout == DAI8_NHWC && fused_config().coop && C <= kFusedMaxC && C % VEfull == 0) {
    FusedArgs a;
    a.npix = npix; a.HW = HW; a.C = C; a.Cp = Cp; a.G = C / VEfull; a.Gp = Cp / VEfull;
    a.rp = 0; a.adv_q = 0; a.adv_rem = 0; a.slots = 0; a.ring_log2 = 0; a.rows_per_warp = 0; a.rpi = 0; a.inv_M = 0.0; a.inv_denom = 0.0; a.pred_ratio = 0.f;
    a.ws = ws; a.gridbar = ws.gridbar; a.sigma_override = sigma_override; a.mp = mp;
    a.s_state = s_state; a.has_prev = has_prev; a.gmax_layer = gmax_layer; a.stats_out = stats;
    a.cls = cls; a.seed = seed; a.q1 = vq; a.q2 = gq; a.status = device_status_address();
    if (!a.status) return DAI8_ERR_CUDA;
    const bool idx32 = npix * C < ((int64_t)1 << 32);   // NCHW element indices fit 32 bits
    note_kernel("gvq_fused_nhwc_kernel");
    log_choice("quantize_grad: gvq_fused_nhwc_kernel, C=%d, %lld pixels", C, (long long)npix);
    return launch_fused_select<T, VEfull>(dY, a, gq != nullptr, idx32, st);
  }
  if (layout == DAI8_NHWC) {
    if (C % VEfull == 0) {
      const NhwcGrid g = nhwc_grid(npix, C / VEfull);
      stats_nhwc_kernel<T, VEfull><<<g.grid, kThreads, 0, st>>>(dY, npix, C, g.G, ws, mp, stats);
      if (mp.mode == DAI8_GRAD_LAYER_MCS) layer_sigma_kernel<<<1, kThreads, 0, st>>>(ws, C, npix, mp, stats);
      count_nhwc_kernel<T, VEfull><<<g.grid, kThreads, 0, st>>>(dY, npix, C, g.G, ws, sigma, mp, s_state,
                                                                has_prev, gmax_layer, stats, cls);
      const NhwcGrid gq_ = nhwc_grid(npix, Cp / VEfull);
      if (layer_wide && gq)
        quantize_nhwc_kernel<T, VEfull, false, true, true><<<gq_.grid, kThreads, 0, st>>>(
            dY, npix, HW, C, Cp, gq_.G, ws.layer_scale, gmax_layer, seed, vq, gq);
      else if (layer_wide)
        quantize_nhwc_kernel<T, VEfull, false, true, false><<<gq_.grid, kThreads, 0, st>>>(
            dY, npix, HW, C, Cp, gq_.G, ws.layer_scale, gmax_layer, seed, vq, nullptr);
      else if (gq)
        quantize_nhwc_kernel<T, VEfull, true, true, true><<<gq_.grid, kThreads, 0, st>>>(
            dY, npix, HW, C, Cp, gq_.G, s_state, gmax_layer, seed, vq, gq);
      else
        quantize_nhwc_kernel<T, VEfull, true, true, false><<<gq_.grid, kThreads, 0, st>>>(
            dY, npix, HW, C, Cp, gq_.G, s_state, gmax_layer, seed, vq, nullptr);
    } else {
      const NhwcGrid g = nhwc_grid(npix, C);
      stats_nhwc_kernel<T, 1><<<g.grid, kThreads, 0, st>>>(dY, npix, C, g.G, ws, mp, stats);
      if (mp.mode == DAI8_GRAD_LAYER_MCS) layer_sigma_kernel<<<1, kThreads, 0, st>>>(ws, C, npix, mp, stats);
      count_nhwc_kernel<T, 1><<<g.grid, kThreads, 0, st>>>(dY, npix, C, g.G, ws, sigma, mp, s_state,
                                                           has_prev, gmax_layer, stats, cls);
      const NhwcGrid gq_ = nhwc_grid(npix, Cp);
      if (layer_wide && gq)
        quantize_nhwc_kernel<T, 1, false, true, true><<<gq_.grid, kThreads, 0, st>>>(
            dY, npix, HW, C, Cp, gq_.G, ws.layer_scale, gmax_layer, seed, vq, gq);
      else if (layer_wide)
        quantize_nhwc_kernel<T, 1, false, true, false><<<gq_.grid, kThreads, 0, st>>>(
            dY, npix, HW, C, Cp, gq_.G, ws.layer_scale, gmax_layer, seed, vq, nullptr);
      else if (gq)
        quantize_nhwc_kernel<T, 1, true, true, true><<<gq_.grid, kThreads, 0, st>>>(
            dY, npix, HW, C, Cp, gq_.G, s_state, gmax_layer, seed, vq, gq);
      else
        quantize_nhwc_kernel<T, 1, true, true, false><<<gq_.grid, kThreads, 0, st>>>(
            dY, npix, HW, C, Cp, gq_.G, s_state, gmax_layer, seed, vq, nullptr);
    }
  } else {
    const dim3 grid((unsigned)C, (unsigned)nchw_slices(N, C), 1);
    stats_nchw_kernel<T><<<grid, kThreads, 0, st>>>(dY, N, C, HW, ws, mp, stats);
    if (mp.mode == DAI8_GRAD_LAYER_MCS) layer_sigma_kernel<<<1, kThreads, 0, st>>>(ws, C, npix, mp, stats);
    count_nchw_kernel<T><<<grid, kThreads, 0, st>>>(dY, N, C, HW, ws, sigma, mp, s_state, has_prev,
                                                    gmax_layer, stats, cls);
    const dim3 qgrid((unsigned)ceil_div64(HW, kTileHW), (unsigned)((Cp + kTileC - 1) / kTileC), (unsigned)N);
    if (layer_wide && gq)
      quantize_nchw_kernel<T, false, true, true><<<qgrid, kThreads, 0, st>>>(dY, C, Cp, HW, ws.layer_scale,
                                                                             gmax_layer, seed, vq, gq);
    else if (layer_wide)
      quantize_nchw_kernel<T, false, true, false><<<qgrid, kThreads, 0, st>>>(dY, C, Cp, HW, ws.layer_scale,
                                                                              gmax_layer, seed, vq, nullptr);
    else if (gq)
      quantize_nchw_kernel<T, true, true, true><<<qgrid, kThreads, 0, st>>>(dY, C, Cp, HW, s_state,
                                                                            gmax_layer, seed, vq, gq);
    else
      quantize_nchw_kernel<T, true, true, false><<<qgrid, kThreads, 0, st>>>(dY, C, Cp, HW, s_state,
                                                                             gmax_layer, seed, vq, nullptr);
  }
  note_kernel("stats / count / quantize kernels (three launches)");
  log_choice("quantize_grad: three launches (statistics, count, codes), mode %d", mp.mode);
  note_launch(3);
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}

// Small tensors (weights): a single launch instead of memset + reduction + quantization.  Every CTA
// finds max|x| of the whole tensor for itself (it is small and sits in L2), so no CTA waits for
// another, and writes its share of the codes.
constexpr int kSmallThreads = 1024;
constexpr int64_t kSmallTensorElems = 131072;

template <typename T, bool NHWC_IN>
__global__ void __launch_bounds__(kSmallThreads)
quantize_small_kernel(const T* __restrict__ x, int N, int C, int HW, int Cp, int absmax_mode, int stochastic,
                      uint32_t seed, float* __restrict__ scale, int8_t* __restrict__ q) {
  grid_dependency_release();
  grid_dependency_wait();
  __shared__ float s_part[kSmallThreads / 32];
  __shared__ float s_scale;
  const int tid = threadIdx.x;
  const int total = N * C * HW;
  if (absmax_mode) {
    float m = 0.f;
    constexpr int VE = 16 / (int)sizeof(T);          // 16-byte loads, several in flight per thread
    const int nvec = total / VE;
#pragma unroll 8
    for (int i = tid; i < nvec; i += kSmallThreads) {
      float v[VE];
      load_vec<T, VE>(x + (size_t)i * VE, v);
#pragma unroll
      for (int e = 0; e < VE; ++e) m = fmaxf(m, fabsf(v[e]));
    }
    for (int i = nvec * VE + tid; i < total; i += kSmallThreads) m = fmaxf(m, fabsf(to_f32(x[i])));
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    if ((tid & 31) == 0) s_part[tid >> 5] = m;
    __syncthreads();
    if (tid < 32) {
      m = s_part[tid];
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
      if (tid == 0) { s_scale = m; if (blockIdx.x == 0) *scale = m; }
    }
  } else if (tid == 0) {
    s_scale = *scale;
  }
  __syncthreads();
  const float inv = inv_scale(s_scale);
  const uint32_t key0 = sr_key(seed, 0u);
  const int codes = N * HW * Cp;
  for (int o = blockIdx.x * kSmallThreads + tid; o < codes; o += gridDim.x * kSmallThreads) {   // o = (n*HW + hw)*Cp + c
    const int c = o % Cp;
    const int pix = o / Cp;
    int code = 0;
    if (c < C) {
      const int n = pix / HW, hw = pix - n * HW;
      const int idx = (n * C + c) * HW + hw;               // NCHW index: the generator's counter
      const float v = to_f32(x[NHWC_IN ? pix * C + c : idx]);
      code = stochastic ? quant_stochastic(v, inv, sr_uniform(sr_bits0(sr_fold((uint32_t)idx, key0))))
                        : quant_nearest(v, inv);
    }
    q[o] = (int8_t)code;
  }
}

// ------------------------------------------------------------------------------------------------
// Weights (an NCHW tensor of N filters with few positions each) in ONE cooperative launch.  A CTA
// copies a contiguous run of whole filters into shared memory while taking their max|x|, the CTAs
// combine the maxima through one atomic word and meet at a grid barrier, and each CTA then writes
// the codes of its filters, transposed to [n][hw][Cp], from shared memory: the tensor is read once,
// and no thread stores single bytes.
// ------------------------------------------------------------------------------------------------
struct RowsArgs {
  const void* x;
  int8_t* q;
  float* scale;          // out: max|x|
  uint32_t* ctrl;        // [0] grid-barrier counter, [1] bit pattern of the running maximum; zeroed before the launch
  int N, C, Cp, HW;
  int rows_per_cta;
  unsigned int* status;
};

constexpr int kRowsThreads = 1024;

template <typename T>
__global__ void __launch_bounds__(kRowsThreads)
quantize_rows_fused_kernel(const RowsArgs a) {
  extern __shared__ __align__(16) uint8_t rows_raw[];     // [rows of this CTA][C][HW] as in global memory
  __shared__ float s_part[kRowsThreads / 32];
  __shared__ uint32_t s_ok;
  const int tid = threadIdx.x;
  const int per_n = a.C * a.HW;
  const int n0 = blockIdx.x * a.rows_per_cta;
  const int rows = min(a.rows_per_cta, a.N - n0);
  const int elems = rows * per_n;
  const T* src = static_cast<const T*>(a.x) + (size_t)n0 * per_n;
  T* raw = reinterpret_cast<T*>(rows_raw);
  constexpr int VE = 16 / (int)sizeof(T);
  float m = 0.f;
  // the CTA's filters are one contiguous range; 16-byte copies when it starts on a 16-byte boundary
  const bool vec_ok = (((size_t)n0 * per_n * sizeof(T)) & 15) == 0;
  const int nvec = vec_ok ? elems / VE : 0;
#pragma unroll 4
  for (int i = tid; i < nvec; i += kRowsThreads) {
    const uint4 r = *reinterpret_cast<const uint4*>(src + (size_t)i * VE);
    *reinterpret_cast<uint4*>(raw + (size_t)i * VE) = r;
    float v[VE];
    unpack_raw(r, v, (const T*)nullptr);
#pragma unroll
    for (int e = 0; e < VE; ++e) m = fmaxf(m, fabsf(v[e]));
  }
  for (int i = nvec * VE + tid; i < elems; i += kRowsThreads) {
    const T t = src[i];
    raw[i] = t;
    m = fmaxf(m, fabsf(to_f32(t)));
  }
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  if ((tid & 31) == 0) s_part[tid >> 5] = m;
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < kRowsThreads / 32; ++w) m = fmaxf(m, s_part[w]);
    if (m > 0.f) atomicMax(a.ctrl + 1, __float_as_uint(m));    // non-negative floats order like their bits
    // grid barrier (bounded): release this CTA's maximum, acquire everybody's
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(a.ctrl) : "memory");
    uint32_t ok = 1u;
    const long long t0 = clock64();
    for (;;) {
      uint32_t seen;
      asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(a.ctrl) : "memory");
      if (seen >= gridDim.x) break;
      if (clock64() - t0 > kWaitTimeoutCycles) {
        atomicExch(a.status, (unsigned int)DAI8_ERR_TIMEOUT);
        ok = 0u;
        break;
      }
    }
    s_ok = ok;
    s_part[0] = __uint_as_float(__ldcg(a.ctrl + 1));
  }
  __syncthreads();
  if (!s_ok) return;
  const float smax = s_part[0];
  if (blockIdx.x == 0 && tid == 0) *a.scale = smax;
  const float inv = inv_scale(smax);
  // a warp takes one (filter, position) at a time, a lane four consecutive channels of it: 4-byte
  // stores, 128 contiguous bytes per warp
  const int cw = a.Cp >> 2;
  const int lane = tid & 31;
  uint32_t* dst = reinterpret_cast<uint32_t*>(a.q + (size_t)n0 * a.HW * a.Cp);
#pragma unroll 1
  for (int pix = tid >> 5; pix < rows * a.HW; pix += kRowsThreads / 32) {
    const int row = pix / a.HW, hw = pix - row * a.HW;
    const T* rbase = raw + (size_t)row * per_n + hw;
#pragma unroll 2
    for (int w = lane; w < cw; w += 32) {
      const int c = w << 2;
      const T* r = rbase + (size_t)c * a.HW;
      uint32_t b[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = c + j < a.C ? quant_nearest_bits(to_f32(r[j * a.HW]), inv) : 0u;
      dst[(size_t)pix * cw + w] = pack_codes4(b[0], b[1], b[2], b[3]);
    }
  }
}

template <typename T>
bool rows_fused_applicable(int N, int C, int HW, size_t* smem_bytes, int* rows_per_cta) {
  const FusedConfig& cfg = fused_config();
  if (!cfg.coop) return false;
  const size_t row_bytes = (size_t)C * HW * sizeof(T);
  int64_t ctas = N < cfg.sms ? N : cfg.sms;
  const int64_t rpc = ceil_div64(N, ctas);
  const size_t smem = (rpc * row_bytes + 15) / 16 * 16;
  if (smem + 1024 > cfg.smem_max) return false;
  *smem_bytes = smem;
  *rows_per_cta = (int)rpc;
  return true;
}

template <typename T>
dai8_status launch_quantize_rows_fused(const T* x, int N, int C, int Cp, int HW, size_t smem, int rows_per_cta,
                                       float* scale, int8_t* q, void* ws, cudaStream_t st) {
  RowsArgs a;
  a.x = x; a.q = q; a.scale = scale; a.ctrl = static_cast<uint32_t*>(ws);
  a.N = N; a.C = C; a.Cp = Cp; a.HW = HW; a.rows_per_cta = rows_per_cta;
  a.status = device_status_address();
  if (!a.status) return DAI8_ERR_CUDA;
  auto kern = quantize_rows_fused_kernel<T>;
  static std::atomic<int> attr_done[64];
  if (set_max_smem_once(attr_done, kern, fused_config().smem_max - 1024) != cudaSuccess) return DAI8_ERR_CUDA;
  DAI8_RETURN_IF_CUDA(cudaMemsetAsync(ws, 0, 16, st));
  const int ctas = (N + rows_per_cta - 1) / rows_per_cta;
  void* args[] = {(void*)&a};
  DAI8_RETURN_IF_CUDA(cudaLaunchCooperativeKernel((void*)kern, dim3((unsigned)ctas), dim3(kRowsThreads), args, smem, st));
  note_launch(1);
  note_kernel("quantize_rows_fused_kernel");
  log_choice("quantize_tensor: quantize_rows_fused_kernel, %d filters of %d x %d, %d CTAs", N, C, HW, ctas);
  return DAI8_OK;
}

constexpr size_t kQuantizeTensorWsBytes = 256;

// One cooperative launch: layer scale and codes of a tensor whose codes have the layout of its values.
template <typename T>
dai8_status launch_quantize_flat_fused(const T* x, int64_t nvec, float* scale, int8_t* q, void* ws, cudaStream_t st) {
  const FusedConfig& cfg = fused_config();
  QtArgs a;
  a.x = reinterpret_cast<const uint8_t*>(x); a.q = q; a.scale = scale; a.ctrl = static_cast<uint32_t*>(ws);
  a.nvec = nvec;
  int64_t ctas = ceil_div64(nvec, kQtPieceVecs);
  if (ctas > cfg.sms) ctas = cfg.sms;
  a.vec_per_cta = ceil_div64(nvec, ctas);
  ctas = ceil_div64(nvec, a.vec_per_cta);                 // no CTA without work
  int64_t slots = ceil_div64(a.vec_per_cta, kQtPieceVecs);
  if (slots > kQtMaxSlots) slots = kQtMaxSlots;
  a.slots = (int)slots;
  a.status = device_status_address();
  if (!a.status) return DAI8_ERR_CUDA;
  auto kern = quantize_flat_fused_kernel<T>;
  static std::atomic<int> attr_done[64];
  if (set_max_smem_once(attr_done, kern, kQtMaxSlots * kQtPieceBytes) != cudaSuccess) return DAI8_ERR_CUDA;
  DAI8_RETURN_IF_CUDA(cudaMemsetAsync(ws, 0, 16, st));
  void* args[] = {(void*)&a};
  DAI8_RETURN_IF_CUDA(cudaLaunchCooperativeKernel((void*)kern, dim3((unsigned)ctas), dim3(kFusedThreads), args,
                                                  (size_t)slots * kQtPieceBytes, st));
  note_launch(1);
  return DAI8_OK;
}

template <typename T>
dai8_status quantize_tensor_typed(const T* x, dai8_layout layout, int N, int C, int H, int W,
                                  dai8_scale_mode mode, float* scale, dai8_round round,
                                  uint32_t seed, int8_t* q, void* ws, cudaStream_t st) {
  const int64_t HW = (int64_t)H * W;
  const int64_t npix = (int64_t)N * HW;
  const int64_t total = npix * C;
  const int Cp = round_up(C, 16);
  constexpr int VEfull = vec_elems<T>();
  if (ws && mode == DAI8_SCALE_ABSMAX && round == DAI8_ROUND_NEAREST_EVEN && layout == DAI8_NHWC && C == Cp &&
      npix * Cp > kSmallTensorElems && fused_config().coop &&
      // measured: the one-launch kernel wins only while the whole tensor stays in shared memory between
      // its sweeps (one read from DRAM instead of two); beyond that the two plain kernels stream faster
      total / VEfull <= (int64_t)fused_config().sms * kQtMaxSlots * kQtPieceVecs &&
      fused_config().smem_max >= (size_t)kQtMaxSlots * kQtPieceBytes + 2048)
  {
    note_kernel("quantize_flat_fused_kernel");
    return launch_quantize_flat_fused<T>(x, total / VEfull, scale, q, ws, st);
  }
  if (ws && mode == DAI8_SCALE_ABSMAX && round == DAI8_ROUND_NEAREST_EVEN && layout == DAI8_NCHW &&
      npix * Cp > kSmallTensorElems && HW <= 64) {
    size_t smem = 0;
    int rpc = 0;
    if (rows_fused_applicable<T>(N, C, (int)HW, &smem, &rpc))
      return launch_quantize_rows_fused<T>(x, N, C, Cp, (int)HW, smem, rpc, scale, q, ws, st);
  }
  if (npix * Cp <= kSmallTensorElems) {
    const int am = mode == DAI8_SCALE_ABSMAX ? 1 : 0, sr = round == DAI8_ROUND_STOCHASTIC ? 1 : 0;
    int small_ctas = (int)ceil_div64(npix * Cp, 4 * kSmallThreads);
    if (small_ctas > 32) small_ctas = 32;
    if (layout == DAI8_NHWC)
      DAI8_RETURN_IF_CUDA(launch_dependent(quantize_small_kernel<T, true>, dim3((unsigned)small_ctas), dim3(kSmallThreads), 0, st, x, N, C, (int)HW, Cp, am, sr, seed, scale, q));
    else
      DAI8_RETURN_IF_CUDA(launch_dependent(quantize_small_kernel<T, false>, dim3((unsigned)small_ctas), dim3(kSmallThreads), 0, st, x, N, C, (int)HW, Cp, am, sr, seed, scale, q));
    note_launch(1);
    note_kernel("quantize_small_kernel");
    DAI8_RETURN_IF_CUDA(cudaGetLastError());
    return DAI8_OK;
  }
  note_kernel(layout == DAI8_NHWC ? "absmax_kernel + quantize_flat_nearest_kernel / quantize_nhwc_kernel"
                                  : "absmax_kernel + quantize_nchw_kernel");
  if (mode == DAI8_SCALE_ABSMAX) {
    DAI8_RETURN_IF_CUDA(cudaMemsetAsync(scale, 0, sizeof(float), st));
    uint32_t* bits = reinterpret_cast<uint32_t*>(scale);
    if (total % VEfull == 0) {
      const int64_t nvec = total / VEfull;
      const int blocks = (int)(ceil_div64(nvec, kThreads * 4) < kMaxPixelBlocks ? ceil_div64(nvec, kThreads * 4) : kMaxPixelBlocks);
      absmax_kernel<T, VEfull><<<blocks, kThreads, 0, st>>>(x, nvec, bits);
    } else {
      const int blocks = (int)(ceil_div64(total, kThreads * 4) < kMaxPixelBlocks ? ceil_div64(total, kThreads * 4) : kMaxPixelBlocks);
      absmax_kernel<T, 1><<<blocks, kThreads, 0, st>>>(x, total, bits);
    }
    note_launch(1);
  }
  const bool stoch = round == DAI8_ROUND_STOCHASTIC;
  if (layout == DAI8_NHWC && !stoch && C == Cp) {
    const int64_t nvec = total / VEfull;      // C is a multiple of 16
    const int blocks = (int)(ceil_div64(nvec, kThreads * 4) < 2 * kMaxPixelBlocks ? ceil_div64(nvec, kThreads * 4) : 2 * kMaxPixelBlocks);
    DAI8_RETURN_IF_CUDA(launch_dependent(quantize_flat_nearest_kernel<T, VEfull>, dim3((unsigned)blocks), dim3(kThreads), 0, st, x, nvec, scale, q));
  } else if (layout == DAI8_NHWC && Cp == 16 && C < 16) {
    const int blocks = (int)(ceil_div64(npix, kThreads) < 8 * kMaxPixelBlocks ? ceil_div64(npix, kThreads) : 8 * kMaxPixelBlocks);
    if (stoch)
      quantize_nhwc_c16_kernel<T, true><<<blocks, kThreads, 0, st>>>(x, npix, HW, C, scale, seed, q);
    else
      quantize_nhwc_c16_kernel<T, false><<<blocks, kThreads, 0, st>>>(x, npix, HW, C, scale, seed, q);
  } else if (layout == DAI8_NHWC) {
    if (C % VEfull == 0) {
      const NhwcGrid g = nhwc_grid(npix, Cp / VEfull);
      if (stoch)
        quantize_nhwc_kernel<T, VEfull, false, true, false><<<g.grid, kThreads, 0, st>>>(x, npix, HW, C, Cp, g.G, scale, nullptr, seed, q, nullptr);
      else
        quantize_nhwc_kernel<T, VEfull, false, false, false><<<g.grid, kThreads, 0, st>>>(x, npix, HW, C, Cp, g.G, scale, nullptr, seed, q, nullptr);
    } else {
      const NhwcGrid g = nhwc_grid(npix, Cp);
      if (stoch)
        quantize_nhwc_kernel<T, 1, false, true, false><<<g.grid, kThreads, 0, st>>>(x, npix, HW, C, Cp, g.G, scale, nullptr, seed, q, nullptr);
      else
        quantize_nhwc_kernel<T, 1, false, false, false><<<g.grid, kThreads, 0, st>>>(x, npix, HW, C, Cp, g.G, scale, nullptr, seed, q, nullptr);
    }
  } else if (HW <= 32 && HW * Cp <= 40 * 1024) {
    // weights: few positions per row
    int blocks = N < 4 * fused_config().sms ? N : 4 * fused_config().sms;
    if (blocks < 1) blocks = 1;
    const size_t smem = (size_t)HW * Cp;
    if (stoch)
      DAI8_RETURN_IF_CUDA(launch_dependent(quantize_nchw_rows_kernel<T, true>, dim3((unsigned)blocks), dim3(kThreads), smem, st, x, N, C, Cp, (int)HW, (const float*)scale, seed, q));
    else
      DAI8_RETURN_IF_CUDA(launch_dependent(quantize_nchw_rows_kernel<T, false>, dim3((unsigned)blocks), dim3(kThreads), smem, st, x, N, C, Cp, (int)HW, (const float*)scale, seed, q));
  } else {
    const dim3 qgrid((unsigned)ceil_div64(HW, kTileHW), (unsigned)((Cp + kTileC - 1) / kTileC), (unsigned)N);
    if (stoch)
      quantize_nchw_kernel<T, false, true, false><<<qgrid, kThreads, 0, st>>>(x, C, Cp, HW, scale, nullptr, seed, q, nullptr);
    else
      quantize_nchw_kernel<T, false, false, false><<<qgrid, kThreads, 0, st>>>(x, C, Cp, HW, scale, nullptr, seed, q, nullptr);
  }
  note_launch(1);
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}

bool bad_dims(int N, int C, int H, int W) {
  return N <= 0 || C <= 0 || H <= 0 || W <= 0 || N > 65535;
}

}  // namespace
}  // namespace dai8

using namespace dai8;

extern "C" size_t dai8_quantize_grad_workspace_bytes(int C) { return C > 0 ? ws_bytes_for(C) : 0; }

extern "C" dai8_status dai8_quantize_grad(const void* dY, dai8_dtype dtype, dai8_layout layout, int N,
                                          int C, int H, int W, const dai8_mcs_params* params,
                                          float* s_state, int has_prev, float* gmax_layer,
                                          float* stats, uint8_t* cls, int8_t* vq, int8_t* gq,
                                          uint32_t seed, const float* sigma_override, void* ws,
                                          size_t ws_bytes, void* stream) {
  if (!dY || !s_state || !gmax_layer || !vq || !ws) return DAI8_ERR_INVALID_ARG;
  if (bad_dims(N, C, H, W)) return DAI8_ERR_INVALID_ARG;
  if (dtype != DAI8_F32 && dtype != DAI8_BF16) return DAI8_ERR_INVALID_ARG;
  if (layout != DAI8_NCHW && layout != DAI8_NHWC) return DAI8_ERR_INVALID_ARG;
  if (!aligned16(dY) || !aligned16(vq) || (gq && !aligned16(gq)) || !aligned16(ws)) return DAI8_ERR_INVALID_ARG;
  if ((int64_t)N * H * W >= (int64_t)1 << 32) return DAI8_ERR_UNSUPPORTED;  // counts are 32-bit
  if (ws_bytes < ws_bytes_for(C)) return DAI8_ERR_WORKSPACE;
  dai8_status a = check_device_arch();
  if (a != DAI8_OK) return a;
  dai8_mcs_params p;
  if (params) p = *params; else dai8_mcs_defaults(&p);
  if (p.mode < DAI8_GRAD_FULL || p.mode > DAI8_GRAD_LAYER_MCS) return DAI8_ERR_INVALID_ARG;
  McsDev mp = make_mcs(p);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  GvqWs w = carve(ws, C);
  DAI8_RETURN_IF_CUDA(cudaMemsetAsync(w.tickets, 0, control_words(C) * 4, st));
  if (dtype == DAI8_F32)
    return quantize_grad_typed<float>(static_cast<const float*>(dY), layout, N, C, H, W, mp, s_state,
                                      has_prev, gmax_layer, stats, cls, vq, gq, seed, sigma_override, w, st);
  return quantize_grad_typed<bf16_t>(static_cast<const bf16_t*>(dY), layout, N, C, H, W, mp, s_state,
                                     has_prev, gmax_layer, stats, cls, vq, gq, seed, sigma_override, w, st);
}

extern "C" size_t dai8_quantize_tensor_workspace_bytes(void) { return kQuantizeTensorWsBytes; }

extern "C" dai8_status dai8_quantize_tensor(const void* x, dai8_dtype dtype, dai8_layout layout, int N,
                                            int C, int H, int W, dai8_scale_mode scale_mode,
                                            float* scale, dai8_round round, uint32_t seed, int8_t* q,
                                            void* ws, size_t ws_bytes, void* stream) {
  if (!x || !scale || !q) return DAI8_ERR_INVALID_ARG;
  if (ws && !aligned16(ws)) return DAI8_ERR_INVALID_ARG;
  if (ws && ws_bytes < kQuantizeTensorWsBytes) return DAI8_ERR_WORKSPACE;
  if (bad_dims(N, C, H, W)) return DAI8_ERR_INVALID_ARG;
  if (dtype != DAI8_F32 && dtype != DAI8_BF16) return DAI8_ERR_INVALID_ARG;
  if (layout != DAI8_NCHW && layout != DAI8_NHWC) return DAI8_ERR_INVALID_ARG;
  if (scale_mode != DAI8_SCALE_ABSMAX && scale_mode != DAI8_SCALE_GIVEN) return DAI8_ERR_INVALID_ARG;
  if (round != DAI8_ROUND_NEAREST_EVEN && round != DAI8_ROUND_STOCHASTIC) return DAI8_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(q)) return DAI8_ERR_INVALID_ARG;
  dai8_status a = check_device_arch();
  if (a != DAI8_OK) return a;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (dtype == DAI8_F32)
    return quantize_tensor_typed<float>(static_cast<const float*>(x), layout, N, C, H, W, scale_mode,
                                        scale, round, seed, q, ws, st);
  return quantize_tensor_typed<bf16_t>(static_cast<const bf16_t*>(x), layout, N, C, H, W, scale_mode,
                                       scale, round, seed, q, ws, st);
}

// ------------------------------------------------------------------------------------------------
// Self-test of the give-up path of the bounded waits.  Nothing is in flight: one CTA initialises an
// mbarrier on which nobody ever arrives and waits for it, then meets a grid barrier whose target is one
// arrival more than there are CTAs -- both with a limit of a few thousand cycles instead of a second.
// Each wait must return false by itself and leave DAI8_ERR_TIMEOUT in the device status word; the
// kernel then ends normally, so the context stays usable.
// ------------------------------------------------------------------------------------------------
namespace dai8 {
namespace {
__global__ void __launch_bounds__(kFT)
expire_waits_kernel(uint32_t* gridbar, unsigned int* status, long long limit, int* report) {
  __shared__ uint64_t bar;
  __shared__ volatile uint32_t s_abort;
  __shared__ uint32_t s_ok;
  if (threadIdx.x == 0) {
    s_abort = 0u;
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const bool ok1 = mbar_wait(&bar, 0u, &s_abort, status, limit);
  __syncthreads();
  if (threadIdx.x == 0) { report[0] = ok1 ? 0 : 1; s_abort = 0u; }
  __syncthreads();
  const bool ok2 = grid_barrier(gridbar, gridDim.x + 1u, status, &s_abort, &s_ok, limit);
  if (threadIdx.x == 0) report[1] = ok2 ? 0 : 1;
}
}  // namespace
dai8_status expire_gvq_waits(long long limit, void* ws, int* report_dev, cudaStream_t st) {
  unsigned int* status = device_status_address();
  if (!status) return DAI8_ERR_CUDA;
  DAI8_RETURN_IF_CUDA(cudaMemsetAsync(ws, 0, 16, st));
  expire_waits_kernel<<<1, kFT, 0, st>>>(static_cast<uint32_t*>(ws), status, limit, report_dev);
  note_launch(1);
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}
}  // namespace dai8

// ------------------------------------------------------------------------------------------------
// dai8_quantize_grad_noalloc: the same kernels as dai8_quantize_grad, with the scratch memory taken
// from an array that is part of the library image instead of from the caller.
//
// It exists for callers that have no way to obtain device memory at the moment they need the
// gradient codes: an extension that is only ever handed the tensors it works on (inputs and
// outputs) by a host framework and must not touch that framework's memory pool, a process whose
// device memory has been handed out completely to other components at start-up, or a
// latency-critical loop in which a cudaMalloc would stall every stream of the device.  Such a caller
// still owns dY, the state and the code tensors; only the reduction scratch comes from here.
//
// The array costs kNoAllocScratchBytes on every GPU on which this library is loaded, for as long as
// the process lives, whether or not this entry point is ever called -- hence the modest limit of
// DAI8_NOALLOC_MAX_CHANNELS channels.  All calls on a device share the array: two calls that can
// overlap on the GPU (different streams, no dependency) race on it.  Nothing in it carries over
// from one call to the next; the control words that must start at zero are cleared on the stream
// at the start of every call, the rest is written before it is read.
//
// In host code the array's name is only a handle.  The device address is looked up once per device
// with cudaGetSymbolAddress, with that device current, on the first call made on that device; do
// that first call outside any stream capture.
// ------------------------------------------------------------------------------------------------
namespace dai8 {
namespace {

constexpr size_t kNoAllocScratchBytes = (size_t)3 << 20;  // 3 MiB
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_noalloc_mutex;
void* g_noalloc_ptr[kMaxDevices] = {};

// Device address of g_noalloc_scratch on the current device (nullptr and a status on failure).
dai8_status noalloc_scratch_address(void** out) {
  int dev = -1;
  DAI8_RETURN_IF_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return DAI8_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (!g_noalloc_ptr[dev]) {
    void* p = nullptr;
    DAI8_RETURN_IF_CUDA(cudaGetSymbolAddress((void**)&p, g_noalloc_scratch));
    if (!p || !aligned16(p)) return DAI8_ERR_CUDA;
    g_noalloc_ptr[dev] = p;
  }
  *out = g_noalloc_ptr[dev];
  return DAI8_OK;
}

}  // namespace
}  // namespace dai8

extern "C" dai8_status dai8_quantize_grad_noalloc(const void* dY, dai8_dtype dtype, dai8_layout layout,
                                                  int N, int C, int H, int W,
                                                  const dai8_mcs_params* params, float* s_state,
                                                  int has_prev, float* gmax_layer, float* stats,
                                                  uint8_t* cls, int8_t* vq, int8_t* gq, uint32_t seed,
                                                  void* stream) {
  if (!dY || !s_state || !gmax_layer || !vq) return DAI8_ERR_INVALID_ARG;
  if (bad_dims(N, C, H, W)) return DAI8_ERR_INVALID_ARG;
  if (dtype != DAI8_F32 && dtype != DAI8_BF16) return DAI8_ERR_INVALID_ARG;
  if (layout != DAI8_NCHW && layout != DAI8_NHWC) return DAI8_ERR_INVALID_ARG;
  if (!aligned16(dY) || !aligned16(vq) || (gq && !aligned16(gq))) return DAI8_ERR_INVALID_ARG;
  if ((int64_t)N * H * W >= (int64_t)1 << 32) return DAI8_ERR_UNSUPPORTED;
  // the built-in scratch is sized for DAI8_NOALLOC_MAX_CHANNELS channels
  if (C > DAI8_NOALLOC_MAX_CHANNELS || ws_bytes_for(C) > kNoAllocScratchBytes) return DAI8_ERR_WORKSPACE;
  dai8_status a = check_device_arch();
  if (a != DAI8_OK) return a;
  void* scratch = nullptr;
  a = noalloc_scratch_address(&scratch);
  if (a != DAI8_OK) return a;
  dai8_mcs_params p;
  if (params) p = *params; else dai8_mcs_defaults(&p);
  if (p.mode < DAI8_GRAD_FULL || p.mode > DAI8_GRAD_LAYER_MCS) return DAI8_ERR_INVALID_ARG;
  McsDev mp = make_mcs(p);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  GvqWs w = carve(scratch, C);
  DAI8_RETURN_IF_CUDA(cudaMemsetAsync(w.tickets, 0, control_words(C) * 4, st));
  if (dtype == DAI8_F32)
    return quantize_grad_typed<float>(static_cast<const float*>(dY), layout, N, C, H, W, mp, s_state,
                                      has_prev, gmax_layer, stats, cls, vq, gq, seed, nullptr, w, st);
  return quantize_grad_typed<bf16_t>(static_cast<const bf16_t*>(dY), layout, N, C, H, W, mp, s_state,
                                     has_prev, gmax_layer, stats, cls, vq, gq, seed, nullptr, w, st);
}
