// Integer convolutions with a depth dimension and channel groups on the CUDA cores: the variants
// the paper names beside the plain 2-D layer -- 3-D convolution, with the depth treated like height
// and width (Sec. 4.4), and depth-wise convolution (groups = channels; the MobileNetV2 paragraph of
// Sec. 4.2).  Same arithmetic as the 2-D entry points: int8 codes, int32 accumulation (wrapping),
// de-quantizing epilogue (Eq. 3-7 with a third spatial index).
//
//   codes    activations / gradients [N][D][H][W][Cp], weights [Cout][T][R][S][Cgp]
//            (Cp, Cgp: channels and channels per group rounded up to 16, padding 0) -- what
//            dai8_quantize_tensor writes for an (N, C, D*H, W) tensor and for weights passed as
//            an NCHW tensor (N = Cout, C = Cin/groups, H = T*R, W = S)
//   forward          one thread per output element (pixel, co), 4 channels per dp4a where the
//                    group width allows
//   input gradient   one thread per (pixel, ci), over the taps that reach it (no zero insertion)
//   weight gradient  one block per (co, channel of its group): the threads walk over the output
//                    positions with one accumulator per tap (T*R*S <= 32), then a block reduction
// These are correctness-first kernels: they cover every geometry, they are not tuned.
#include "conv_internal.cuh"

namespace dai8 {
namespace {

constexpr int kNdThreads = 256;
constexpr int kNdMaxTaps = 32;

struct Shape3 {
  int N, Cin, Cout, D, H, W, T, R, S, sd, sh, sw, pd, ph, pw, groups;
  int Do, P, Q, Cinp, Coutp, cpg, opg, Cgp;
};

Shape3 make_shape3(const dai8_conv3d_geom& g) {
  Shape3 s;
  s.N = g.N; s.Cin = g.Cin; s.Cout = g.Cout; s.D = g.D; s.H = g.H; s.W = g.W; s.T = g.T; s.R = g.R; s.S = g.S;
  s.sd = g.stride_d; s.sh = g.stride_h; s.sw = g.stride_w; s.pd = g.pad_d; s.ph = g.pad_h; s.pw = g.pad_w;
  s.groups = g.groups > 0 ? g.groups : 1;
  s.Do = (g.D + 2 * g.pad_d - g.T) / g.stride_d + 1;
  s.P = (g.H + 2 * g.pad_h - g.R) / g.stride_h + 1;
  s.Q = (g.W + 2 * g.pad_w - g.S) / g.stride_w + 1;
  s.Cinp = round_up(g.Cin, 16); s.Coutp = round_up(g.Cout, 16);
  s.cpg = g.Cin / s.groups; s.opg = g.Cout / s.groups;
  s.Cgp = round_up(s.cpg, 16);
  return s;
}

__global__ void __launch_bounds__(kNdThreads)
nd_fwd_kernel(const int8_t* __restrict__ qX, const int8_t* __restrict__ qW, const float* __restrict__ sX,
              const float* __restrict__ sW, Shape3 s, void* __restrict__ Y, dai8_dtype dtype) {
  const int64_t total = (int64_t)s.N * s.Do * s.P * s.Q * s.Cout;
  const float scale = dtype == DAI8_I32 ? 0.f : dequant_scale(*sX, *sW);
  const bool words = s.cpg % 4 == 0;
  for (int64_t i = (int64_t)blockIdx.x * kNdThreads + threadIdx.x; i < total; i += (int64_t)gridDim.x * kNdThreads) {
    int64_t f = i;
    const int co = (int)(f % s.Cout); f /= s.Cout;
    const int q = (int)(f % s.Q); f /= s.Q;
    const int p = (int)(f % s.P); f /= s.P;
    const int od = (int)(f % s.Do);
    const int n = (int)(f / s.Do);
    const int c0 = (co / s.opg) * s.cpg;
    int acc = 0;
    for (int t = 0; t < s.T; ++t) {
      const int d = od * s.sd + t - s.pd;
      if (d < 0 || d >= s.D) continue;
      for (int r = 0; r < s.R; ++r) {
        const int h = p * s.sh + r - s.ph;
        if (h < 0 || h >= s.H) continue;
        for (int ss = 0; ss < s.S; ++ss) {
          const int w = q * s.sw + ss - s.pw;
          if (w < 0 || w >= s.W) continue;
          const int8_t* x = qX + ((((int64_t)n * s.D + d) * s.H + h) * s.W + w) * s.Cinp + c0;
          const int8_t* wt = qW + ((((int64_t)co * s.T + t) * s.R + r) * s.S + ss) * s.Cgp;
          if (words) {
            for (int c = 0; c < s.cpg; c += 4)
              acc = __dp4a(*reinterpret_cast<const int*>(x + c), *reinterpret_cast<const int*>(wt + c), acc);
          } else {
            for (int c = 0; c < s.cpg; ++c) acc += (int)x[c] * (int)wt[c];
          }
        }
      }
    }
    store_result(Y, dtype, (size_t)i, acc, scale);     // [N][Do][P][Q][Cout], channels unpadded
  }
}

__global__ void __launch_bounds__(kNdThreads)
nd_bwd_data_kernel(const int8_t* __restrict__ gq, const int8_t* __restrict__ qW, const float* __restrict__ gmax,
                   const float* __restrict__ sW, Shape3 s, void* __restrict__ dX, dai8_dtype dtype) {
  const int64_t total = (int64_t)s.N * s.D * s.H * s.W * s.Cin;
  const float scale = dtype == DAI8_I32 ? 0.f : dequant_scale(*gmax, *sW);
  const int64_t wco = (int64_t)s.T * s.R * s.S * s.Cgp;        // weight codes per output channel
  for (int64_t i = (int64_t)blockIdx.x * kNdThreads + threadIdx.x; i < total; i += (int64_t)gridDim.x * kNdThreads) {
    int64_t f = i;
    const int ci = (int)(f % s.Cin); f /= s.Cin;
    const int w = (int)(f % s.W); f /= s.W;
    const int h = (int)(f % s.H); f /= s.H;
    const int d = (int)(f % s.D);
    const int n = (int)(f / s.D);
    const int grp = ci / s.cpg, cl = ci - grp * s.cpg, co0 = grp * s.opg;
    int acc = 0;
    for (int t = 0; t < s.T; ++t) {
      const int dd = d + s.pd - t;
      if (dd < 0 || dd % s.sd != 0 || dd / s.sd >= s.Do) continue;
      for (int r = 0; r < s.R; ++r) {
        const int hp = h + s.ph - r;
        if (hp < 0 || hp % s.sh != 0 || hp / s.sh >= s.P) continue;
        for (int ss = 0; ss < s.S; ++ss) {
          const int wq = w + s.pw - ss;
          if (wq < 0 || wq % s.sw != 0 || wq / s.sw >= s.Q) continue;
          const int8_t* g = gq + ((((int64_t)n * s.Do + dd / s.sd) * s.P + hp / s.sh) * s.Q + wq / s.sw) * s.Coutp + co0;
          const int8_t* wt = qW + (int64_t)co0 * wco + (((int64_t)t * s.R + r) * s.S + ss) * s.Cgp + cl;
          for (int o = 0; o < s.opg; ++o) acc += (int)g[o] * (int)wt[(int64_t)o * wco];
        }
      }
    }
    store_result(dX, dtype, (size_t)i, acc, scale);    // [N][D][H][W][Cin]
  }
}

// grid = (Cout, cpg); dW[co][cl][t][r][s]
__global__ void __launch_bounds__(kNdThreads)
nd_bwd_filter_kernel(const int8_t* __restrict__ qX, const int8_t* __restrict__ vq, const float* __restrict__ sX,
                     const float* __restrict__ sc, Shape3 s, void* __restrict__ dW, dai8_dtype dtype) {
  __shared__ int red[kNdThreads / 32][kNdMaxTaps];
  const int co = blockIdx.x, cl = blockIdx.y;
  const int ci = (co / s.opg) * s.cpg + cl;
  const int taps = s.T * s.R * s.S;
  int acc[kNdMaxTaps];
#pragma unroll
  for (int k = 0; k < kNdMaxTaps; ++k) acc[k] = 0;
  const int64_t npos = (int64_t)s.N * s.Do * s.P * s.Q;
  for (int64_t i = threadIdx.x; i < npos; i += kNdThreads) {
    int64_t f = i;
    const int q = (int)(f % s.Q); f /= s.Q;
    const int p = (int)(f % s.P); f /= s.P;
    const int od = (int)(f % s.Do);
    const int n = (int)(f / s.Do);
    const int g = (int)vq[i * s.Coutp + co];
    if (g == 0) continue;
#pragma unroll
    for (int k = 0; k < kNdMaxTaps; ++k) {
      if (k < taps) {
        const int ss = k % s.S, r = (k / s.S) % s.R, t = k / (s.S * s.R);
        const int d = od * s.sd + t - s.pd, h = p * s.sh + r - s.ph, w = q * s.sw + ss - s.pw;
        if (d >= 0 && d < s.D && h >= 0 && h < s.H && w >= 0 && w < s.W)
          acc[k] += g * (int)qX[((((int64_t)n * s.D + d) * s.H + h) * s.W + w) * s.Cinp + ci];
      }
    }
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int k = 0; k < kNdMaxTaps; ++k) {
    int v = acc[k];
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    if (lane == 0) red[warp][k] = v;
  }
  __syncthreads();
  if (threadIdx.x < taps) {
    int v = 0;
    for (int w = 0; w < kNdThreads / 32; ++w) v += red[w][threadIdx.x];
    const float scale = dtype == DAI8_I32 ? 0.f : dequant_scale(*sX, sc[co]);
    store_result(dW, dtype, ((size_t)co * s.cpg + cl) * taps + threadIdx.x, v, scale);
  }
}

dai8_status check_geom3(const dai8_conv3d_geom* g) {
  if (!g) return DAI8_ERR_INVALID_ARG;
  if (g->N <= 0 || g->Cin <= 0 || g->Cout <= 0 || g->D <= 0 || g->H <= 0 || g->W <= 0 || g->T <= 0 || g->R <= 0 ||
      g->S <= 0 || g->stride_d <= 0 || g->stride_h <= 0 || g->stride_w <= 0 || g->pad_d < 0 || g->pad_h < 0 ||
      g->pad_w < 0 || g->groups < 0)
    return DAI8_ERR_INVALID_ARG;
  const int groups = g->groups > 0 ? g->groups : 1;
  if (g->Cin % groups != 0 || g->Cout % groups != 0) return DAI8_ERR_INVALID_ARG;
  if (g->D + 2 * g->pad_d < g->T || g->H + 2 * g->pad_h < g->R || g->W + 2 * g->pad_w < g->S) return DAI8_ERR_INVALID_ARG;
  if (g->T * g->R * g->S > kNdMaxTaps) return DAI8_ERR_UNSUPPORTED;
  const Shape3 s = make_shape3(*g);
  const int64_t lim = (int64_t)1 << 31;
  if ((int64_t)s.N * s.D * s.H * s.W >= lim || (int64_t)s.N * s.Do * s.P * s.Q >= lim) return DAI8_ERR_UNSUPPORTED;
  // with several groups a group must start on a code word of its own channels
  if (groups > 1 && s.cpg % 4 != 0 && s.cpg != 1) return DAI8_ERR_UNSUPPORTED;
  return DAI8_OK;
}

int grid_for(int64_t total) {
  int64_t b = (total + kNdThreads - 1) / kNdThreads;
  const int64_t cap = (int64_t)sm_count() * 16;
  if (b > cap) b = cap;
  return (int)(b < 1 ? 1 : b);
}

}  // namespace
}  // namespace dai8

using namespace dai8;

extern "C" dai8_status dai8_conv3d_fwd(const int8_t* qX, const int8_t* qW, const float* sX, const float* sW,
                                       const dai8_conv3d_geom* geom, void* Y, dai8_dtype out_dtype, void* stream) {
  dai8_status g = check_geom3(geom);
  if (g != DAI8_OK) return g;
  if (!qX || !qW || !Y || (out_dtype != DAI8_F32 && out_dtype != DAI8_BF16 && out_dtype != DAI8_I32)) return DAI8_ERR_INVALID_ARG;
  if (out_dtype != DAI8_I32 && (!sX || !sW)) return DAI8_ERR_INVALID_ARG;
  if (!aligned16(qX) || !aligned16(qW) || !aligned16(Y)) return DAI8_ERR_INVALID_ARG;
  dai8_status a = check_device_arch();
  if (a != DAI8_OK) return a;
  const Shape3 s = make_shape3(*geom);
  const int64_t total = (int64_t)s.N * s.Do * s.P * s.Q * s.Cout;
  nd_fwd_kernel<<<grid_for(total), kNdThreads, 0, static_cast<cudaStream_t>(stream)>>>(qX, qW, sX, sW, s, Y, out_dtype);
  note_launch(1);
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}

extern "C" dai8_status dai8_conv3d_bwd_data(const int8_t* gq, const int8_t* qW, const float* gmax, const float* sW,
                                            const dai8_conv3d_geom* geom, void* dX, dai8_dtype out_dtype,
                                            void* stream) {
  dai8_status g = check_geom3(geom);
  if (g != DAI8_OK) return g;
  if (!gq || !qW || !dX || (out_dtype != DAI8_F32 && out_dtype != DAI8_BF16 && out_dtype != DAI8_I32)) return DAI8_ERR_INVALID_ARG;
  if (out_dtype != DAI8_I32 && (!gmax || !sW)) return DAI8_ERR_INVALID_ARG;
  if (!aligned16(gq) || !aligned16(qW) || !aligned16(dX)) return DAI8_ERR_INVALID_ARG;
  dai8_status a = check_device_arch();
  if (a != DAI8_OK) return a;
  const Shape3 s = make_shape3(*geom);
  const int64_t total = (int64_t)s.N * s.D * s.H * s.W * s.Cin;
  nd_bwd_data_kernel<<<grid_for(total), kNdThreads, 0, static_cast<cudaStream_t>(stream)>>>(gq, qW, gmax, sW, s, dX, out_dtype);
  note_launch(1);
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}

extern "C" dai8_status dai8_conv3d_bwd_filter(const int8_t* qX, const int8_t* vq, const float* sX, const float* s_c,
                                              const dai8_conv3d_geom* geom, void* dW, dai8_dtype out_dtype,
                                              void* stream) {
  dai8_status g = check_geom3(geom);
  if (g != DAI8_OK) return g;
  if (!qX || !vq || !dW || (out_dtype != DAI8_F32 && out_dtype != DAI8_I32)) return DAI8_ERR_INVALID_ARG;
  if (out_dtype != DAI8_I32 && (!sX || !s_c)) return DAI8_ERR_INVALID_ARG;
  if (!aligned16(qX) || !aligned16(vq) || !aligned16(dW)) return DAI8_ERR_INVALID_ARG;
  dai8_status a = check_device_arch();
  if (a != DAI8_OK) return a;
  const Shape3 s = make_shape3(*geom);
  if (s.cpg > 65535) return DAI8_ERR_UNSUPPORTED;
  nd_bwd_filter_kernel<<<dim3((unsigned)s.Cout, (unsigned)s.cpg), kNdThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      qX, vq, sX, s_c, s, dW, out_dtype);
  note_launch(1);
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}
