// CPU oracle for Distribution Adaptive INT8 quantization of the convolution backward pass.
//
// TEST INFRASTRUCTURE ONLY.  This file is a slow, direct restatement of the method's definitions
// (symmetric uniform quantizer Eq. 1, gradient vectorized quantization Sec. 3.2, the gradient
// discriminator Eq. 15, the clip update Eq. 14, Algorithm 1, and the convolution gradients Eq. 3/4).
// It shares no code, header, table or constant with the CUDA library and is never called by it.
// Only the tests, the smoke check and the benchmark's CPU-baseline leg load it.
//
// Conventions
//   * Tensors are plain row-major NCHW (activations, gradients) and (Cout,Cin,R,S) (weights).
//   * Per-element floating-point arithmetic is IEEE binary32, round-to-nearest, one operation at a
//     time (build with -ffp-contract=off).  Statistics are accumulated in binary64.
//   * Integer convolutions accumulate in int64 so that overflow of an int32 accumulator can be
//     detected instead of silently reproduced.
//   * OpenMP only splits independent channels / output elements across cores; no blocking,
//     no reordering inside an element.
//
// Pinned by tests/test_oracle_*.py (closed forms, brute force, library routines, invariants).

#include <cmath>
#include <cstdint>
#include <cstring>
#include <cfenv>
#ifdef _OPENMP
#include <omp.h>
#endif

extern "C" {

int dai8o_num_threads() {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

// ---------------------------------------------------------------------------------------------
// Algorithm 1, statistics step: per-channel |g|max, mean and sigma; layer |g|max (the scale of
// the layer-wide codes).
// Eq. 15 names mu "the mean of gradient": sigma is taken about the mean unless center_mean == 0
// (then it is the root mean square, which Assumption 1 makes equivalent).  Population variance
// (divide by M) unless std_unbiased != 0 (divide by M-1).
// g: NCHW fp32.  Outputs: absmax[C], mean[C], sigma[C] (fp32), gmax_layer[1].
// ---------------------------------------------------------------------------------------------
void dai8o_channel_stats(const float* g, int N, int C, int H, int W, int std_unbiased,
                         int center_mean, float* absmax, float* mean, float* sigma,
                         float* gmax_layer) {
  const int64_t HW = (int64_t)H * W;
  const int64_t M = (int64_t)N * HW;
#pragma omp parallel for schedule(static)
  for (int c = 0; c < C; ++c) {
    float amax = 0.0f;
    double sum = 0.0;
    for (int n = 0; n < N; ++n) {
      const float* p = g + ((int64_t)n * C + c) * HW;
      for (int64_t i = 0; i < HW; ++i) {
        float a = std::fabs(p[i]);
        if (a > amax) amax = a;
        sum += (double)p[i];
      }
    }
    const double mu = (M > 0) ? sum / (double)M : 0.0;
    const double pivot = center_mean ? mu : 0.0;
    double ss = 0.0;
    for (int n = 0; n < N; ++n) {
      const float* p = g + ((int64_t)n * C + c) * HW;
      for (int64_t i = 0; i < HW; ++i) {
        double d = (double)p[i] - pivot;
        ss += d * d;
      }
    }
    const double denom = std_unbiased ? (double)(M - 1) : (double)M;
    absmax[c] = amax;
    mean[c] = (float)mu;
    sigma[c] = (denom > 0.0) ? (float)std::sqrt(ss / denom) : 0.0f;
  }
  float gl = 0.0f;
  for (int c = 0; c < C; ++c)
    if (absmax[c] > gl) gl = absmax[c];
  *gmax_layer = gl;
}

// ---------------------------------------------------------------------------------------------
// Algorithm 1, density step: number of elements of channel c with |g| > sigma_c (strict, on |g| and not
// on |g - mu|, compared in binary32).  cnt[C].
// ---------------------------------------------------------------------------------------------
void dai8o_density_count(const float* g, int N, int C, int H, int W, const float* sigma,
                         uint32_t* cnt) {
  const int64_t HW = (int64_t)H * W;
#pragma omp parallel for schedule(static)
  for (int c = 0; c < C; ++c) {
    uint32_t k = 0;
    const float sg = sigma[c];
    for (int n = 0; n < N; ++n) {
      const float* p = g + ((int64_t)n * C + c) * HW;
      for (int64_t i = 0; i < HW; ++i)
        if (std::fabs(p[i]) > sg) ++k;
    }
    cnt[c] = k;
  }
}

// ---------------------------------------------------------------------------------------------
// Algorithm 1, the if/else on P, with Eq. 15 (discriminator) and Eq. 14 (clip update).
//   P = cnt / M ;  P > lambda  -> bell-shaped (cls = 1):  s_t = |g|max,c            (Eq. 11)
//                  otherwise    -> Inverted-T  (cls = 0):  s_t = (1-kA) s_{t-1} + A |g|max,c
// The test P > lambda is evaluated as cnt > lambda*M in binary64 (lambda is the binary32 value).
// has_prev == 0 (first iteration): s_{t-1} := |g|max,c.  The recurrence is evaluated in binary32
// as t = 1 - k*A; s = t*s_prev; s = s + A*gmax, each operation rounded.
// s_state[C] is read (if has_prev) and overwritten with s_t in both branches.
// ---------------------------------------------------------------------------------------------
void dai8o_classify_clip(const uint32_t* cnt, const float* absmax, int C, int64_t M, float lambda,
                         float k, float A, float* s_state, int has_prev, uint8_t* cls) {
  for (int c = 0; c < C; ++c) {
    const bool bell = (double)cnt[c] > (double)lambda * (double)M;
    const float gmax = absmax[c];
    float s;
    if (bell) {
      s = gmax;
    } else {
      const float s_prev = has_prev ? s_state[c] : gmax;
      volatile float t = 1.0f - k * A;  // k*A rounded, then the subtraction rounded
      volatile float a = t * s_prev;
      volatile float b = A * gmax;
      s = a + b;
    }
    s_state[c] = s;
    cls[c] = bell ? 1 : 0;
  }
}

// ---------------------------------------------------------------------------------------------
// Counter-based uniform numbers for stochastic rounding.  The paper names the rounding mode
// (Sec. 3) but fixes no generator; this one is defined by its integer arithmetic:
//   key = finalise32(seed xor 0x9E3779B9 * (high half of the index + 1))       (once per 2^32 elements)
//   x   = low half of the index * 0x9E3779B1 + key                            (mod 2^32)
//   f   = high half xor low half of the 64-bit product x * 0x85EBCA6B         (a folded multiply)
//   h   = f * 0xC2B2AE35 for stream 0 (per-channel codes), f * 0x2C1B3C6D for stream 1 (layer-wide codes)
//   u   = (h >> 9) * 2^-23, in [0, 1).
// finalise32 is a 32-bit avalanche function (xor-shift 16, multiply, xor-shift 13, multiply,
// xor-shift 16).
static inline uint32_t finalise32(uint32_t h) {
  h ^= h >> 16;
  h *= 0x85EBCA6Bu;
  h ^= h >> 13;
  h *= 0xC2B2AE35u;
  h ^= h >> 16;
  return h;
}

uint32_t dai8o_rand_bits(uint32_t seed, uint32_t stream, uint64_t index) {
  const uint32_t hi = (uint32_t)(index >> 32);
  const uint32_t lo = (uint32_t)index;
  const uint32_t key = finalise32(seed ^ (0x9E3779B9u * (hi + 1u)));
  const uint32_t x = lo * 0x9E3779B1u + key;
  const uint64_t p = (uint64_t)x * 0x85EBCA6Bull;
  const uint32_t f = (uint32_t)(p >> 32) ^ (uint32_t)p;
  return f * (stream != 0 ? 0x2C1B3C6Du : 0xC2B2AE35u);
}

float dai8o_rand_uniform(uint32_t seed, uint32_t stream, uint64_t index) {
  return (float)(dai8o_rand_bits(seed, stream, index) >> 9) * 0x1p-23f;
}

// ---------------------------------------------------------------------------------------------
// Eq. 1: q(x) = round(127 * clamp(x, s) / s), codes in [-127, 127].
//   inv = 127 / s (one binary32 division per scale); v = x * inv; v clamped to [-127, 127];
//   round_mode 0: nearest, ties to even;  round_mode 1: stochastic, q = min(127, floor(v + u))
//   with u from dai8o_rand_uniform(seed, stream, NCHW index of the element).
//   s <= 0 (an all-zero channel) gives code 0.
// x: NCHW fp32.  scale: C values if per_channel else 1.  q: NCHW int8.
// ---------------------------------------------------------------------------------------------
static inline int8_t quantize_one(float x, float s, int round_mode, uint32_t seed, uint32_t stream,
                                  uint64_t index) {
  if (!(s > 0.0f)) return 0;
  const float inv = 127.0f / s;
  float v = x * inv;
  if (v < -127.0f) v = -127.0f;
  if (v > 127.0f) v = 127.0f;
  if (v != v) return 0;  // NaN input: code 0
  int q;
  if (round_mode == 0) {
    q = (int)std::nearbyintf(v);  // default rounding direction: to nearest, ties to even
  } else {
    const float u = dai8o_rand_uniform(seed, stream, index);
    const float t = v + u;
    q = (int)std::floor(t);
    if (q > 127) q = 127;
  }
  return (int8_t)q;
}

// x holds images first_image .. first_image + N - 1 of a larger NCHW tensor: the generator's counter
// is the element's index in that whole tensor (first_image = 0: x is the whole tensor).
void dai8o_quantize_at(const float* x, int N, int C, int H, int W, int64_t first_image, const float* scale,
                       int per_channel, int round_mode, uint32_t seed, uint32_t stream, int8_t* q) {
  std::fesetround(FE_TONEAREST);
  const int64_t HW = (int64_t)H * W;
  const uint64_t offset = (uint64_t)first_image * (uint64_t)C * (uint64_t)HW;
#pragma omp parallel for schedule(static) collapse(2)
  for (int n = 0; n < N; ++n)
    for (int c = 0; c < C; ++c) {
      const float s = per_channel ? scale[c] : scale[0];
      const int64_t base = ((int64_t)n * C + c) * HW;
      for (int64_t i = 0; i < HW; ++i)
        q[base + i] = quantize_one(x[base + i], s, round_mode, seed, stream, offset + (uint64_t)(base + i));
    }
}

void dai8o_quantize(const float* x, int N, int C, int H, int W, const float* scale,
                    int per_channel, int round_mode, uint32_t seed, uint32_t stream, int8_t* q) {
  dai8o_quantize_at(x, N, C, H, W, 0, scale, per_channel, round_mode, seed, stream, q);
}

// De-quantizer of Eq. 1: x_hat = q * s / 127 (binary32: (float)q * (s / 127)).
void dai8o_dequantize(const int8_t* q, int N, int C, int H, int W, const float* scale,
                      int per_channel, float* x_hat) {
  const int64_t HW = (int64_t)H * W;
  for (int n = 0; n < N; ++n)
    for (int c = 0; c < C; ++c) {
      const float step = (per_channel ? scale[c] : scale[0]) / 127.0f;
      const int64_t base = ((int64_t)n * C + c) * HW;
      for (int64_t i = 0; i < HW; ++i) x_hat[base + i] = (float)q[base + i] * step;
    }
}

// ---------------------------------------------------------------------------------------------
// Integer convolutions (cross-correlation, dilation 1, groups 1).  P, Q are the output extents:
// P = (H + 2*pad_h - R)/stride_h + 1, Q likewise.
// ---------------------------------------------------------------------------------------------
struct Geom {
  int N, Cin, Cout, H, W, R, S, stride_h, stride_w, pad_h, pad_w;
};

static inline int out_extent(int in, int pad, int k, int stride) {
  return (in + 2 * pad - k) / stride + 1;
}

// Forward: Y[n,co,p,q] = sum_{ci,r,s} X[n,ci,p*st+r-pad,q*st+s-pad] * W[co,ci,r,s].
static int64_t fwd_at(const int8_t* X, const int8_t* Wt, const Geom& g, int n, int co, int p,
                      int q) {
  int64_t acc = 0;
  for (int ci = 0; ci < g.Cin; ++ci)
    for (int r = 0; r < g.R; ++r) {
      const int h = p * g.stride_h + r - g.pad_h;
      if (h < 0 || h >= g.H) continue;
      for (int s = 0; s < g.S; ++s) {
        const int w = q * g.stride_w + s - g.pad_w;
        if (w < 0 || w >= g.W) continue;
        acc += (int64_t)X[(((int64_t)n * g.Cin + ci) * g.H + h) * g.W + w] *
               (int64_t)Wt[(((int64_t)co * g.Cin + ci) * g.R + r) * g.S + s];
      }
    }
  return acc;
}

// Eq. 3 (input gradient, the transposed convolution):
// dX[n,ci,h,w] = sum over (co,r,s,p,q) with h = p*st+r-pad, w = q*st+s-pad of G[n,co,p,q]*W[co,ci,r,s].
static int64_t bwd_data_at(const int8_t* G, const int8_t* Wt, const Geom& g, int P, int Q, int n,
                           int ci, int h, int w) {
  int64_t acc = 0;
  for (int co = 0; co < g.Cout; ++co)
    for (int r = 0; r < g.R; ++r) {
      const int hp = h + g.pad_h - r;
      if (hp < 0 || hp % g.stride_h != 0) continue;
      const int p = hp / g.stride_h;
      if (p >= P) continue;
      for (int s = 0; s < g.S; ++s) {
        const int wq = w + g.pad_w - s;
        if (wq < 0 || wq % g.stride_w != 0) continue;
        const int q = wq / g.stride_w;
        if (q >= Q) continue;
        acc += (int64_t)G[(((int64_t)n * g.Cout + co) * P + p) * Q + q] *
               (int64_t)Wt[(((int64_t)co * g.Cin + ci) * g.R + r) * g.S + s];
      }
    }
  return acc;
}

// Eq. 4 (weight gradient, contraction over n and the output pixels):
// dW[co,ci,r,s] = sum_{n,p,q} G[n,co,p,q] * X[n,ci,p*st+r-pad,q*st+s-pad].
static int64_t bwd_filter_at(const int8_t* X, const int8_t* G, const Geom& g, int P, int Q, int co,
                             int ci, int r, int s) {
  int64_t acc = 0;
  for (int n = 0; n < g.N; ++n)
    for (int p = 0; p < P; ++p) {
      const int h = p * g.stride_h + r - g.pad_h;
      if (h < 0 || h >= g.H) continue;
      for (int q = 0; q < Q; ++q) {
        const int w = q * g.stride_w + s - g.pad_w;
        if (w < 0 || w >= g.W) continue;
        acc += (int64_t)G[(((int64_t)n * g.Cout + co) * P + p) * Q + q] *
               (int64_t)X[(((int64_t)n * g.Cin + ci) * g.H + h) * g.W + w];
      }
    }
  return acc;
}

// Each entry point computes either the whole output tensor (n_idx == 0; acc has one int64 per
// output element, row-major) or only the flat output indices listed in idx (acc has n_idx entries).
// Return value: number of computed outputs that do not fit an int32 accumulator.
int64_t dai8o_conv_fwd_acc(const int8_t* X, const int8_t* Wt, const int* geom, const int64_t* idx,
                           int64_t n_idx, int64_t* acc) {
  Geom g;
  std::memcpy(&g, geom, sizeof(Geom));
  const int P = out_extent(g.H, g.pad_h, g.R, g.stride_h);
  const int Q = out_extent(g.W, g.pad_w, g.S, g.stride_w);
  const int64_t total = n_idx > 0 ? n_idx : (int64_t)g.N * g.Cout * P * Q;
  int64_t overflow = 0;
#pragma omp parallel for schedule(dynamic, 256) reduction(+ : overflow)
  for (int64_t i = 0; i < total; ++i) {
    int64_t f = n_idx > 0 ? idx[i] : i;
    const int q = (int)(f % Q); f /= Q;
    const int p = (int)(f % P); f /= P;
    const int co = (int)(f % g.Cout);
    const int n = (int)(f / g.Cout);
    const int64_t a = fwd_at(X, Wt, g, n, co, p, q);
    acc[i] = a;
    if (a > INT32_MAX || a < INT32_MIN) ++overflow;
  }
  return overflow;
}

int64_t dai8o_conv_bwd_data_acc(const int8_t* G, const int8_t* Wt, const int* geom,
                                const int64_t* idx, int64_t n_idx, int64_t* acc) {
  Geom g;
  std::memcpy(&g, geom, sizeof(Geom));
  const int P = out_extent(g.H, g.pad_h, g.R, g.stride_h);
  const int Q = out_extent(g.W, g.pad_w, g.S, g.stride_w);
  const int64_t total = n_idx > 0 ? n_idx : (int64_t)g.N * g.Cin * g.H * g.W;
  int64_t overflow = 0;
#pragma omp parallel for schedule(dynamic, 256) reduction(+ : overflow)
  for (int64_t i = 0; i < total; ++i) {
    int64_t f = n_idx > 0 ? idx[i] : i;
    const int w = (int)(f % g.W); f /= g.W;
    const int h = (int)(f % g.H); f /= g.H;
    const int ci = (int)(f % g.Cin);
    const int n = (int)(f / g.Cin);
    const int64_t a = bwd_data_at(G, Wt, g, P, Q, n, ci, h, w);
    acc[i] = a;
    if (a > INT32_MAX || a < INT32_MIN) ++overflow;
  }
  return overflow;
}

int64_t dai8o_conv_bwd_filter_acc(const int8_t* X, const int8_t* G, const int* geom,
                                  const int64_t* idx, int64_t n_idx, int64_t* acc) {
  Geom g;
  std::memcpy(&g, geom, sizeof(Geom));
  const int P = out_extent(g.H, g.pad_h, g.R, g.stride_h);
  const int Q = out_extent(g.W, g.pad_w, g.S, g.stride_w);
  const int64_t total = n_idx > 0 ? n_idx : (int64_t)g.Cout * g.Cin * g.R * g.S;
  int64_t overflow = 0;
#pragma omp parallel for schedule(dynamic, 1) reduction(+ : overflow)
  for (int64_t i = 0; i < total; ++i) {
    int64_t f = n_idx > 0 ? idx[i] : i;
    const int s = (int)(f % g.S); f /= g.S;
    const int r = (int)(f % g.R); f /= g.R;
    const int ci = (int)(f % g.Cin);
    const int co = (int)(f / g.Cin);
    const int64_t a = bwd_filter_at(X, G, g, P, Q, co, ci, r, s);
    acc[i] = a;
    if (a > INT32_MAX || a < INT32_MIN) ++overflow;
  }
  return overflow;
}

// ---------------------------------------------------------------------------------------------
// The same three integer convolutions with a depth dimension and channel groups: the variants the
// paper names beside the plain 2-D layer -- 3-D convolution, "treating depth dimension in the same
// way as height and width" (Sec. 4.4), and depth-wise convolution (groups = channels, the
// MobileNetV2 paragraph of Sec. 4.2).  X (N,Cin,D,H,W), W (Cout,Cin/groups,T,R,S), Y (N,Cout,Do,P,Q);
// output channel co belongs to group co / (Cout/groups) and reads input channels
// group*(Cin/groups) .. +Cin/groups-1.  With D = T = 1 and groups = 1 these are the functions above.
// ---------------------------------------------------------------------------------------------
struct Geom3 {
  int N, Cin, Cout, D, H, W, T, R, S, stride_d, stride_h, stride_w, pad_d, pad_h, pad_w, groups;
};

static int64_t fwd3_at(const int8_t* X, const int8_t* Wt, const Geom3& g, int n, int co, int od, int p, int q) {
  const int cpg = g.Cin / g.groups, opg = g.Cout / g.groups;
  const int grp = co / opg;
  int64_t acc = 0;
  for (int cl = 0; cl < cpg; ++cl) {
    const int ci = grp * cpg + cl;
    for (int t = 0; t < g.T; ++t) {
      const int d = od * g.stride_d + t - g.pad_d;
      if (d < 0 || d >= g.D) continue;
      for (int r = 0; r < g.R; ++r) {
        const int h = p * g.stride_h + r - g.pad_h;
        if (h < 0 || h >= g.H) continue;
        for (int s = 0; s < g.S; ++s) {
          const int w = q * g.stride_w + s - g.pad_w;
          if (w < 0 || w >= g.W) continue;
          acc += (int64_t)X[((((int64_t)n * g.Cin + ci) * g.D + d) * g.H + h) * g.W + w] *
                 (int64_t)Wt[((((int64_t)co * cpg + cl) * g.T + t) * g.R + r) * g.S + s];
        }
      }
    }
  }
  return acc;
}

static int64_t bwd_data3_at(const int8_t* G, const int8_t* Wt, const Geom3& g, int Do, int P, int Q, int n, int ci,
                            int d, int h, int w) {
  const int cpg = g.Cin / g.groups, opg = g.Cout / g.groups;
  const int grp = ci / cpg, cl = ci - grp * cpg;
  int64_t acc = 0;
  for (int ol = 0; ol < opg; ++ol) {
    const int co = grp * opg + ol;
    for (int t = 0; t < g.T; ++t) {
      const int dd = d + g.pad_d - t;
      if (dd < 0 || dd % g.stride_d != 0 || dd / g.stride_d >= Do) continue;
      for (int r = 0; r < g.R; ++r) {
        const int hp = h + g.pad_h - r;
        if (hp < 0 || hp % g.stride_h != 0 || hp / g.stride_h >= P) continue;
        for (int s = 0; s < g.S; ++s) {
          const int wq = w + g.pad_w - s;
          if (wq < 0 || wq % g.stride_w != 0 || wq / g.stride_w >= Q) continue;
          acc += (int64_t)G[((((int64_t)n * g.Cout + co) * Do + dd / g.stride_d) * P + hp / g.stride_h) * Q + wq / g.stride_w] *
                 (int64_t)Wt[((((int64_t)co * cpg + cl) * g.T + t) * g.R + r) * g.S + s];
        }
      }
    }
  }
  return acc;
}

static int64_t bwd_filter3_at(const int8_t* X, const int8_t* G, const Geom3& g, int Do, int P, int Q, int co, int cl,
                              int t, int r, int s) {
  const int cpg = g.Cin / g.groups, opg = g.Cout / g.groups;
  const int ci = (co / opg) * cpg + cl;
  int64_t acc = 0;
  for (int n = 0; n < g.N; ++n)
    for (int od = 0; od < Do; ++od) {
      const int d = od * g.stride_d + t - g.pad_d;
      if (d < 0 || d >= g.D) continue;
      for (int p = 0; p < P; ++p) {
        const int h = p * g.stride_h + r - g.pad_h;
        if (h < 0 || h >= g.H) continue;
        for (int q = 0; q < Q; ++q) {
          const int w = q * g.stride_w + s - g.pad_w;
          if (w < 0 || w >= g.W) continue;
          acc += (int64_t)G[((((int64_t)n * g.Cout + co) * Do + od) * P + p) * Q + q] *
                 (int64_t)X[((((int64_t)n * g.Cin + ci) * g.D + d) * g.H + h) * g.W + w];
        }
      }
    }
  return acc;
}

// op: 0 forward, 1 input gradient, 2 weight gradient.  Whole output (n_idx == 0) or the listed flat
// indices of it; returns the number of results outside int32.
int64_t dai8o_conv3_acc(int op, const int8_t* A, const int8_t* B, const int* geom, const int64_t* idx, int64_t n_idx,
                        int64_t* acc) {
  Geom3 g;
  std::memcpy(&g, geom, sizeof(Geom3));
  const int Do = out_extent(g.D, g.pad_d, g.T, g.stride_d);
  const int P = out_extent(g.H, g.pad_h, g.R, g.stride_h);
  const int Q = out_extent(g.W, g.pad_w, g.S, g.stride_w);
  const int cpg = g.Cin / g.groups;
  const int64_t full = op == 0 ? (int64_t)g.N * g.Cout * Do * P * Q
                               : (op == 1 ? (int64_t)g.N * g.Cin * g.D * g.H * g.W : (int64_t)g.Cout * cpg * g.T * g.R * g.S);
  const int64_t total = n_idx > 0 ? n_idx : full;
  int64_t overflow = 0;
#pragma omp parallel for schedule(dynamic, 64) reduction(+ : overflow)
  for (int64_t i = 0; i < total; ++i) {
    int64_t f = n_idx > 0 ? idx[i] : i;
    int64_t a;
    if (op == 0) {
      const int q = (int)(f % Q); f /= Q;
      const int p = (int)(f % P); f /= P;
      const int od = (int)(f % Do); f /= Do;
      const int co = (int)(f % g.Cout);
      a = fwd3_at(A, B, g, (int)(f / g.Cout), co, od, p, q);
    } else if (op == 1) {
      const int w = (int)(f % g.W); f /= g.W;
      const int h = (int)(f % g.H); f /= g.H;
      const int d = (int)(f % g.D); f /= g.D;
      const int ci = (int)(f % g.Cin);
      a = bwd_data3_at(A, B, g, Do, P, Q, (int)(f / g.Cin), ci, d, h, w);
    } else {
      const int s = (int)(f % g.S); f /= g.S;
      const int r = (int)(f % g.R); f /= g.R;
      const int t = (int)(f % g.T); f /= g.T;
      const int cl = (int)(f % cpg);
      a = bwd_filter3_at(A, B, g, Do, P, Q, (int)(f / cpg), cl, t, r, s);
    }
    acc[i] = a;
    if (a > INT32_MAX || a < INT32_MIN) ++overflow;
  }
  return overflow;
}

// ---------------------------------------------------------------------------------------------
// De-quantization of an accumulator (Sec. 3.2, the vectorized de-quantization, and Algorithm 1
// final two steps, with the scales the equations imply: s_X for G_W, s_W for G_X).
//   out = (float)acc * ((sa / 127) * (sb / 127)), the scale product formed in binary32.
// rows x cols accumulators; sb is per row (per_row != 0: sb[rows]) or a single value.
// ---------------------------------------------------------------------------------------------
void dai8o_dequant_acc(const int64_t* acc, int64_t rows, int64_t cols, float sa, const float* sb,
                       int per_row, float* out) {
  for (int64_t r = 0; r < rows; ++r) {
    const float b = per_row ? sb[r] : sb[0];
    volatile float fa = sa / 127.0f;
    volatile float fb = b / 127.0f;
    const float scale = fa * fb;
    for (int64_t c = 0; c < cols; ++c) out[r * cols + c] = (float)acc[r * cols + c] * scale;
  }
}

}  // extern "C"
