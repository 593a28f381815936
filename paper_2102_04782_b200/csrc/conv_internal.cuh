// Interfaces shared by the convolution kernel families and the C-ABI dispatch (conv_api.cu).
#pragma once

#include "dai8_common.cuh"

namespace dai8 {

struct ConvShape {
  int N, Cin, Cout, H, W, R, S, sh, sw, ph, pw;
  int P, Q;        // output extent
  int Cinp, Coutp; // channel counts of the code tensors (multiples of 16)
};

inline ConvShape make_shape(const dai8_conv_geom& g) {
  ConvShape s;
  s.N = g.N; s.Cin = g.Cin; s.Cout = g.Cout; s.H = g.H; s.W = g.W; s.R = g.R; s.S = g.S;
  s.sh = g.stride_h; s.sw = g.stride_w; s.ph = g.pad_h; s.pw = g.pad_w;
  s.P = (g.H + 2 * g.pad_h - g.R) / g.stride_h + 1;
  s.Q = (g.W + 2 * g.pad_w - g.S) / g.stride_w + 1;
  s.Cinp = round_up(g.Cin, 16);
  s.Coutp = round_up(g.Cout, 16);
  return s;
}

struct ConvOut {
  void* ptr;
  dai8_dtype dtype;    // F32, BF16 or I32 (raw accumulators)
  dai8_layout layout;  // NCHW or NHWC (C unpadded)
};

// De-quantization scale (Eq. 7 and the last two steps of Algorithm 1): (a/127)*(b/127), each step rounded.
__device__ __forceinline__ float dequant_scale(float a, float b) {
  return __fmul_rn(__fdiv_rn(a, 127.0f), __fdiv_rn(b, 127.0f));
}

__device__ __forceinline__ uint16_t f32_to_bf16_bits(float f) {
  const uint32_t u = __float_as_uint(f);
  if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x40u);  // NaN
  return (uint16_t)((u + 0x7FFFu + ((u >> 16) & 1u)) >> 16);                  // nearest even
}

// Two fp32 values -> packed bfloat16 pair (lo in bits 0-15), round to nearest even, one instruction.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}

// Writes one output element: the raw accumulator, or float(acc)*scale as fp32 / bf16.
__device__ __forceinline__ void store_result(void* out, dai8_dtype dtype, size_t idx, int acc, float scale) {
  if (dtype == DAI8_I32) {
    static_cast<int*>(out)[idx] = acc;
  } else {
    const float v = __fmul_rn(__int2float_rn(acc), scale);
    if (dtype == DAI8_F32) static_cast<float*>(out)[idx] = v;
    else static_cast<uint16_t*>(out)[idx] = f32_to_bf16_bits(v);
  }
}

// Residue classes of the input gradient (see conv_umma.cu): class (a, b) owns the output pixels with
// h mod stride_h = a, w mod stride_w = b and the filter taps r = r0 + stride_h*j, s = s0 + stride_w*j.
struct DgradClass {
  int a, b, r0, s0, Tr, Ts;      // Tr*Ts taps; 0 when the class has none
  int Ha, Wb;                    // output pixels of the class per image
  int lower_h, lower_w;          // first q(G) row / column read by output (0, 0) of the class
  long long w_off;               // offset of the class's weights [Cinp][Tr][Ts][Coutp] in the repacked buffer
};
struct DgradClasses {
  DgradClass cls[16];
  int n, any_empty;
};

// ---- direct (CUDA-core, dp4a) kernels: every geometry --------------------------------------------
dai8_status direct_fwd(const int8_t* qX, const int8_t* qW, const float* sX, const float* sW,
                       const ConvShape& cs, const ConvOut& out, cudaStream_t st);
// wT: weights repacked as [Cinp][R][S][Coutp] (repack_weights_transposed, flip = 0)
dai8_status direct_bwd_data(const int8_t* gq, const int8_t* wT, const float* gmax, const float* sW,
                            const ConvShape& cs, const ConvOut& out, cudaStream_t st);
// accumulates into acc[Cout][R][S][Cinp] (int32, zeroed by the caller)
dai8_status direct_bwd_filter_acc(const int8_t* qX, const int8_t* vq, const ConvShape& cs, int* acc,
                                  cudaStream_t st);

// [Cout][R][S][Cinp] -> [Cinp][R][S][Coutp]; flip != 0 also mirrors the taps (r,s) -> (R-1-r,S-1-s).
dai8_status repack_weights_transposed(const int8_t* qW, const ConvShape& cs, int8_t* wT, int flip,
                                      cudaStream_t st);
// sum over `splits` partial images acc[split][Cout][R][S][Cinp] -> dW (Cout,Cin,R,S), scaled by
// (sX/127)(s[co]/127) unless dtype is I32.
// With packed_from != nullptr, `cs` is the pointwise form of the layer *packed_from (see
// packed_small_cin) and channel k' of the images is element (ci, r, s) of the real filter.
dai8_status finalize_bwd_filter(const int* acc, int splits, const float* sX, const float* s,
                                const ConvShape& cs, const ConvShape* packed_from, void* dW, dai8_dtype dtype,
                                cudaStream_t st);

// Layers with at most 16 input channels: A'[N*P*Q][Kp] gathers the real channels of all taps
// (k' = (r*S+s)*cc + ci with cc = packed_channels, zero padded to Kp = multiple of 32), W'[Cout][Kp]
// likewise; the layer then
// is a pointwise convolution with Kp input channels.
// Channels per pixel in the gathered matrix: up to four real channels are kept as one 32-bit word
// (the gather then moves whole words), more are kept as they are.
__host__ __device__ inline int packed_channels(const ConvShape& cs) { return cs.Cin <= 4 ? 4 : cs.Cin; }
inline int packed_small_cin(const ConvShape& cs, ConvShape* pw) {
  if (cs.Cinp != 16) return 0;
  const int Kp = round_up(cs.R * cs.S * packed_channels(cs), 32);
  if (Kp > 2048) return 0;
  if (pw) {
    *pw = cs;
    pw->Cin = Kp; pw->Cinp = Kp; pw->H = cs.P; pw->W = cs.Q; pw->R = 1; pw->S = 1;
    pw->sh = 1; pw->sw = 1; pw->ph = 0; pw->pw = 0;
  }
  return Kp;
}
dai8_status pack_small_cin(const int8_t* qX, const ConvShape& cs, int Kp, int8_t* A, cudaStream_t st);
dai8_status pack_small_cin_weights(const int8_t* qW, const ConvShape& cs, int Kp, int8_t* Wp, cudaStream_t st);

// ---- tensor-core kernel for multi-tap filters at stride 1 (conv_halo.cu) --------------------------
// D[n][y][x][j] = sum over taps (r, s) and channels k of A[n][y + r + lower_h][x + s + lower_w][k] * B[j][r*S+s][k]
struct HaloProblem {
  const int8_t* A;   // [N][H][W][Kc] codes
  const int8_t* B;   // K-major [Brows][R*S][Kc], or (b_mn) the forward weights [Bk][b_taps][Brows] read in place
  int N, H, W, Kc, Brows;
  int P, Q, Nout, R, S, lower_h, lower_w;
  int b_mn = 0, Bk = 0, b_taps = 0, b_tap_base = 0, b_tap_dr = 0, b_tap_ds = 0;
};
bool halo_supported(const HaloProblem& pb, dai8_dtype out_dtype, dai8_layout out_layout);
dai8_status launch_halo(const HaloProblem& pb, const float* sa, const float* sb, const ConvOut& out, cudaStream_t st);
// 0: the patch form (conv_halo.cu) wherever it applies; 1: the im2col form only (set by the tests through
// dai8_set_conv_backend to compare the two forms)
void set_halo_disabled(int disabled);

// ---- tensor-core (tcgen05) kernels: see conv_umma.cu for the geometries covered ------------------
bool umma_fwd_supported(const ConvShape& cs);
bool umma_bwd_data_supported(const ConvShape& cs);
bool umma_bwd_filter_supported(const ConvShape& cs);
dai8_status umma_fwd(const int8_t* qX, const int8_t* qW, const float* sX, const float* sW,
                     const ConvShape& cs, const ConvOut& out, cudaStream_t st);
// wT: workspace of Cinp*R*S*Coutp bytes for the class-ordered weights
dai8_status umma_bwd_data(const int8_t* gq, const int8_t* qW, int8_t* wT, const float* gmax, const float* sW,
                          const ConvShape& cs, const ConvOut& out, cudaStream_t st);
// [Cout][R][S][Cinp] -> for every class [Cinp][Tr][Ts][Coutp] with the class's taps mirrored
dai8_status repack_weights_classes(const int8_t* qW, const ConvShape& cs, const DgradClasses& dc, int8_t* wT,
                                   cudaStream_t st);
// writes *splits partial images acc[split][Cout][R][S][Cinp] (no zeroing needed), to be added up by
// finalize_bwd_filter; umma_bwd_filter_splits gives their number for sizing the workspace
dai8_status umma_bwd_filter_acc(const int8_t* qX, const int8_t* vq, const ConvShape& cs, int* acc,
                                int* splits, cudaStream_t st);
int umma_bwd_filter_splits(const ConvShape& cs);

}  // namespace dai8
