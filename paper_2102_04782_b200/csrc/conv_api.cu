// C-ABI entry points of the convolutions: argument checks, workspace carving, kernel-family choice.
#include "conv_internal.cuh"

namespace dai8 {
namespace {

std::atomic<int> g_backend{0};  // 0 auto, 1 direct only, 2 tensor-core only

dai8_status check_geom(const dai8_conv_geom* g) {
  if (!g) return DAI8_ERR_INVALID_ARG;
  if (g->N <= 0 || g->Cin <= 0 || g->Cout <= 0 || g->H <= 0 || g->W <= 0 || g->R <= 0 || g->S <= 0 ||
      g->stride_h <= 0 || g->stride_w <= 0 || g->pad_h < 0 || g->pad_w < 0)
    return DAI8_ERR_INVALID_ARG;
  if (g->H + 2 * g->pad_h < g->R || g->W + 2 * g->pad_w < g->S) return DAI8_ERR_INVALID_ARG;
  const ConvShape cs = make_shape(*g);
  const int64_t lim = (int64_t)1 << 31;
  if ((int64_t)g->N * cs.P * cs.Q >= lim || (int64_t)g->N * g->H * g->W >= lim) return DAI8_ERR_UNSUPPORTED;
  return DAI8_OK;
}

bool bad_out(dai8_dtype t) { return t != DAI8_F32 && t != DAI8_BF16 && t != DAI8_I32; }
bool bad_layout(dai8_layout l) { return l != DAI8_NCHW && l != DAI8_NHWC; }

size_t wt_bytes(const ConvShape& cs) { return (size_t)cs.Cinp * cs.R * cs.S * cs.Coutp; }
size_t dw_acc_bytes(const ConvShape& cs) { return (size_t)cs.Coutp * cs.R * cs.S * cs.Cinp * sizeof(int); }
size_t up256(size_t b) { return (b + 255) / 256 * 256; }

// Packed pointwise form of a layer with at most 16 input channels, if the tensor-core kernels take it.
int packed_fwd(const ConvShape& cs, ConvShape* pw) {
  ConvShape tmp;
  const int Kp = packed_small_cin(cs, &tmp);
  if (Kp == 0 || !umma_fwd_supported(tmp)) return 0;
  if (pw) *pw = tmp;
  return Kp;
}
int packed_bwd_filter(const ConvShape& cs, ConvShape* pw) {
  ConvShape tmp;
  const int Kp = packed_small_cin(cs, &tmp);
  if (Kp == 0 || !umma_bwd_filter_supported(tmp)) return 0;
  if (pw) *pw = tmp;
  return Kp;
}
size_t packed_a_bytes(const ConvShape& cs, int Kp) { return up256((size_t)cs.N * cs.P * cs.Q * Kp); }

// The input gradient of a stride-1 layer is the forward convolution of the gradient codes with the
// mirrored, transposed filter.  With at most 16 output channels that forward problem has "few input
// channels" and can take the packed pointwise route on the tensor cores.  Returns Kp (0: not applicable).
int packed_bwd_data(const ConvShape& cs, ConvShape* as_fwd, ConvShape* pw) {
  if (cs.Coutp != 16 || cs.sh != 1 || cs.sw != 1 || cs.ph > cs.R - 1 || cs.pw > cs.S - 1) return 0;
  ConvShape f = cs;
  f.Cin = cs.Cout; f.Cout = cs.Cin; f.Cinp = cs.Coutp; f.Coutp = cs.Cinp;
  f.H = cs.P; f.W = cs.Q; f.P = cs.H; f.Q = cs.W;
  f.ph = cs.R - 1 - cs.ph; f.pw = cs.S - 1 - cs.pw;
  ConvShape tmp;
  const int Kp = packed_fwd(f, &tmp);
  if (Kp == 0) return 0;
  if (as_fwd) *as_fwd = f;
  if (pw) *pw = tmp;
  return Kp;
}

}  // namespace
}  // namespace dai8

using namespace dai8;

extern "C" void dai8_set_conv_backend(int mode) {
  if (mode < 0 || mode > 3) mode = 0;
  set_halo_disabled(mode == 3);
  g_backend.store(mode == 3 ? 2 : mode);
}

extern "C" size_t dai8_conv_workspace_bytes(dai8_conv_op op, const dai8_conv_geom* geom) {
  if (check_geom(geom) != DAI8_OK) return 0;
  const ConvShape cs = make_shape(*geom);
  switch (op) {
    case DAI8_OP_FWD: {
      const int Kp = umma_fwd_supported(cs) ? 0 : packed_fwd(cs, nullptr);
      return Kp ? packed_a_bytes(cs, Kp) + up256((size_t)cs.Coutp * Kp) + 256 : 256;
    }
    case DAI8_OP_BWD_DATA: {
      ConvShape f;
      const int Kp = umma_bwd_data_supported(cs) ? 0 : packed_bwd_data(cs, &f, nullptr);
      return up256(wt_bytes(cs)) + (Kp ? packed_a_bytes(f, Kp) + up256((size_t)f.Coutp * Kp) : 0) + 256;
    }
    case DAI8_OP_BWD_FILTER: {
      // one int32 image, or one per pixel slice of the tensor-core kernel
      ConvShape pw;
      const int Kp = umma_bwd_filter_supported(cs) ? 0 : packed_bwd_filter(cs, &pw);
      if (Kp) return up256(dw_acc_bytes(pw) * (size_t)umma_bwd_filter_splits(pw)) + packed_a_bytes(cs, Kp) + 256;
      const int splits = umma_bwd_filter_splits(cs);
      return (dw_acc_bytes(cs) * (size_t)(splits > 1 ? splits : 1) + 255) / 256 * 256 + 256;
    }
  }
  return 0;
}

extern "C" dai8_status dai8_conv_fwd(const int8_t* qX, const int8_t* qW, const float* sX, const float* sW,
                                     const dai8_conv_geom* geom, void* Y, dai8_dtype out_dtype,
                                     dai8_layout out_layout, void* ws, size_t ws_bytes, void* stream) {
  dai8_status g = check_geom(geom);
  if (g != DAI8_OK) return g;
  if (!qX || !qW || !Y || bad_out(out_dtype) || bad_layout(out_layout)) return DAI8_ERR_INVALID_ARG;
  if (out_dtype != DAI8_I32 && (!sX || !sW)) return DAI8_ERR_INVALID_ARG;
  if (!aligned16(qX) || !aligned16(qW) || !aligned16(Y)) return DAI8_ERR_INVALID_ARG;
  dai8_status a = check_device_arch();
  if (a != DAI8_OK) return a;
  const ConvShape cs = make_shape(*geom);
  const ConvOut out{Y, out_dtype, out_layout};
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int mode = g_backend.load();
  if (mode != 1 && umma_fwd_supported(cs)) return umma_fwd(qX, qW, sX, sW, cs, out, st);
  ConvShape pw;
  const int Kp = mode != 1 ? packed_fwd(cs, &pw) : 0;
  if (Kp && ws && aligned16(ws) && ws_bytes >= dai8_conv_workspace_bytes(DAI8_OP_FWD, geom)) {
    // few input channels: gather the real channels of all taps, then a pointwise convolution
    int8_t* A = static_cast<int8_t*>(ws);
    int8_t* Wp = A + packed_a_bytes(cs, Kp);
    dai8_status r = pack_small_cin(qX, cs, Kp, A, st);
    if (r == DAI8_OK) r = pack_small_cin_weights(qW, cs, Kp, Wp, st);
    if (r != DAI8_OK) return r;
    r = umma_fwd(A, Wp, sX, sW, pw, out, st);
    note_kernel("pack_small_cin_kernel + igemm_kmajor_kernel");
    return r;
  }
  if (mode == 2) return Kp ? DAI8_ERR_WORKSPACE : DAI8_ERR_UNSUPPORTED;
  note_kernel("direct_fwd_kernel");
  log_choice("conv_fwd: direct kernel");
  return direct_fwd(qX, qW, sX, sW, cs, out, st);
}

extern "C" dai8_status dai8_conv_bwd_data(const int8_t* gq, const int8_t* qW, const float* gmax,
                                          const float* sW, const dai8_conv_geom* geom, void* dX,
                                          dai8_dtype out_dtype, dai8_layout out_layout, void* ws,
                                          size_t ws_bytes, void* stream) {
  dai8_status g = check_geom(geom);
  if (g != DAI8_OK) return g;
  if (!gq || !qW || !dX || !ws || bad_out(out_dtype) || bad_layout(out_layout)) return DAI8_ERR_INVALID_ARG;
  if (out_dtype != DAI8_I32 && (!gmax || !sW)) return DAI8_ERR_INVALID_ARG;
  if (!aligned16(gq) || !aligned16(qW) || !aligned16(dX) || !aligned16(ws)) return DAI8_ERR_INVALID_ARG;
  if (ws_bytes < dai8_conv_workspace_bytes(DAI8_OP_BWD_DATA, geom)) return DAI8_ERR_WORKSPACE;
  dai8_status a = check_device_arch();
  if (a != DAI8_OK) return a;
  const ConvShape cs = make_shape(*geom);
  const ConvOut out{dX, out_dtype, out_layout};
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int8_t* wT = static_cast<int8_t*>(ws);
  const int mode = g_backend.load();
  if (mode != 1 && umma_bwd_data_supported(cs)) return umma_bwd_data(gq, qW, wT, gmax, sW, cs, out, st);
  ConvShape f, pw;
  if (const int Kp = mode != 1 ? packed_bwd_data(cs, &f, &pw) : 0) {
    // few output channels: forward form of the input gradient on the packed pointwise route
    int8_t* A = wT + up256(wt_bytes(cs));
    int8_t* Wp = A + packed_a_bytes(f, Kp);
    dai8_status r = repack_weights_transposed(qW, cs, wT, /*flip=*/1, st);   // [Cinp][R][S][Coutp], taps mirrored
    if (r == DAI8_OK) r = pack_small_cin(gq, f, Kp, A, st);
    if (r == DAI8_OK) r = pack_small_cin_weights(wT, f, Kp, Wp, st);
    if (r != DAI8_OK) return r;
    r = umma_fwd(A, Wp, gmax, sW, pw, out, st);
    note_kernel("pack_small_cin_kernel + igemm_kmajor_kernel");
    return r;
  }
  if (mode == 2) return DAI8_ERR_UNSUPPORTED;
  dai8_status r = repack_weights_transposed(qW, cs, wT, /*flip=*/0, st);
  if (r != DAI8_OK) return r;
  note_kernel("direct_bwd_data_kernel");
  log_choice("conv_bwd_data: direct kernel");
  return direct_bwd_data(gq, wT, gmax, sW, cs, out, st);
}

extern "C" dai8_status dai8_conv_bwd_filter(const int8_t* qX, const int8_t* vq, const float* sX,
                                            const float* s, const dai8_conv_geom* geom, void* dW,
                                            dai8_dtype out_dtype, void* ws, size_t ws_bytes,
                                            void* stream) {
  dai8_status g = check_geom(geom);
  if (g != DAI8_OK) return g;
  if (!qX || !vq || !dW || !ws || bad_out(out_dtype)) return DAI8_ERR_INVALID_ARG;
  if (out_dtype != DAI8_I32 && (!sX || !s)) return DAI8_ERR_INVALID_ARG;
  if (!aligned16(qX) || !aligned16(vq) || !aligned16(dW) || !aligned16(ws)) return DAI8_ERR_INVALID_ARG;
  if (ws_bytes < dai8_conv_workspace_bytes(DAI8_OP_BWD_FILTER, geom)) return DAI8_ERR_WORKSPACE;
  dai8_status a = check_device_arch();
  if (a != DAI8_OK) return a;
  const ConvShape cs = make_shape(*geom);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int* acc = static_cast<int*>(ws);
  const int mode = g_backend.load();
  int splits = 1;
  dai8_status r;
  ConvShape pw;
  if (mode != 1 && umma_bwd_filter_supported(cs)) {
    r = umma_bwd_filter_acc(qX, vq, cs, acc, &splits, st);   // every slice writes its whole image
  } else if (const int Kp = mode != 1 ? packed_bwd_filter(cs, &pw) : 0) {
    // few input channels: the weight gradient of the packed pointwise form, unpacked by finalize
    int8_t* A = static_cast<int8_t*>(ws) + up256(dw_acc_bytes(pw) * (size_t)umma_bwd_filter_splits(pw));
    r = pack_small_cin(qX, cs, Kp, A, st);
    if (r == DAI8_OK) r = umma_bwd_filter_acc(A, vq, pw, acc, &splits, st);
    if (r != DAI8_OK) return r;
    note_kernel("pack_small_cin_kernel + wgrad_mnmajor_kernel");
    return finalize_bwd_filter(acc, splits, sX, s, pw, &cs, dW, out_dtype, st);
  } else if (mode == 2) {
    return DAI8_ERR_UNSUPPORTED;
  } else {
    DAI8_RETURN_IF_CUDA(cudaMemsetAsync(acc, 0, dw_acc_bytes(cs), st));
    note_kernel("direct_bwd_filter_kernel");
    log_choice("conv_bwd_filter: direct kernel");
    r = direct_bwd_filter_acc(qX, vq, cs, acc, st);
  }
  if (r != DAI8_OK) return r;
  return finalize_bwd_filter(acc, splits, sX, s, cs, nullptr, dW, out_dtype, st);
}
