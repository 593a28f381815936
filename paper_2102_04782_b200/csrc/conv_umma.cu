// Tensor-core (tcgen05) convolution kernels.  Placeholder: nothing is routed here yet.
#include "conv_internal.cuh"

namespace dai8 {

__device__ unsigned int g_device_status = 0;

dai8_status read_clear_device_status(int* host_status, cudaStream_t stream) {
  unsigned int v = 0, zero = 0;
  DAI8_RETURN_IF_CUDA(cudaMemcpyFromSymbolAsync(&v, g_device_status, sizeof(v), 0, cudaMemcpyDeviceToHost, stream));
  DAI8_RETURN_IF_CUDA(cudaMemcpyToSymbolAsync(g_device_status, &zero, sizeof(zero), 0, cudaMemcpyHostToDevice, stream));
  DAI8_RETURN_IF_CUDA(cudaStreamSynchronize(stream));
  *host_status = (int)v;
  return DAI8_OK;
}

bool umma_fwd_supported(const ConvShape&) { return false; }
bool umma_bwd_data_supported(const ConvShape&) { return false; }
bool umma_bwd_filter_supported(const ConvShape&) { return false; }
dai8_status umma_fwd(const int8_t*, const int8_t*, const float*, const float*, const ConvShape&,
                     const ConvOut&, cudaStream_t) { return DAI8_ERR_UNSUPPORTED; }
dai8_status umma_bwd_data(const int8_t*, const int8_t*, const float*, const float*, const ConvShape&,
                          const ConvOut&, cudaStream_t) { return DAI8_ERR_UNSUPPORTED; }
dai8_status umma_bwd_filter_acc(const int8_t*, const int8_t*, const ConvShape&, int*, cudaStream_t) {
  return DAI8_ERR_UNSUPPORTED;
}

}  // namespace dai8
