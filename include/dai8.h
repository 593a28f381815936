/* dai8 -- Distribution Adaptive INT8 quantization of the convolution backward pass, for B200
 * (sm_100a).  C ABI of libdai8.so.
 *
 * The library implements one training step of one convolution layer as the paper defines it:
 *
 *   forward   q(X), q(W) with layer-wide scales and nearest rounding (Sec. 3, Eq. 1; Fig. 2)
 *             Y = (q(X) * q(W)) . (s_X/127)(s_W/127)                       -> dai8_conv_fwd
 *   backward  Algorithm 1: per-channel |g|max and sigma of dY, density P(|g| > sigma), the
 *             discriminator (Eq. 15), the clip rule (Eq. 11 / Eq. 14), per-channel codes vq(dY)
 *             and layer-wide codes q(dY) with stochastic rounding        -> dai8_quantize_grad
 *             G_W = q(X') (x) vq(G'), de-quantized per output channel (Eq. 4-7)
 *                                                                        -> dai8_conv_bwd_filter
 *             G_X = q(G) (.) q(W), de-quantized with |g|max and s_W (Eq. 3)
 *                                                                        -> dai8_conv_bwd_data
 *
 * General rules
 *   - Every pointer is DEVICE memory owned by the caller unless its comment says "host".
 *     All device pointers must be 16-byte aligned.
 *   - The library allocates nothing, never synchronises the stream (except
 *     dai8_get_device_status) and never copies a scale to the host: each call only enqueues
 *     work on `stream` (a cudaStream_t passed as void*; NULL = the legacy default stream).
 *   - Scratch memory is passed in (`ws`, `ws_bytes`); ask dai8_*_workspace_bytes for the size.
 *     Its contents are undefined between calls.  Calls that share a workspace must be ordered
 *     on one stream.
 *   - Work enqueued on one stream takes effect in order, as usual.  Most kernels are launched as
 *     programmatic dependents of the kernel before them on the stream: their set-up may run while
 *     that kernel finishes, but they touch global memory only after it has completed.
 *   - Errors are return codes; arguments are checked on the host before anything is enqueued.
 *     A geometry the kernels do not cover returns DAI8_ERR_UNSUPPORTED: there is no CPU path.
 *   - Device-side waits are bounded.  A wait that runs out records DAI8_ERR_TIMEOUT in a device
 *     status word that dai8_get_device_status reads; the affected output is then undefined.
 *
 * Code tensors (int8, values in [-127, 127])
 *   - activations / gradients:  [N][H][W][Cp]       Cp = C rounded up to a multiple of 16
 *   - weights:                  [Cout][R][S][Cinp]  Cinp = Cin rounded up to a multiple of 16
 *   The padding channels hold code 0.  dai8_quantize_tensor produces the weight layout when the
 *   weights are passed as an NCHW tensor with N=Cout, C=Cin, H=R, W=S.
 */
#ifndef DAI8_H
#define DAI8_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  DAI8_OK = 0,
  DAI8_ERR_INVALID_ARG = 1, /* null / misaligned pointer, non-positive size, bad enum        */
  DAI8_ERR_UNSUPPORTED = 2, /* valid request outside what the kernels implement               */
  DAI8_ERR_WORKSPACE = 3,   /* ws_bytes smaller than dai8_*_workspace_bytes reports           */
  DAI8_ERR_ARCH = 4,        /* current device is not compute capability 10.x                  */
  DAI8_ERR_CUDA = 5,        /* a CUDA runtime / driver call failed                            */
  DAI8_ERR_TIMEOUT = 6      /* a bounded device-side wait expired (device status word)        */
} dai8_status;

typedef enum { DAI8_F32 = 0, DAI8_BF16 = 1, DAI8_I32 = 2 } dai8_dtype; /* I32: raw accumulators */
typedef enum { DAI8_NCHW = 0, DAI8_NHWC = 1 } dai8_layout;
typedef enum { DAI8_ROUND_NEAREST_EVEN = 0, DAI8_ROUND_STOCHASTIC = 1 } dai8_round;
typedef enum { DAI8_SCALE_ABSMAX = 0, DAI8_SCALE_GIVEN = 1 } dai8_scale_mode;

/* Convolution geometry: X (N,Cin,H,W), W (Cout,Cin,R,S), Y (N,Cout,P,Q) with
 * P = (H + 2*pad_h - R)/stride_h + 1, Q likewise (Sec. 3.2).  Cross-correlation, dilation 1,
 * one group. */
typedef struct {
  int N, Cin, Cout, H, W, R, S, stride_h, stride_w, pad_h, pad_w;
} dai8_conv_geom;

/* Which quantization strategy dai8_quantize_grad applies to the per-channel codes `vq` (the rows of
 * the ablation study, Sec. 4.1; the layer-wide codes `gq` always use |g|max of the layer):
 *   FULL       the method: per-channel statistics, discriminator (Eq. 15), clip rule (Eq. 11 / 14)
 *   GQ         global quantization, the ablation baseline: one scale |g|max of the layer for every channel
 *   GVQ_MAX    "Ours_GVQ": per-channel |g|max, no discriminator, no clipping
 *   LAYER_MCS  "Ours_MCS": Eq. 15 and Eq. 14 on the statistics of the whole layer, one clip value for
 *              every channel (s_state[c] all equal; s_state[0] is the state that is read back) */
typedef enum { DAI8_GRAD_FULL = 0, DAI8_GRAD_GQ = 1, DAI8_GRAD_GVQ_MAX = 2, DAI8_GRAD_LAYER_MCS = 3 } dai8_grad_mode;

/* Hyper-parameters of the Magnitude-aware Clipping Strategy.  Paper values: lambda = 0.3
 * (Eq. 15), k = 1, A = 0.8 (Sec. 4.1).  sigma is the population standard deviation about the
 * channel mean unless std_unbiased (divide by M-1) or center_mean = 0 (root mean square).
 * mode: a dai8_grad_mode, DAI8_GRAD_FULL by default. */
typedef struct {
  float lambda, k, A;
  int std_unbiased;
  int center_mean;
  int mode;
} dai8_mcs_params;

/* Rows of the `stats` output of dai8_quantize_grad: stats[c*4 + i]. */
enum { DAI8_STAT_ABSMAX = 0, DAI8_STAT_MEAN = 1, DAI8_STAT_SIGMA = 2, DAI8_STAT_P = 3 };

const char* dai8_status_string(dai8_status s);

/* Fills *p with the paper's hyper-parameters (host pointer). */
void dai8_mcs_defaults(dai8_mcs_params* p);

/* Number of channels of a code tensor holding C logical channels (C rounded up to 16). */
int dai8_padded_channels(int C);

/* ----------------------------------------------------------------------------------------------
 * dai8_quantize_tensor -- Eq. 1 with one scale for the whole tensor (forward quantization of X
 * and W, Fig. 2; also usable for layer-wide gradient codes).
 *   x          input, N*C*H*W elements of `dtype` (F32 or BF16) in `layout`
 *   scale_mode ABSMAX: *scale is written with max|x| and then used; GIVEN: *scale is read
 *   scale      device, 1 float
 *   round      nearest-even (weights, activations) or stochastic (gradients); the stochastic
 *              mode draws u from a counter-based hash of (seed, stream 0, NCHW index)
 *   q          out, int8 [N][H][W][Cp]; padding channels are written with 0
 *   ws         scratch of dai8_quantize_tensor_workspace_bytes() bytes, or NULL.  With scratch, a
 *              tensor whose codes have the layout of its values (NHWC, C a multiple of 16) and
 *              which fits into the shared memory of the whole GPU (about 30 MB) gets its scale and
 *              its codes from ONE launch that reads it from DRAM once; larger tensors, other
 *              layouts and ws == NULL take two launches (scale, then codes).  The results are
 *              identical.  A non-NULL ws that is too small returns DAI8_ERR_WORKSPACE.
 * q(x) = round(clamp(x*(127/s), -127, 127)); s <= 0 gives all-zero codes.
 * -------------------------------------------------------------------------------------------- */
size_t dai8_quantize_tensor_workspace_bytes(void);

dai8_status dai8_quantize_tensor(const void* x, dai8_dtype dtype, dai8_layout layout, int N, int C,
                                 int H, int W, dai8_scale_mode scale_mode, float* scale,
                                 dai8_round round, uint32_t seed, int8_t* q, void* ws,
                                 size_t ws_bytes, void* stream);

/* ----------------------------------------------------------------------------------------------
 * dai8_quantize_grad -- Algorithm 1, the quantization half: Gradient Vectorized Quantization with the
 * Magnitude-aware Clipping Strategy.
 *   dY         gradient of the layer output, (N,C,H,W) elements of `dtype` in `layout`
 *              (C = Cout, H x W = output extent)
 *   params     host pointer; NULL = paper defaults
 *   s_state    device [C]: in  s_{c,t-1} (read only if has_prev != 0; otherwise s_{c,t-1} is
 *              taken as |g|max,c), out s_{c,t} -- the per-channel clip values used for `vq`
 *   gmax_layer device [1], out: |g|max of the layer, the scale of `gq`
 *   stats      device [C][4] or NULL, out: |g|max,c, mean, sigma, P = #{|g|>sigma}/M (per channel; in
 *              mode LAYER_MCS mean, sigma and P of every row are those of the whole layer)
 *   cls        device [C] or NULL, out: 1 = bell-shaped (P > lambda), 0 = Inverted-T.  When has_prev
 *              != 0 its previous contents are read as a hint (the classes of the last iteration):
 *              the fused kernel writes the codes while it counts, with the clip value of the hinted
 *              class, and redoes only the channels whose class turned out different.  The hint
 *              affects speed only, never a result.
 *   vq         out, int8 [N][H][W][Cp]: per-channel codes (for dai8_conv_bwd_filter)
 *   gq         out or NULL, int8 [N][H][W][Cp]: layer-wide codes (for dai8_conv_bwd_data)
 *   seed       stochastic-rounding seed; vq uses stream 0, gq stream 1 of the generator
 *   sigma_override  device [C] or NULL: when given, the density count uses these values instead
 *              of the sigma computed from dY (lets a checker feed identical sigma to both sides)
 * Workspace: dai8_quantize_grad_workspace_bytes(C).
 * -------------------------------------------------------------------------------------------- */
size_t dai8_quantize_grad_workspace_bytes(int C);

dai8_status dai8_quantize_grad(const void* dY, dai8_dtype dtype, dai8_layout layout, int N, int C,
                               int H, int W, const dai8_mcs_params* params, float* s_state,
                               int has_prev, float* gmax_layer, float* stats, uint8_t* cls,
                               int8_t* vq, int8_t* gq, uint32_t seed,
                               const float* sigma_override, void* ws, size_t ws_bytes,
                               void* stream);

/* ----------------------------------------------------------------------------------------------
 * dai8_quantize_grad_noalloc -- dai8_quantize_grad for callers that cannot provide scratch memory.
 * (The paper has no counterpart: this is a property of the library's interface, not of the
 * method.)  Same arguments and results as dai8_quantize_grad without `ws`, `ws_bytes` and
 * `sigma_override`; the reduction scratch is a 3 MiB array built into the library image.
 *
 * Meant for code that cannot allocate on the device when it runs: an extension that a host
 * framework hands nothing but its input and output tensors, a process whose device memory was
 * divided up completely at start-up, a loop that cannot afford the device-wide stall of an
 * allocation.  The caller still owns every input and output.
 *
 *   - C must not exceed DAI8_NOALLOC_MAX_CHANNELS; larger C returns DAI8_ERR_WORKSPACE (the
 *     built-in scratch is too small) and nothing is enqueued.
 *   - The array occupies 3 MiB on every GPU that has loaded the library, until the process exits.
 *   - All calls on one device share the array.  Calls that may overlap on the GPU (different
 *     streams without a dependency between them) race on it: order them.  No call depends on what
 *     the previous one left there.
 *   - The first call on each device looks up the array's device address (a host-side set-up
 *     step): make that first call outside any stream capture.
 *   - It calls no allocation routine of CUDA or of any other library.
 * -------------------------------------------------------------------------------------------- */
#define DAI8_NOALLOC_MAX_CHANNELS 256

dai8_status dai8_quantize_grad_noalloc(const void* dY, dai8_dtype dtype, dai8_layout layout, int N,
                                       int C, int H, int W, const dai8_mcs_params* params,
                                       float* s_state, int has_prev, float* gmax_layer,
                                       float* stats, uint8_t* cls, int8_t* vq, int8_t* gq,
                                       uint32_t seed, void* stream);

/* ----------------------------------------------------------------------------------------------
 * Convolutions on int8 codes with int32 accumulation and a de-quantizing epilogue.
 *
 * dai8_conv_fwd        Y[n,co,p,q]   = acc . ((sX/127)(sW/127)),
 *                      acc = sum_{ci,r,s} qX[n,p*st+r-pad,q*st+s-pad,ci] qW[co,r,s,ci]   (Fig. 2)
 * dai8_conv_bwd_data   dX[n,ci,h,w]  = acc . ((gmax/127)(sW/127)),
 *                      acc = sum over (co,r,s,p,q) with h=p*st+r-pad, w=q*st+s-pad of
 *                      gq[n,p,q,co] qW[co,r,s,ci]                      (Eq. 3; Algorithm 1)
 * dai8_conv_bwd_filter dW[co,ci,r,s] = acc . ((sX/127)(s[co]/127)),
 *                      acc = sum_{n,p,q} vq[n,p,q,co] qX[n,p*st+r-pad,q*st+s-pad,ci]
 *                                                                      (Eq. 4-7; Algorithm 1)
 *   sX, sW, gmax   device, 1 float each;  s: device [Cout] (the s_state of dai8_quantize_grad)
 *   out_dtype      F32 or BF16 (de-quantized), or I32: the raw accumulators, scales ignored
 *   out_layout     NCHW or NHWC for Y / dX (C unpadded); dW is always (Cout,Cin,R,S)
 * Accumulators are int32 and wrap on overflow (possible only for K*127^2 > 2^31, far beyond
 * what zero-mean gradients reach).  Workspace: dai8_conv_workspace_bytes(op, geom).
 * -------------------------------------------------------------------------------------------- */
typedef enum { DAI8_OP_FWD = 0, DAI8_OP_BWD_DATA = 1, DAI8_OP_BWD_FILTER = 2 } dai8_conv_op;

size_t dai8_conv_workspace_bytes(dai8_conv_op op, const dai8_conv_geom* geom /* host */);

dai8_status dai8_conv_fwd(const int8_t* qX, const int8_t* qW, const float* sX, const float* sW,
                          const dai8_conv_geom* geom /* host */, void* Y, dai8_dtype out_dtype,
                          dai8_layout out_layout, void* ws, size_t ws_bytes, void* stream);

dai8_status dai8_conv_bwd_data(const int8_t* gq, const int8_t* qW, const float* gmax,
                               const float* sW, const dai8_conv_geom* geom /* host */, void* dX,
                               dai8_dtype out_dtype, dai8_layout out_layout, void* ws,
                               size_t ws_bytes, void* stream);

dai8_status dai8_conv_bwd_filter(const int8_t* qX, const int8_t* vq, const float* sX,
                                 const float* s, const dai8_conv_geom* geom /* host */, void* dW,
                                 dai8_dtype out_dtype, void* ws, size_t ws_bytes, void* stream);

/* ----------------------------------------------------------------------------------------------
 * The same three convolutions with a depth dimension and channel groups: 3-D convolution, "treating
 * depth dimension in the same way as height and width" (Sec. 4.4), and depth-wise convolution
 * (groups = Cin = Cout; the MobileNetV2 paragraph of Sec. 4.2).  Arithmetic as above (int8 codes,
 * wrapping int32 accumulators, de-quantization by the two scales); CUDA-core kernels for every
 * geometry with T*R*S <= 32 taps, no workspace.
 *   X (N,Cin,D,H,W), W (Cout,Cin/groups,T,R,S), Y (N,Cout,Do,P,Q); groups 0 or 1 = one group; with
 *   several groups the channels per group must be 1 or a multiple of 4
 *   codes: activations / gradients [N][D][H][W][Cp]; weights [Cout][T][R][S][Cgp], Cgp = Cin/groups
 *   rounded up to 16 -- i.e. dai8_quantize_tensor of the (N, C, D*H, W) tensor, and of the weights
 *   passed as an NCHW tensor with N = Cout, C = Cin/groups, H = T*R, W = S.  The gradient quantizer
 *   takes a 5-D gradient the same way, as (N, C, Do*P, Q): its statistics run over everything but
 *   the channel, and its random numbers follow the flat index, which is the same.
 *   outputs: channels last, unpadded: Y [N][Do][P][Q][Cout], dX [N][D][H][W][Cin] (F32, BF16 or
 *   I32 = raw accumulators); dW (Cout,Cin/groups,T,R,S) F32 or I32.
 * -------------------------------------------------------------------------------------------- */
typedef struct {
  int N, Cin, Cout, D, H, W, T, R, S, stride_d, stride_h, stride_w, pad_d, pad_h, pad_w, groups;
} dai8_conv3d_geom;

dai8_status dai8_conv3d_fwd(const int8_t* qX, const int8_t* qW, const float* sX, const float* sW,
                            const dai8_conv3d_geom* geom /* host */, void* Y, dai8_dtype out_dtype,
                            void* stream);
dai8_status dai8_conv3d_bwd_data(const int8_t* gq, const int8_t* qW, const float* gmax,
                                 const float* sW, const dai8_conv3d_geom* geom /* host */, void* dX,
                                 dai8_dtype out_dtype, void* stream);
dai8_status dai8_conv3d_bwd_filter(const int8_t* qX, const int8_t* vq, const float* sX,
                                   const float* s, const dai8_conv3d_geom* geom /* host */, void* dW,
                                   dai8_dtype out_dtype, void* stream);

/* ----------------------------------------------------------------------------------------------
 * Batch-sharded (data-parallel) operation: every rank holds N_local of the batch's images.  The
 * statistics, the density count, the classes and the clip values of Algorithm 1 belong to the WHOLE
 * batch, so the gradient quantizer is split into stages between which the caller exchanges
 * per-channel scalars among the ranks (any collective library; none is called here):
 *
 *   dai8_dp_grad_pivot     pivot[C] = the channel values of the shard's first pixel
 *        exchange          pivot: broadcast from one rank
 *   dai8_dp_grad_moments   local |g|max[C] and sums[2][C] = sum (g - pivot_c), sum (g - pivot_c)^2 over
 *                          the rank's pixels; pivot[C] must be the same on all ranks (e.g. pixel 0 of
 *                          rank 0's shard, broadcast): it keeps the second moment free of cancellation
 *        exchange          absmax: maximum over ranks; sums: sum over ranks
 *   dai8_dp_grad_sigma     mean[C], sigma[C] (Eq. 15's sigma; flags of dai8_mcs_params) and the layer
 *                          |g|max from the exchanged moments, M_global = pixels of the whole batch
 *   dai8_dp_grad_count     local cnt[C] = #{|g| > sigma_c} (64-bit integers, so that any integer
 *                          all-reduce can add them)
 *        exchange          cnt: sum over ranks
 *   dai8_dp_grad_solve     Eq. 15 on cnt / M_global, Eq. 11 / 14: s_state[C] in/out, cls[C] (may be NULL)
 *   dai8_dp_grad_codes     vq (clip values s[C]) and gq (layer |g|max; may be NULL) of the rank's images,
 *                          stochastic rounding; first_image = index of the rank's first image in the
 *                          whole batch: the random numbers follow the element's index there, so the
 *                          codes equal those dai8_quantize_grad writes for the same images of the
 *                          unsharded tensor
 *
 * NHWC only (DAI8_ERR_UNSUPPORTED otherwise); ws: dai8_dp_grad_workspace_bytes(C) bytes, 16-byte
 * aligned; everything else as for dai8_quantize_grad.  mode must be DAI8_GRAD_FULL in dai8_dp_grad_solve.
 *
 * The rest of a sharded layer step uses the ordinary entry points: dai8_absmax gives the local
 * max|x| (exchange: maximum) for dai8_quantize_tensor with DAI8_SCALE_GIVEN; dai8_conv_bwd_filter
 * with DAI8_I32 output gives the rank's integer partial of dW (exchange: integer sum, exact), and
 * dai8_dequant_filter applies Eq. 7 to the sum: dW[co][...] = acc * (sX/127) * (s[co]/127), per_cout =
 * Cin*R*S values per output channel.
 * -------------------------------------------------------------------------------------------- */
size_t dai8_dp_grad_workspace_bytes(int C);
dai8_status dai8_dp_grad_pivot(const void* dY, dai8_dtype dtype, dai8_layout layout, int C, float* pivot,
                               void* stream);
dai8_status dai8_dp_grad_moments(const void* dY, dai8_dtype dtype, dai8_layout layout, int N_local, int C,
                                 int H, int W, const float* pivot, float* absmax, double* sums, void* ws,
                                 size_t ws_bytes, void* stream);
dai8_status dai8_dp_grad_sigma(const float* absmax, const double* sums, const float* pivot, int C,
                               int64_t M_global, const dai8_mcs_params* params /* host, may be NULL */,
                               float* mean, float* sigma, float* gmax_layer, void* stream);
dai8_status dai8_dp_grad_count(const void* dY, dai8_dtype dtype, dai8_layout layout, int N_local, int C, int H,
                               int W, const float* sigma, long long* cnt, void* ws, size_t ws_bytes,
                               void* stream);
dai8_status dai8_dp_grad_solve(const long long* cnt, const float* absmax, int C, int64_t M_global,
                               const dai8_mcs_params* params /* host, may be NULL */, float* s_state,
                               int has_prev, uint8_t* cls, void* stream);
dai8_status dai8_dp_grad_codes(const void* dY, dai8_dtype dtype, dai8_layout layout, int N_local, int C, int H,
                               int W, int64_t first_image, const float* s, const float* gmax_layer,
                               uint32_t seed, int8_t* vq, int8_t* gq, void* stream);
dai8_status dai8_absmax(const void* x, dai8_dtype dtype, int64_t count, float* out, void* stream);
dai8_status dai8_dequant_filter(const int32_t* acc, const float* sX, const float* s, int Cout,
                                int64_t per_cout, float* dW, void* stream);

/* Kernel family selection for the convolutions (process-wide, host side): 0 = automatic
 * (tensor-core kernels where the geometry allows, direct kernels otherwise), 1 = direct kernels
 * only, 2 = tensor-core kernels only (DAI8_ERR_UNSUPPORTED where they do not apply), 3 = like 2 but
 * multi-tap filters use the copy engine's im2col loads even where the patch form applies.  Used
 * by the tests to compare the kernel families bit for bit. */
void dai8_set_conv_backend(int mode);

/* Number of kernels the library has launched from this process so far (host counter). */
uint64_t dai8_launch_count(void);

/* Reads and clears the device status word (DAI8_OK or DAI8_ERR_TIMEOUT).  Synchronises `stream`.
 * host_status: host pointer. */
dai8_status dai8_get_device_status(int* host_status, void* stream);

/* Self-test of the give-up path of the bounded device-side waits.  Runs the library's own wait
 * helpers (the mbarrier wait and the grid barrier of the gradient quantizer, the mbarrier wait of the
 * convolution kernels) on barriers that nobody completes, with nothing in flight and a limit of
 * `limit_cycles` SM cycles (1 .. 1e8) instead of the usual second.  Every wait must return by
 * itself: report[0..2] (host, 3 ints) get 1 for each wait that gave up, and the device status word
 * then holds DAI8_ERR_TIMEOUT until dai8_get_device_status reads and clears it.  The kernels end
 * normally, so the context stays usable.  ws: 32 bytes of device scratch.  Synchronises `stream`. */
dai8_status dai8_debug_expire_waits(uint64_t limit_cycles, int* report /* host */, void* ws,
                                    size_t ws_bytes, void* stream);

/* Name of the kernel (family) that the calling thread's most recent entry-point call launched, e.g.
 * "igemm_halo_kernel" -- for harnesses that attribute device time to kernels.  Host only; the string is
 * static.  "" before the first call. */
const char* dai8_debug_last_kernel(void);

/* Two micro-measurements behind the library's tiling decisions (`python bench.py --probe`).  Both
 * synchronise `stream`; ws: 32 bytes of device scratch.
 *   dai8_debug_probe_mma  cycles per tcgen05.mma.kind::i8 of M = 128, K = 32 and `n_cols` (16..256,
 *       multiple of 16) accumulator columns, operands resident in shared memory in rows of `row_bytes`
 *       (32, 64, 128), `count` (multiple of 4) instructions issued back to back on every SM:
 *       *issue_cycles until the last issue returned, *complete_cycles until the last one finished,
 *       both divided by count (host pointers).
 *   dai8_debug_probe_sr   elements per second (host pointer) of the code sweep's per-element
 *       arithmetic (index hash, two uniforms, two stochastic roundings, packing) on values held in
 *       registers, `iters` vectors of 8 elements per thread, whole GPU. */
dai8_status dai8_debug_probe_mma(int n_cols, int row_bytes, int count, double* issue_cycles,
                                 double* complete_cycles, void* ws, size_t ws_bytes, void* stream);
dai8_status dai8_debug_probe_sr(int iters, double* elements_per_second, void* ws, size_t ws_bytes,
                                void* stream);

#ifdef __cplusplus
}
#endif
#endif /* DAI8_H */
