// Direct int8 convolutions on the CUDA cores (dp4a).  They cover every geometry the boundary
// accepts (any stride, padding, filter size, channel count) and serve the shapes the tensor-core
// kernels do not take, e.g. 3-channel stems.  Codes are NHWC with channels padded to 16, so every
// operand fetch is one 16-byte load and four dp4a.
#include "conv_internal.cuh"

namespace dai8 {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ int dot16(const uint4& a, const uint4& b, int acc) {
  acc = __dp4a((int)a.x, (int)b.x, acc);
  acc = __dp4a((int)a.y, (int)b.y, acc);
  acc = __dp4a((int)a.z, (int)b.z, acc);
  acc = __dp4a((int)a.w, (int)b.w, acc);
  return acc;
}

// Forward convolution (Fig. 2): thread = (output pixel, output channel), channel fastest.
__global__ void __launch_bounds__(kThreads)
direct_fwd_kernel(const int8_t* __restrict__ qX, const int8_t* __restrict__ qW,
                  const float* __restrict__ sX, const float* __restrict__ sW, ConvShape cs,
                  ConvOut out) {
  const int64_t total = (int64_t)cs.N * cs.P * cs.Q * cs.Cout;
  const int64_t t = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  if (t >= total) return;
  const int co = (int)(t % cs.Cout);
  int64_t m = t / cs.Cout;
  const int q = (int)(m % cs.Q); m /= cs.Q;
  const int p = (int)(m % cs.P);
  const int n = (int)(m / cs.P);
  int acc = 0;
  for (int r = 0; r < cs.R; ++r) {
    const int h = p * cs.sh + r - cs.ph;
    if (h < 0 || h >= cs.H) continue;
    for (int s = 0; s < cs.S; ++s) {
      const int w = q * cs.sw + s - cs.pw;
      if (w < 0 || w >= cs.W) continue;
      const uint4* xa = reinterpret_cast<const uint4*>(qX + (((int64_t)n * cs.H + h) * cs.W + w) * cs.Cinp);
      const uint4* wa = reinterpret_cast<const uint4*>(qW + (((int64_t)co * cs.R + r) * cs.S + s) * cs.Cinp);
      for (int k = 0; k < cs.Cinp / 16; ++k) acc = dot16(__ldg(xa + k), __ldg(wa + k), acc);
    }
  }
  const float scale = out.dtype == DAI8_I32 ? 0.f : dequant_scale(*sX, *sW);
  const size_t pix = ((size_t)n * cs.P + p) * cs.Q + q;
  const size_t idx = out.layout == DAI8_NHWC ? pix * cs.Cout + co
                                             : (((size_t)n * cs.Cout + co) * cs.P + p) * cs.Q + q;
  store_result(out.ptr, out.dtype, idx, acc, scale);
}

// Input gradient (Eq. 3): thread = (input pixel, input channel); gathers the output positions
// (p, q) with h = p*stride + r - pad, w = q*stride + s - pad.
__global__ void __launch_bounds__(kThreads)
direct_bwd_data_kernel(const int8_t* __restrict__ gq, const int8_t* __restrict__ wT,
                       const float* __restrict__ gmax, const float* __restrict__ sW, ConvShape cs,
                       ConvOut out) {
  const int64_t total = (int64_t)cs.N * cs.H * cs.W * cs.Cin;
  const int64_t t = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  if (t >= total) return;
  const int ci = (int)(t % cs.Cin);
  int64_t m = t / cs.Cin;
  const int w = (int)(m % cs.W); m /= cs.W;
  const int h = (int)(m % cs.H);
  const int n = (int)(m / cs.H);
  int acc = 0;
  for (int r = 0; r < cs.R; ++r) {
    const int hp = h + cs.ph - r;
    if (hp < 0 || hp % cs.sh != 0) continue;
    const int p = hp / cs.sh;
    if (p >= cs.P) continue;
    for (int s = 0; s < cs.S; ++s) {
      const int wq = w + cs.pw - s;
      if (wq < 0 || wq % cs.sw != 0) continue;
      const int q = wq / cs.sw;
      if (q >= cs.Q) continue;
      const uint4* ga = reinterpret_cast<const uint4*>(gq + (((int64_t)n * cs.P + p) * cs.Q + q) * cs.Coutp);
      const uint4* wa = reinterpret_cast<const uint4*>(wT + (((int64_t)ci * cs.R + r) * cs.S + s) * cs.Coutp);
      for (int k = 0; k < cs.Coutp / 16; ++k) acc = dot16(__ldg(ga + k), __ldg(wa + k), acc);
    }
  }
  const float scale = out.dtype == DAI8_I32 ? 0.f : dequant_scale(*gmax, *sW);
  const size_t pix = ((size_t)n * cs.H + h) * cs.W + w;
  const size_t idx = out.layout == DAI8_NHWC ? pix * cs.Cin + ci
                                             : (((size_t)n * cs.Cin + ci) * cs.H + h) * cs.W + w;
  store_result(out.ptr, out.dtype, idx, acc, scale);
}

// Weight gradient (Eq. 4).  A warp owns an 8 (co) x 16 (ci) tile of one filter tap and a range of
// output pixels; each lane takes groups of four consecutive pixels, transposes their codes so that
// one 32-bit word holds the four pixels of one channel, and accumulates with dp4a.  Partial sums
// are reduced across the warp and added to acc[Cout][R][S][Cinp] with integer atomics (exact in
// any order).
constexpr int kDwCo = 8, kDwCi = 16, kDwWarps = 4;

__device__ __forceinline__ uint32_t gather_byte4(uint32_t p0, uint32_t p1, uint32_t p2, uint32_t p3, int b) {
  const uint32_t sel = (uint32_t)b | ((uint32_t)(4 + b) << 4);
  const uint32_t lo = __byte_perm(p0, p1, sel);
  const uint32_t hi = __byte_perm(p2, p3, sel);
  return __byte_perm(lo, hi, 0x5410);
}

__global__ void __launch_bounds__(kDwWarps * 32)
direct_bwd_filter_kernel(const int8_t* __restrict__ qX, const int8_t* __restrict__ vq, ConvShape cs,
                         int* __restrict__ acc_out, int ksplit) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int tile = blockIdx.x;
  const int ci_tiles = cs.Cinp / kDwCi;
  const int ci0 = (tile % ci_tiles) * kDwCi; tile /= ci_tiles;
  const int s = tile % cs.S; tile /= cs.S;
  const int r = tile % cs.R; tile /= cs.R;
  const int co0 = tile * kDwCo;

  const int64_t npix = (int64_t)cs.N * cs.P * cs.Q;
  const int64_t nquads = (npix + 3) / 4;
  const int64_t parts = (int64_t)ksplit * kDwWarps;
  const int64_t per = (nquads + parts - 1) / parts;
  const int64_t qbeg = ((int64_t)blockIdx.y * kDwWarps + warp) * per;
  const int64_t qend = min(nquads, qbeg + per);

  int acc[kDwCo][kDwCi];
#pragma unroll
  for (int i = 0; i < kDwCo; ++i)
#pragma unroll
    for (int j = 0; j < kDwCi; ++j) acc[i][j] = 0;

  for (int64_t qd = qbeg + lane; qd < qend; qd += 32) {
    uint2 g[4];   // 8 co codes of each of the 4 pixels
    uint4 x[4];   // 16 ci codes
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int64_t pix = qd * 4 + k;
      g[k] = make_uint2(0u, 0u);
      x[k] = make_uint4(0u, 0u, 0u, 0u);
      if (pix < npix) {
        const int q = (int)(pix % cs.Q);
        const int64_t t = pix / cs.Q;
        const int p = (int)(t % cs.P);
        const int n = (int)(t / cs.P);
        const int h = p * cs.sh + r - cs.ph, w = q * cs.sw + s - cs.pw;
        if (h >= 0 && h < cs.H && w >= 0 && w < cs.W) {
          g[k] = __ldg(reinterpret_cast<const uint2*>(vq + pix * cs.Coutp + co0));
          x[k] = __ldg(reinterpret_cast<const uint4*>(qX + (((int64_t)n * cs.H + h) * cs.W + w) * cs.Cinp + ci0));
        }
      }
    }
    uint32_t gw[kDwCo], xw[kDwCi];
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      gw[b] = gather_byte4(g[0].x, g[1].x, g[2].x, g[3].x, b);
      gw[4 + b] = gather_byte4(g[0].y, g[1].y, g[2].y, g[3].y, b);
      xw[b] = gather_byte4(x[0].x, x[1].x, x[2].x, x[3].x, b);
      xw[4 + b] = gather_byte4(x[0].y, x[1].y, x[2].y, x[3].y, b);
      xw[8 + b] = gather_byte4(x[0].z, x[1].z, x[2].z, x[3].z, b);
      xw[12 + b] = gather_byte4(x[0].w, x[1].w, x[2].w, x[3].w, b);
    }
#pragma unroll
    for (int i = 0; i < kDwCo; ++i)
#pragma unroll
      for (int j = 0; j < kDwCi; ++j) acc[i][j] = __dp4a((int)gw[i], (int)xw[j], acc[i][j]);
  }

#pragma unroll
  for (int i = 0; i < kDwCo; ++i)
#pragma unroll
    for (int j = 0; j < kDwCi; ++j) {
      int v = acc[i][j];
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
      acc[i][j] = v;
    }
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < kDwCo; ++i) {
      const int co = co0 + i;
      if (co >= cs.Cout) continue;
#pragma unroll
      for (int j = 0; j < kDwCi; ++j)
        if (acc[i][j] != 0)
          atomicAdd(acc_out + (((int64_t)co * cs.R + r) * cs.S + s) * cs.Cinp + ci0 + j, acc[i][j]);
    }
  }
}

__global__ void __launch_bounds__(kThreads)
repack_weights_kernel(const int8_t* __restrict__ qW, ConvShape cs, int8_t* __restrict__ wT, int flip) {
  const int64_t total = (int64_t)cs.Cinp * cs.R * cs.S * cs.Coutp;
  const int64_t t = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  if (t >= total) return;
  const int co = (int)(t % cs.Coutp);
  int64_t m = t / cs.Coutp;
  const int s = (int)(m % cs.S); m /= cs.S;
  const int r = (int)(m % cs.R);
  const int ci = (int)(m / cs.R);
  const int rs = flip ? cs.R - 1 - r : r, ss = flip ? cs.S - 1 - s : s;
  int8_t v = 0;
  if (co < cs.Cout) v = qW[(((int64_t)co * cs.R + rs) * cs.S + ss) * cs.Cinp + ci];  // ci >= Cin holds 0
  wT[t] = v;
}

// Layers with at most 16 input channels (network stems) would leave the tensor core's K = 32
// mostly empty.  Their activations are gathered once into a matrix A'[pixel][k'], k' = (r*S+s)*Cin + ci
// over the REAL channels, padded with zeros to Kp (a multiple of 32); forward and weight-gradient
// convolutions then run as pointwise convolutions with Kp input channels on the tensor-core kernels.
__global__ void __launch_bounds__(kThreads)
pack_im2col_kernel(const int8_t* __restrict__ qX, ConvShape cs, int Kp, int8_t* __restrict__ A) {
  grid_dependency_release();
  grid_dependency_wait();
  const int groups = Kp / 16;                                   // 16-byte groups per pixel row of A'
  const int64_t total = (int64_t)cs.N * cs.P * cs.Q * groups;
  const int64_t t = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  if (t >= total) return;
  const int kg = (int)(t % groups);
  int64_t m = t / groups;
  const int q = (int)(m % cs.Q); m /= cs.Q;
  const int p = (int)(m % cs.P);
  const int n = (int)(m / cs.P);
  const int cc = packed_channels(cs);                          // channels >= Cin of X hold zeros
  const int Kreal = cs.R * cs.S * cc;
  uint32_t w[4] = {0u, 0u, 0u, 0u};
  int k = kg * 16;
  int tap = k / cc, ci = k - tap * cc;
  int r = tap / cs.S, s = tap - r * cs.S;
#pragma unroll
  for (int j = 0; j < 16; ++j, ++k) {
    if (k < Kreal) {
      const int h = p * cs.sh + r - cs.ph, x = q * cs.sw + s - cs.pw;
      if (h >= 0 && h < cs.H && x >= 0 && x < cs.W) {
        const uint32_t v = (uint8_t)qX[(((int64_t)n * cs.H + h) * cs.W + x) * cs.Cinp + ci];
        w[j >> 2] |= v << (8 * (j & 3));
      }
      if (++ci == cc) { ci = 0; if (++s == cs.S) { s = 0; ++r; } }
    }
  }
  reinterpret_cast<uint4*>(A)[t] = make_uint4(w[0], w[1], w[2], w[3]);
}

// Exactly 16 input channels: every tap of every pixel is one 16-byte vector of X.
__global__ void __launch_bounds__(kThreads)
pack_im2col_c16_kernel(const int8_t* __restrict__ qX, ConvShape cs, int Kp, int8_t* __restrict__ A) {
  grid_dependency_release();
  grid_dependency_wait();
  const int groups = Kp / 16, T = cs.R * cs.S;
  const int64_t total = (int64_t)cs.N * cs.P * cs.Q * groups;
  for (int64_t t = (int64_t)blockIdx.x * kThreads + threadIdx.x; t < total; t += (int64_t)gridDim.x * kThreads) {
    const int tap = (int)(t % groups);
    int64_t m = t / groups;
    const int q = (int)(m % cs.Q); m /= cs.Q;
    const int p = (int)(m % cs.P);
    const int n = (int)(m / cs.P);
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (tap < T) {
      const int r = tap / cs.S, s = tap - r * cs.S;
      const int h = p * cs.sh + r - cs.ph, x = q * cs.sw + s - cs.pw;
      if (h >= 0 && h < cs.H && x >= 0 && x < cs.W)
        v = *reinterpret_cast<const uint4*>(qX + (((int64_t)n * cs.H + h) * cs.W + x) * 16);
    }
    reinterpret_cast<uint4*>(A)[t] = v;
  }
}

// The same matrix, kPackRows output rows (n, p .. p+3) per block: the input rows they need are first
// compacted to their real channels in shared memory, where the S*Cin bytes of one filter row of one
// output pixel are contiguous, so every input vector is fetched once per block (neighbouring output
// rows share most of their input rows) and the rows of A' leave as full 16-byte stores.
constexpr int kPackRows = 4;
__global__ void __launch_bounds__(kThreads)
pack_im2col_rows_kernel(const int8_t* __restrict__ qX, ConvShape cs, int Kp, int rowpix, int rowbytes,
                        int8_t* __restrict__ A) {
  grid_dependency_release();
  grid_dependency_wait();
  extern __shared__ uint8_t xrows[];                            // [(np-1)*sh + R][rowbytes]
  const int cc = packed_channels(cs);
  const int pblocks = (cs.P + kPackRows - 1) / kPackRows;
  const int n = blockIdx.x / pblocks, p0 = (blockIdx.x - n * pblocks) * kPackRows;
  const int np = min(kPackRows, cs.P - p0);
  const int nrows = (np - 1) * cs.sh + cs.R;
  const int total_in = nrows * rowpix;
#pragma unroll 1
  for (int i0 = threadIdx.x; i0 < total_in; i0 += 4 * kThreads) {
    uint32_t first[4];                                          // only channels 0..3 can be real when Cin <= 4
    uint4 full[4];
    int r[4], xi[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {                               // four independent loads in flight
      const int i = i0 + u * kThreads;
      r[u] = i / rowpix; xi[u] = i - r[u] * rowpix;
      const int h = p0 * cs.sh + r[u] - cs.ph, x = xi[u] - cs.pw;
      full[u] = make_uint4(0u, 0u, 0u, 0u);
      if (i < total_in && h >= 0 && h < cs.H && x >= 0 && x < cs.W) {
        const int8_t* src = qX + (((int64_t)n * cs.H + h) * cs.W + x) * 16;
        if (cs.Cin <= 4) full[u].x = *reinterpret_cast<const uint32_t*>(src);
        else full[u] = *reinterpret_cast<const uint4*>(src);
      }
      first[u] = full[u].x;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (i0 + u * kThreads >= total_in) break;
      uint8_t* dst = xrows + r[u] * rowbytes + xi[u] * cc;
      if (cs.Cin <= 4) {
        *reinterpret_cast<uint32_t*>(dst) = first[u];         // channels >= Cin of X hold zeros
      } else {
        const uint32_t w[4] = {full[u].x, full[u].y, full[u].z, full[u].w};
#pragma unroll
        for (int c = 0; c < 16; ++c)
          if (c < cs.Cin) dst[c] = (uint8_t)(w[c >> 2] >> (8 * (c & 3)));
      }
    }
  }
  __syncthreads();
  const int groups = Kp / 16, SC = cs.S * cc, Kreal = cs.R * SC;
  uint4* out = reinterpret_cast<uint4*>(A) + ((int64_t)n * cs.P + p0) * cs.Q * groups;
  const int per_row = cs.Q * groups;
  if (cc == 4) {
    // one 32-bit word per pixel: word j of the row of A' is pixel (r, s) = (j / S, j % S) of the window
    const int T = cs.R * cs.S;
    for (int i = threadIdx.x; i < np * per_row; i += kThreads) {
      const int pl = i / per_row, j = i - pl * per_row;
      const int q = j / groups, kg = j - q * groups;
      int tap = kg * 4;
      int r = tap / cs.S, s = tap - r * cs.S;
      const uint8_t* src = xrows + (pl * cs.sh) * rowbytes + q * cs.sw * 4;
      uint32_t w[4];
#pragma unroll
      for (int jj = 0; jj < 4; ++jj, ++tap) {
        w[jj] = tap < T ? *reinterpret_cast<const uint32_t*>(src + r * rowbytes + s * 4) : 0u;
        if (++s == cs.S) { s = 0; ++r; }
      }
      out[i] = make_uint4(w[0], w[1], w[2], w[3]);
    }
    return;
  }
  for (int i = threadIdx.x; i < np * per_row; i += kThreads) {
    const int pl = i / per_row, j = i - pl * per_row;
    const int q = j / groups, kg = j - q * groups;
    int k = kg * 16;
    int r = k / SC, off = k - r * SC;
    const uint8_t* src = xrows + (pl * cs.sh) * rowbytes + q * cs.sw * cc;
    uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int jj = 0; jj < 16; ++jj, ++k) {
      if (k < Kreal) {
        w[jj >> 2] |= (uint32_t)src[r * rowbytes + off] << (8 * (jj & 3));
        if (++off == SC) { off = 0; ++r; }
      }
    }
    out[i] = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

// [Cout][R][S][Cinp] -> [Cout][Kp] in the same k' order.
__global__ void __launch_bounds__(kThreads)
pack_weights_kernel(const int8_t* __restrict__ qW, ConvShape cs, int Kp, int8_t* __restrict__ Wp) {
  grid_dependency_release();
  grid_dependency_wait();
  const int64_t total = (int64_t)cs.Cout * Kp;
  const int64_t t = (int64_t)blockIdx.x * kThreads + threadIdx.x;
  if (t >= total) return;
  const int k = (int)(t % Kp), co = (int)(t / Kp);
  int8_t v = 0;
  const int cc = packed_channels(cs);
  if (k < cs.R * cs.S * cc) {
    const int tap = k / cc, ci = k - tap * cc;
    v = qW[((int64_t)co * cs.R * cs.S + tap) * cs.Cinp + ci];     // channels >= Cin of qW hold zeros
  }
  Wp[t] = v;
}

// One block transposes a 64 (co) x 64 (ci) tile of one filter tap through shared memory: 16-byte reads
// along ci, 16-byte writes along co.  blockIdx.z runs over the taps in class order.
__global__ void __launch_bounds__(kThreads)
repack_weights_classes_kernel(const int8_t* __restrict__ qW, ConvShape cs, DgradClasses dc, int8_t* __restrict__ wT) {
  grid_dependency_release();
  grid_dependency_wait();
  __shared__ __align__(16) uint8_t tile[64][80];              // [co][ci], rows padded against bank conflicts
  int k = 0, local = blockIdx.z;
  while (k + 1 < dc.n && local >= dc.cls[k].Tr * dc.cls[k].Ts) { local -= dc.cls[k].Tr * dc.cls[k].Ts; ++k; }
  const DgradClass& c = dc.cls[k];
  if (local >= c.Tr * c.Ts) return;
  const int tr = local / c.Ts, ts = local - tr * c.Ts;
  const int r = c.r0 + cs.sh * (c.Tr - 1 - tr), s = c.s0 + cs.sw * (c.Ts - 1 - ts);   // mirrored order
  const int co0 = blockIdx.x * 64, ci0 = blockIdx.y * 64;
  {
    const int co = co0 + threadIdx.x / 4, ci = ci0 + (threadIdx.x & 3) * 16;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (co < cs.Cout && ci < cs.Cinp)     // channels ci >= Cin hold zeros in qW
      v = *reinterpret_cast<const uint4*>(qW + (((int64_t)co * cs.R + r) * cs.S + s) * cs.Cinp + ci);
    *reinterpret_cast<uint4*>(&tile[threadIdx.x / 4][(threadIdx.x & 3) * 16]) = v;
  }
  __syncthreads();
  const int ci = ci0 + threadIdx.x / 4, cq = (threadIdx.x & 3) * 16;
  if (ci >= cs.Cinp || co0 + cq >= cs.Coutp) return;
  uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
  for (int j = 0; j < 16; ++j) w[j >> 2] |= (uint32_t)tile[cq + j][threadIdx.x / 4] << (8 * (j & 3));
  *reinterpret_cast<uint4*>(wT + c.w_off + (((int64_t)ci * c.Tr + tr) * c.Ts + ts) * cs.Coutp + co0 + cq) =
      make_uint4(w[0], w[1], w[2], w[3]);
}

__device__ __forceinline__ void add4(int4& a, const int4& b) { a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w; }

template <int GROUPS>
__global__ void __launch_bounds__(kThreads)
finalize_bwd_filter_kernel(const int* __restrict__ acc, int splits, const float* __restrict__ sX,
                           const float* __restrict__ s, ConvShape cs, int pack_cin, int pack_R, int pack_S,
                           void* __restrict__ dW, dai8_dtype dtype) {
  grid_dependency_release();
  grid_dependency_wait();
  // A block sums kThreads/GROUPS consecutive groups of four accumulators [co][r][s][ci..ci+3] over the
  // partial images: GROUPS groups of threads take every GROUPS-th image (16-byte coalesced reads,
  // several in flight), shared memory combines the groups in a fixed order.  Integer sums: exact
  // whatever the order.  GROUPS is chosen by the host so that small images still fill the device.
  constexpr int PER = kThreads / GROUPS;
  __shared__ int4 part[GROUPS > 1 ? GROUPS - 1 : 1][PER];
  const int lane = threadIdx.x % PER, grp = threadIdx.x / PER;
  const int64_t per_image = (int64_t)cs.Coutp * cs.R * cs.S * cs.Cinp;
  const int64_t valid = (int64_t)cs.Cout * cs.R * cs.S * cs.Cinp;      // a multiple of 16
  const int64_t e = ((int64_t)blockIdx.x * PER + lane) * 4;           // index into one partial image
  int4 a = make_int4(0, 0, 0, 0);
  if (e < valid) {
    const int* src = acc + e;
    int k = grp;
    for (; k + 3 * GROUPS < splits; k += 4 * GROUPS) {
      const int4 v0 = __ldg(reinterpret_cast<const int4*>(src + (size_t)k * per_image));
      const int4 v1 = __ldg(reinterpret_cast<const int4*>(src + (size_t)(k + GROUPS) * per_image));
      const int4 v2 = __ldg(reinterpret_cast<const int4*>(src + (size_t)(k + 2 * GROUPS) * per_image));
      const int4 v3 = __ldg(reinterpret_cast<const int4*>(src + (size_t)(k + 3 * GROUPS) * per_image));
      add4(a, v0); add4(a, v1); add4(a, v2); add4(a, v3);
    }
    for (; k < splits; k += GROUPS) add4(a, __ldg(reinterpret_cast<const int4*>(src + (size_t)k * per_image)));
  }
  if (GROUPS > 1) {
    if (grp != 0) part[grp - 1][lane] = a;
    __syncthreads();
    if (grp != 0) return;
#pragma unroll
    for (int g = 1; g < GROUPS; ++g) add4(a, part[g - 1][lane]);
  }
  if (e >= valid) return;
  const int ci0 = (int)(e % cs.Cinp);                      // the four share (co, r, s): Cinp is a multiple of 16
  int64_t m = e / cs.Cinp;
  const int ss0 = (int)(m % cs.S); m /= cs.S;
  const int r0 = (int)(m % cs.R);
  const int co = (int)(m / cs.R);
  const float scale = dtype == DAI8_I32 ? 0.f : dequant_scale(*sX, s[co]);
  const int v[4] = {a.x, a.y, a.z, a.w};
  if (pack_cin == 0 && cs.R * cs.S == 1 && dtype == DAI8_F32 && (cs.Cin & 3) == 0) {
    // pointwise filters: dW is [co][ci], the four results are one aligned 16-byte store
    if (ci0 < cs.Cin)
      *reinterpret_cast<float4*>(static_cast<float*>(dW) + (size_t)co * cs.Cin + ci0) =
          make_float4(__fmul_rn((float)v[0], scale), __fmul_rn((float)v[1], scale), __fmul_rn((float)v[2], scale),
                      __fmul_rn((float)v[3], scale));
    return;
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    int ci = ci0 + j, r = r0, ss = ss0, Cin = cs.Cin, R = cs.R, S = cs.S;
    if (ci >= cs.Cin) continue;                            // padding channel
    if (pack_cin > 0) {
      // the images come from the packed pointwise form: `ci` is k' = (r*S + s)*Cin + ci of the real filter
      const int k = ci;
      const int cc = pack_cin <= 4 ? 4 : pack_cin;          // packed_channels of the real layer
      if (k >= pack_R * pack_S * cc) continue;
      const int tap = k / cc;
      ci = k - tap * cc; r = tap / pack_S; ss = tap - r * pack_S;
      if (ci >= pack_cin) continue;                         // word padding
      Cin = pack_cin; R = pack_R; S = pack_S;
    }
    store_result(dW, dtype, (((size_t)co * Cin + ci) * R + r) * S + ss, v[j], scale);
  }
}

// Few partial images, large filters: one block per output channel.  The sums are taken in the order
// of the images ([tap][ci], coalesced reads) into shared memory and written in the order of dW
// ([ci][tap], one contiguous run per output channel), so both sides move whole cache lines.
__global__ void __launch_bounds__(kThreads)
finalize_bwd_filter_rows_kernel(const int* __restrict__ acc, int splits, const float* __restrict__ sX,
                                const float* __restrict__ s, ConvShape cs, void* __restrict__ dW, dai8_dtype dtype) {
  grid_dependency_release();
  grid_dependency_wait();
  extern __shared__ int row[];                         // [T][Cinp]
  const int co = blockIdx.x, T = cs.R * cs.S, n = T * cs.Cinp;
  const size_t per_image = (size_t)cs.Coutp * n;
  const int* src = acc + (size_t)co * n;
  for (int i = threadIdx.x * 4; i < n; i += kThreads * 4) {     // n is a multiple of 16
    int4 a = make_int4(0, 0, 0, 0);
    int k = 0;
    for (; k + 3 < splits; k += 4) {
      const int4 v0 = __ldg(reinterpret_cast<const int4*>(src + (size_t)k * per_image + i));
      const int4 v1 = __ldg(reinterpret_cast<const int4*>(src + (size_t)(k + 1) * per_image + i));
      const int4 v2 = __ldg(reinterpret_cast<const int4*>(src + (size_t)(k + 2) * per_image + i));
      const int4 v3 = __ldg(reinterpret_cast<const int4*>(src + (size_t)(k + 3) * per_image + i));
      add4(a, v0); add4(a, v1); add4(a, v2); add4(a, v3);
    }
    for (; k < splits; ++k) add4(a, __ldg(reinterpret_cast<const int4*>(src + (size_t)k * per_image + i)));
    *reinterpret_cast<int4*>(row + i) = a;
  }
  __syncthreads();
  const float scale = dtype == DAI8_I32 ? 0.f : dequant_scale(*sX, s[co]);
  const size_t out0 = (size_t)co * cs.Cin * T;
  for (int j = threadIdx.x; j < cs.Cin * T; j += kThreads) {
    const int ci = j / T, tap = j - ci * T;
    store_result(dW, dtype, out0 + j, row[tap * cs.Cinp + ci], scale);
  }
}

unsigned blocks_for(int64_t total) { return (unsigned)ceil_div64(total, kThreads); }

}  // namespace

dai8_status direct_fwd(const int8_t* qX, const int8_t* qW, const float* sX, const float* sW,
                       const ConvShape& cs, const ConvOut& out, cudaStream_t st) {
  const int64_t total = (int64_t)cs.N * cs.P * cs.Q * cs.Cout;
  direct_fwd_kernel<<<blocks_for(total), kThreads, 0, st>>>(qX, qW, sX, sW, cs, out);
  note_launch();
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}

dai8_status direct_bwd_data(const int8_t* gq, const int8_t* wT, const float* gmax, const float* sW,
                            const ConvShape& cs, const ConvOut& out, cudaStream_t st) {
  const int64_t total = (int64_t)cs.N * cs.H * cs.W * cs.Cin;
  direct_bwd_data_kernel<<<blocks_for(total), kThreads, 0, st>>>(gq, wT, gmax, sW, cs, out);
  note_launch();
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}

dai8_status direct_bwd_filter_acc(const int8_t* qX, const int8_t* vq, const ConvShape& cs, int* acc,
                                  cudaStream_t st) {
  const int64_t tiles = (int64_t)(cs.Coutp / kDwCo) * cs.R * cs.S * (cs.Cinp / kDwCi);
  const int64_t nquads = ((int64_t)cs.N * cs.P * cs.Q + 3) / 4;
  // enough blocks to fill the machine a few times, at least 8 quads per lane
  int64_t ksplit = ceil_div64(148 * 16, tiles);
  const int64_t kmax = ceil_div64(nquads, (int64_t)kDwWarps * 32 * 8);
  if (ksplit > kmax) ksplit = kmax;
  if (ksplit < 1) ksplit = 1;
  if (ksplit > 65535) ksplit = 65535;
  direct_bwd_filter_kernel<<<dim3((unsigned)tiles, (unsigned)ksplit), kDwWarps * 32, 0, st>>>(
      qX, vq, cs, acc, (int)ksplit);
  note_launch();
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}

dai8_status repack_weights_transposed(const int8_t* qW, const ConvShape& cs, int8_t* wT, int flip,
                                      cudaStream_t st) {
  const int64_t total = (int64_t)cs.Cinp * cs.R * cs.S * cs.Coutp;
  repack_weights_kernel<<<blocks_for(total), kThreads, 0, st>>>(qW, cs, wT, flip);
  note_launch();
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}

dai8_status repack_weights_classes(const int8_t* qW, const ConvShape& cs, const DgradClasses& dc, int8_t* wT,
                                   cudaStream_t st) {
  const dim3 grid((unsigned)((cs.Coutp + 63) / 64), (unsigned)((cs.Cinp + 63) / 64), (unsigned)(cs.R * cs.S));
  DAI8_RETURN_IF_CUDA(launch_dependent(repack_weights_classes_kernel, dim3(grid), dim3(kThreads), 0, st, qW, cs, dc, wT));
  note_launch();
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}

dai8_status pack_small_cin(const int8_t* qX, const ConvShape& cs, int Kp, int8_t* A, cudaStream_t st) {
  const int rowpix = (cs.Q - 1) * cs.sw + cs.S;
  const int rowbytes = round_up(rowpix * packed_channels(cs), 4);
  if (cs.Cin == 16) {
    const int64_t total = (int64_t)cs.N * cs.P * cs.Q * (Kp / 16);
    const int64_t want = ceil_div64(total, kThreads * 4);
    DAI8_RETURN_IF_CUDA(launch_dependent(pack_im2col_c16_kernel, dim3((unsigned)(want < 148 * 16 ? want : 148 * 16)), dim3(kThreads), 0, st, qX, cs, Kp, A));
  } else if ((size_t)((kPackRows - 1) * cs.sh + cs.R) * rowbytes <= 48 * 1024 && (int64_t)cs.N * cs.P < ((int64_t)1 << 31)) {
    const int pblocks = (cs.P + kPackRows - 1) / kPackRows;
    const size_t smem = (size_t)((kPackRows - 1) * cs.sh + cs.R) * rowbytes;
    DAI8_RETURN_IF_CUDA(launch_dependent(pack_im2col_rows_kernel, dim3((unsigned)(cs.N * pblocks)), dim3(kThreads), smem, st, qX, cs, Kp, rowpix, rowbytes, A));
  } else {
    const int64_t total = (int64_t)cs.N * cs.P * cs.Q * (Kp / 16);
    DAI8_RETURN_IF_CUDA(launch_dependent(pack_im2col_kernel, dim3(blocks_for(total)), dim3(kThreads), 0, st, qX, cs, Kp, A));
  }
  note_launch();
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}

dai8_status pack_small_cin_weights(const int8_t* qW, const ConvShape& cs, int Kp, int8_t* Wp, cudaStream_t st) {
  DAI8_RETURN_IF_CUDA(launch_dependent(pack_weights_kernel, dim3(blocks_for((int64_t)cs.Cout * Kp)), dim3(kThreads), 0, st, qW, cs, Kp, Wp));
  note_launch();
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}

dai8_status finalize_bwd_filter(const int* acc, int splits, const float* sX, const float* s,
                                const ConvShape& cs, const ConvShape* packed_from, void* dW, dai8_dtype dtype,
                                cudaStream_t st) {
  const int64_t valid = (int64_t)cs.Cout * cs.R * cs.S * cs.Cinp;
  const int pc = packed_from ? packed_from->Cin : 0, pr = packed_from ? packed_from->R : 0, ps = packed_from ? packed_from->S : 0;
  const size_t row_bytes = (size_t)cs.R * cs.S * cs.Cinp * sizeof(int);
  if (!packed_from && splits <= 16 && row_bytes <= 48 * 1024 && row_bytes >= 4096) {
    DAI8_RETURN_IF_CUDA(launch_dependent(finalize_bwd_filter_rows_kernel, dim3((unsigned)cs.Cout), dim3(kThreads), row_bytes, st, acc, splits, sX, s, cs, dW, dtype));
  } else {
    // enough groups to put some 150 thousand threads to work, as far as there are images to share out
    const int64_t quads = valid / 4;
    int groups = 1;
    while (groups < 8 && groups * 2 <= splits && quads * groups < 150000) groups *= 2;
    if (groups == 8)
      DAI8_RETURN_IF_CUDA(launch_dependent(finalize_bwd_filter_kernel<8>, dim3((unsigned)ceil_div64(quads, kThreads / 8)), dim3(kThreads), 0, st, acc, splits, sX, s, cs, pc, pr, ps, dW, dtype));
    else if (groups == 4)
      DAI8_RETURN_IF_CUDA(launch_dependent(finalize_bwd_filter_kernel<4>, dim3((unsigned)ceil_div64(quads, kThreads / 4)), dim3(kThreads), 0, st, acc, splits, sX, s, cs, pc, pr, ps, dW, dtype));
    else if (groups == 2)
      DAI8_RETURN_IF_CUDA(launch_dependent(finalize_bwd_filter_kernel<2>, dim3((unsigned)ceil_div64(quads, kThreads / 2)), dim3(kThreads), 0, st, acc, splits, sX, s, cs, pc, pr, ps, dW, dtype));
    else
      DAI8_RETURN_IF_CUDA(launch_dependent(finalize_bwd_filter_kernel<1>, dim3((unsigned)ceil_div64(quads, kThreads)), dim3(kThreads), 0, st, acc, splits, sX, s, cs, pc, pr, ps, dW, dtype));
  }
  note_launch();
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}

}  // namespace dai8
