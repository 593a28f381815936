// Tensor-core convolutions for sm_100a: implicit GEMM on tcgen05.mma.kind::i8 with int32
// accumulators in tensor memory, operands staged in shared memory by TMA.
//
// Forward and input-gradient convolutions (Fig. 2; Eq. 3) share one kernel: the output is a
// matrix [pixels][channels], D[m][j] = sum over filter taps t and contraction channels k of
// A[pixel(m) + offset(t)][k] * B[j][t][k].  A is an NHWC code tensor read with TMA in im2col mode
// (128 consecutive output pixels per tile, padding filled with zeros by the copy engine), B the
// weight codes [rows][taps][channels] read with a tiled TMA box; both land in shared memory in the
// K-major swizzled layout the MMA descriptors name.  For the input gradient A is q(G), the filter
// taps are mirrored (padding R-1-pad) and the contraction runs over Cout, which is the strided index
// of the stored weights [Cout][taps][Cinp]: B is then read in place as an MN-major operand (boxes of
// kc output channels x 32/64/128 input channels), or, where the tile width is not a multiple of 32
// channels, from a transposed K-major copy.
//
// Roles inside a CTA: warp 0 issues TMA loads, warp 1 owns the tensor memory and issues the MMAs
// (one elected lane), the remaining warps (eight in the persistent forward / input-gradient kernel,
// four in the weight-gradient kernel) read the accumulators back (tcgen05.ld), apply the
// de-quantization scale and store.  Stages are handed over with mbarriers; every wait is bounded
// and a wait that expires records DAI8_ERR_TIMEOUT in the device status word instead of hanging.
//
// Measured tcgen05 rates that shaped the tiling (operands resident in shared memory, nothing else
// running): one kind::i8 MMA of M = 128, K = 32 takes 128 cycles with N = 256 and never less than 73
// cycles whatever N, and M = 64 costs what M = 128 costs.  Hence tiles as wide as the output allows
// (up to 256 columns), and in the weight gradient several filter taps side by side in one MMA.
#include <cuda.h>

#include <cstring>
#include <mutex>

#include "umma_ptx.cuh"

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

unsigned int* device_status_address() {
  void* p = nullptr;
  if (cudaGetSymbolAddress(&p, g_device_status) != cudaSuccess) return nullptr;
  return static_cast<unsigned int*>(p);
}

namespace {

using namespace umma;

// Self-test of the bounded wait of the convolution kernels: an mbarrier nobody arrives on, waited for
// with a limit of a few thousand cycles and nothing in flight (see dai8_debug_expire_waits).
__global__ void expire_conv_wait_kernel(long long limit, int* report) {
  __shared__ uint64_t bar;
  __shared__ volatile uint32_t abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0u;
    mbar_init(&bar, 1);
    fence_mbar_init();
  }
  __syncthreads();
  const bool ok = mbar_wait(&bar, 0u, &abort_flag, &g_device_status, limit);
  if (threadIdx.x == 0) report[2] = ok ? 0 : 1;
}

constexpr int kThreadsIgemm = 192;      // weight-gradient kernel: TMA warp, MMA warp, 4 epilogue warps
constexpr int kEpiWarps = 8;             // persistent kernel: two epilogue warps per tensor-memory lane quarter
constexpr int kThreadsPersist = 64 + 32 * kEpiWarps;
constexpr int kOutBlockBytes = 32 * 128; // epilogue staging block: 32 pixel rows x 128 bytes of channels

struct IgemmParams {
  int Mtot, P, Q;        // output pixels and output extent (pixel m = (n*P + p)*Q + q)
  int Nout;              // real output channels
  int R, S;              // filter taps
  int kc_bytes;          // contraction bytes per chunk: 32, 64 or 128
  int chunks_per_tap;    // ceil(contraction channels / kc_bytes)
  int G;                 // chunks per pipeline stage
  int k_iters;           // ceil(R*S*chunks_per_tap / G)
  int BN;                // output channels per tile (multiple of 16, <= 256)
  int tmem_cols;         // power of two >= max(32, 2*BN): two accumulator buffers
  int stages;
  int m_tiles, n_tiles;  // tiles of 128 pixels x BN channels; tile t = m_tile*n_tiles + n_tile
  int b_resident;        // the CTA's whole weight tile stays in shared memory (loaded once)
  // B read straight from the forward weight layout [Cout][taps][Cinp] as an MN-major operand (input
  // gradient: the contraction runs over Cout): b_nb boxes of kc rows x b_bw bytes per chunk, and the
  // tap of the full filter that class tap (r, s) stands for is b_tap_base - r*b_tap_dr - s*b_tap_ds
  int b_mn, b_bw, b_nb, b_tap_base, b_tap_dr, b_tap_ds;
  int tma_store;         // NHWC output rows are staged in shared memory and written with tile stores
  int out_elem_bytes;    // 2 (bf16) or 4 (fp32, int32)
  int sh, sw, lower_h, lower_w;  // pixel (p,q) reads input (lower_h + p*sh + r, lower_w + q*sw + s)
  // tile pixel (img, p, q) is written to pixel (img, oh_off + p*oh_step, ow_off + q*ow_step) of an
  // oH x oW output image (identity for the forward and stride-1 input-gradient convolutions)
  int oH, oW, oh_step, oh_off, ow_step, ow_off;
  ConvOut out;
  const float* sa;
  const float* sb;
};

// The MMAs of one pipeline stage: up to 4/KK chunks of KK instructions (K = 32 each), issued by one
// lane from straight-line code.  What a tcgen05.mma costs the issuing thread depends on the code
// around it far more than on the instruction itself (about 180 cycles each from a loop nest, 50 to 100
// from an unrolled block inside a single elected-lane region), hence the template over the chunk width.
template <int KK>
__device__ __forceinline__ void issue_stage(uint32_t d_tmem, uint32_t a_lo, uint32_t a_step, uint32_t a_hi, uint32_t b_lo,
                                            uint32_t b_step, uint32_t b_kstep, uint32_t b_hi, uint32_t idesc, int nch,
                                            uint32_t accumulate) {
#pragma unroll
  for (int j = 0; j < 4 / KK; ++j) {
    if (j < nch) {
#pragma unroll
      for (int kk = 0; kk < KK; ++kk)
        mma_i8_parts2(d_tmem, a_lo + (uint32_t)j * a_step + 2u * kk, a_hi, b_lo + (uint32_t)j * b_step + b_kstep * kk, b_hi, idesc,
                      (j | kk) ? 1u : accumulate);
    }
  }
}

// Persistent: a CTA walks over output tiles t = blockIdx.x, blockIdx.x + gridDim.x, ...  The operand
// ring keeps filling across tile boundaries and the accumulator is double-buffered in tensor
// memory, so the epilogue of one tile overlaps the loads and MMAs of the next.  When the weight
// tile of the CTA fits (it does for every ResNet / MobileNet layer with up to ~100 KB of weights per
// BN output channels) it is loaded once and only activations stream; gridDim.x is then a multiple
// of n_tiles so that a CTA always works on the same output channels.
__global__ void __launch_bounds__(kThreadsPersist, 1)
igemm_kmajor_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                    const __grid_constant__ CUtensorMap mapC, const IgemmParams prm) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t full_bar[8], empty_bar[8], acc_full[2], acc_empty[2], b_full;
  __shared__ uint32_t tmem_base_slot;
  __shared__ volatile uint32_t abort_flag;

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int a_chunk_bytes = kBM * prm.kc_bytes;
  const int b_chunk_bytes = prm.BN * prm.kc_bytes;
  const int total_chunks = prm.R * prm.S * prm.chunks_per_tap;
  const int b_res_bytes = prm.b_resident ? total_chunks * b_chunk_bytes : 0;
  const int chunk_pair_bytes = a_chunk_bytes + (prm.b_resident ? 0 : b_chunk_bytes);   // per chunk of a stage
  const int stage_bytes = prm.G * chunk_pair_bytes;
  // A tile whose output rows fit one column block would leave one epilogue warp of every lane quarter
  // idle; there the two warps take alternate TILES instead (warp group g drains accumulator g), so two
  // tiles are in the epilogue at a time.
  const bool by_tile = prm.tma_store ? prm.BN * prm.out_elem_bytes <= 128 : prm.BN <= 32;
  uint8_t* stage_out = smem + ((b_res_bytes + 1023) & ~1023);   // [kEpiWarps][2][4 KB] when tma_store
  uint8_t* ring = stage_out + (prm.tma_store ? kEpiWarps * 2 * kOutBlockBytes : 0);
  const int num_tiles = prm.m_tiles * prm.n_tiles;

  if (threadIdx.x == 0) {
    abort_flag = 0u;
    for (int s = 0; s < prm.stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], by_tile ? kEpiWarps / 2 : kEpiWarps); }
    mbar_init(&b_full, 1);
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(&tmem_base_slot, (uint32_t)prm.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  grid_dependency_release();
  grid_dependency_wait();   // everything above overlapped the tail of the previous kernel

  if (warp == 0) {
    // Copy-engine issue.  The whole warp runs the loops (ring stage, tile position and filter tap are
    // running counters: no divisions per load); one elected lane issues a stage's loads from an
    // unrolled block, where the compiler can keep the many operands of a bulk-tensor copy in
    // uniform registers.
    const bool leader = elect_one();
    if (leader) {
      tma_prefetch_desc(&mapA);
      tma_prefetch_desc(&mapB);
      if (prm.tma_store) tma_prefetch_desc(&mapC);
      if (prm.b_resident) {
        const int n0 = (blockIdx.x % prm.n_tiles) * prm.BN;
        mbar_expect_tx(&b_full, (uint32_t)b_res_bytes);
        for (int c = 0; c < total_chunks; ++c) {
          const int tap = c / prm.chunks_per_tap;
          const int k0 = (c - tap * prm.chunks_per_tap) * prm.kc_bytes;
          if (prm.b_mn) {
            const int tr = tap / prm.S, ts = tap - tr * prm.S;
            const int ftap = prm.b_tap_base - tr * prm.b_tap_dr - ts * prm.b_tap_ds;
            for (int b = 0; b < prm.b_nb; ++b)
              tma_load_tile_3d(&mapB, &b_full, smem + (size_t)c * b_chunk_bytes + (size_t)b * prm.kc_bytes * prm.b_bw,
                               n0 + b * prm.b_bw, ftap, k0);
          } else {
            tma_load_tile_3d(&mapB, &b_full, smem + (size_t)c * b_chunk_bytes, k0, tap, n0);
          }
        }
      }
    }
    const uint64_t pa = reinterpret_cast<uint64_t>(&mapA), pb = reinterpret_cast<uint64_t>(&mapB);
    const uint32_t ring_a = smem_u32(ring), full_a = smem_u32(&full_bar[0]);
    const int G = prm.G, S = prm.S, cpt = prm.chunks_per_tap, kc = prm.kc_bytes, nst = prm.stages, kit = prm.k_iters;
    const bool resident = prm.b_resident != 0, b_mn = prm.b_mn != 0;
    int stage = 0;
    uint32_t phase = 0;            // parity of the current pass over the ring
    bool first_pass = true;        // nothing to wait for until the ring has wrapped once
    bool ok = true;
    int m_tile = blockIdx.x / prm.n_tiles, n_tile = blockIdx.x - m_tile * prm.n_tiles;
    const int dm = gridDim.x / prm.n_tiles, dn = gridDim.x - dm * prm.n_tiles;   // tile step of this CTA
    for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) {
      const int n0 = n_tile * prm.BN;
      // the last tile is shifted back so that every tile covers 128 existing pixels
      int m0 = m_tile * kBM;
      if (m0 + kBM > prm.Mtot) m0 = prm.Mtot - kBM;
      const int tq = m0 / prm.Q;               // one division pair per tile (not per load)
      const int q0 = m0 - tq * prm.Q;
      const int img = tq / prm.P, p0 = tq - img * prm.P;
      const int cw = prm.lower_w + q0 * prm.sw, ch = prm.lower_h + p0 * prm.sh;
      int c = 0, k0 = 0, kchunk = 0, r = 0, ss = 0;    // chunk, its channel offset, tap row and column
      for (int it = 0; it < kit; ++it) {
        if (!first_pass) ok = mbar_wait(&empty_bar[stage], phase ^ 1u, &abort_flag, &g_device_status) && ok;
        const int nch = min(total_chunks - c, G);
        // channel offset and tap of the (up to four) chunks of this stage
        int ck0[4], cr[4], cs[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          ck0[j] = k0; cr[j] = r; cs[j] = ss;
          if (j < nch) {
            k0 += kc;
            if (++kchunk == cpt) { kchunk = 0; k0 = 0; if (++ss == S) { ss = 0; ++r; } }
          }
        }
        if (leader && ok) {
          const uint32_t bar = full_a + 8u * (uint32_t)stage;
          mbar_expect_tx_a(bar, (uint32_t)(nch * chunk_pair_bytes));
          const uint32_t sa = ring_a + (uint32_t)(stage * stage_bytes);
          const uint32_t sb = sa + (uint32_t)(G * a_chunk_bytes);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            if (j < nch) {
              tma_load_im2col_4d_a(pa, bar, sa + (uint32_t)(j * a_chunk_bytes), ck0[j], cw, ch, img, (uint16_t)cs[j], (uint16_t)cr[j]);
              if (!resident) {
                const uint32_t dst = sb + (uint32_t)(j * b_chunk_bytes);
                if (b_mn) {
                  const int ftap = prm.b_tap_base - cr[j] * prm.b_tap_dr - cs[j] * prm.b_tap_ds;
                  for (int b = 0; b < prm.b_nb; ++b)
                    tma_load_tile_3d_a(pb, bar, dst + (uint32_t)(b * kc * prm.b_bw), n0 + b * prm.b_bw, ftap, ck0[j]);
                } else {
                  tma_load_tile_3d_a(pb, bar, dst, ck0[j], cr[j] * S + cs[j], n0);
                }
              }
            }
          }
        }
        c += nch;
        if (++stage == nst) { stage = 0; phase ^= 1u; first_pass = false; }
      }
      m_tile += dm; n_tile += dn;
      if (n_tile >= prm.n_tiles) { n_tile -= prm.n_tiles; ++m_tile; }
    }
  } else if (warp == 1) {
    // MMA issue.  The whole warp runs the loops (trip counts depend only on the launch parameters; a
    // wait that gives up sets the abort flag, after which every later wait returns at once), and one
    // elected lane issues a stage's instructions from straight-line code: see issue_stage().
    const bool leader = elect_one();
    const bool b_mn = prm.b_mn != 0;
    const uint32_t idesc = idesc_i8_kmajor(prm.BN) | (b_mn ? (1u << 16) : 0u);
    // MN-major B: the low descriptor word carries the distance between the boxes (one box =
    // kc rows of b_bw bytes), a K slice of 32 rows lies 32 * b_bw bytes further
    const uint32_t b_hi = b_mn ? kmajor_desc_hi(prm.b_bw) : kmajor_desc_hi(prm.kc_bytes);
    const uint32_t b_lbo = b_mn ? ((uint32_t)(prm.kc_bytes * prm.b_bw) >> 4) << 16 : (1u << 16);
    const uint32_t b_kstep = b_mn ? (uint32_t)(32 * prm.b_bw) >> 4 : 2u;
    if (prm.b_resident) mbar_wait(&b_full, 0, &abort_flag, &g_device_status);
    int stage = 0, tile_i = 0;
    uint32_t phase = 0;
    const int kk_n = prm.kc_bytes / 32, G = prm.G, nst = prm.stages, kit = prm.k_iters;
    const bool resident = prm.b_resident != 0;
    const uint32_t dhi = kmajor_desc_hi(prm.kc_bytes);
    const uint32_t ring_lo = kmajor_desc_lo(smem_u32(ring));
    const uint32_t bres_lo = ((smem_u32(smem) & 0x3FFFFu) >> 4) | b_lbo;
    const uint32_t lbo_fix = b_lbo - (1u << 16);   // turns a K-major low word into B's
    const uint32_t stage_step = (uint32_t)stage_bytes >> 4, a_step = (uint32_t)a_chunk_bytes >> 4,
                   b_step = (uint32_t)b_chunk_bytes >> 4;
    const uint32_t empty_a = smem_u32(&empty_bar[0]);
    for (int t = blockIdx.x; t < num_tiles; t += gridDim.x, ++tile_i) {
      const int buf = tile_i & 1;
      if (tile_i >= 2) mbar_wait(&acc_empty[buf], ((tile_i >> 1) - 1) & 1, &abort_flag, &g_device_status);
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + (uint32_t)(buf * prm.BN);
      int c = 0;
      uint32_t bres = bres_lo;                 // descriptor low word of the next resident weight chunk
      for (int it = 0; it < kit; ++it) {
        mbar_wait(&full_bar[stage], phase, &abort_flag, &g_device_status);
        tc_fence_after();
        const int nch = min(total_chunks - c, G);
        const uint32_t a_lo = ring_lo + (uint32_t)stage * stage_step;
        const uint32_t b_lo = resident ? bres : a_lo + (uint32_t)G * a_step + lbo_fix;
        if (leader) {
          const uint32_t first = it > 0 ? 1u : 0u;
          if (kk_n == 4) issue_stage<4>(d_tmem, a_lo, a_step, dhi, b_lo, b_step, b_kstep, b_hi, idesc, nch, first);
          else if (kk_n == 2) issue_stage<2>(d_tmem, a_lo, a_step, dhi, b_lo, b_step, b_kstep, b_hi, idesc, nch, first);
          else issue_stage<1>(d_tmem, a_lo, a_step, dhi, b_lo, b_step, b_kstep, b_hi, idesc, nch, first);
          tc_commit_a(empty_a + 8u * (uint32_t)stage);   // frees the stage once these MMAs have read it
          if (it == kit - 1) tc_commit(&acc_full[buf]);  // accumulator of this tile complete
        }
        c += nch;
        bres += (uint32_t)nch * b_step;
        if (++stage == nst) { stage = 0; phase ^= 1u; }
      }
    }
  } else {
    // epilogue: warp w may touch tensor-memory lanes 32*(w%4) .. 32*(w%4)+31; the two warps of a
    // lane quarter take alternate groups of 32 accumulator columns
    const int quarter = warp & 3;
    const int half = (warp - 2) >> 2;
    const bool nhwc = prm.out.layout == DAI8_NHWC;
    // 16-byte stores need the pixel rows to be 16-byte multiples: 8 bf16 or 4 fp32 / int32 channels
    const bool vec_ok = nhwc && (prm.Nout % (prm.out_elem_bytes == 2 ? 8 : 4)) == 0;
    const size_t plane = (size_t)prm.oH * prm.oW;
    const float scale = prm.out.dtype == DAI8_I32 ? 0.f : dequant_scale(*prm.sa, *prm.sb);
    int tile_i = by_tile ? half : 0, n_store = 0;
    const int t_step = by_tile ? 2 : 1, c_first = by_tile ? 0 : half, c_step = by_tile ? 1 : 2;
    for (int t = blockIdx.x + tile_i * (int)gridDim.x; t < num_tiles; t += t_step * (int)gridDim.x, tile_i += t_step) {
      const int buf = tile_i & 1;
      if (!mbar_wait(&acc_full[buf], (tile_i >> 1) & 1, &abort_flag, &g_device_status)) break;
      tc_fence_after();
      const int m_tile = t / prm.n_tiles;
      const int n0 = (t - m_tile * prm.n_tiles) * prm.BN;
      int m0 = m_tile * kBM;
      if (m0 + kBM > prm.Mtot) m0 = prm.Mtot - kBM;
      const int m = m0 + quarter * 32 + lane;
      const int q = m % prm.Q;
      const int tq = m / prm.Q;
      const int p = tq % prm.P, img = tq / prm.P;
      const size_t opix = (size_t)(prm.oh_off + p * prm.oh_step) * prm.oW + (size_t)(prm.ow_off + q * prm.ow_step);   // within the image
      const size_t pix_base = nhwc ? ((size_t)img * plane + opix) * prm.Nout : 0;
      const uint32_t t_tmem = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * prm.BN);
      if (prm.tma_store) {
        // Rows of this warp's 32 pixels go through a 128-byte-swizzled staging block and leave as one
        // tile store per 128 bytes of channels: the copy engine writes whole row segments, where
        // per-lane stores would scatter 16-byte pieces over 32 rows.
        const int cols_per_block = 128 / prm.out_elem_bytes;          // 32 (fp32, int32) or 64 (bf16)
        const int row_bytes = prm.BN * prm.out_elem_bytes;
        uint8_t* my_stage = stage_out + (size_t)(warp - 2) * 2 * kOutBlockBytes;
        for (int blk = c_first; blk * 128 < row_bytes; blk += c_step) {
          const int col = blk * cols_per_block;
          if (n0 + col >= prm.Nout) break;
          uint8_t* st = my_stage + (size_t)(n_store & 1) * kOutBlockBytes;
          if (lane == 0 && n_store >= 2) bulk_wait_read<1>();   // the store that last used this block has read it
          __syncwarp();
          uint8_t* row = st + lane * 128;
#pragma unroll 1
          for (int sub = 0; sub * 32 < cols_per_block; ++sub) {
            int va[2][16];
            tmem_ld16(t_tmem + (uint32_t)(col + sub * 32), va[0]);
            tmem_ld16(t_tmem + (uint32_t)(col + sub * 32 + 16), va[1]);
            tmem_ld_wait();
            if (prm.out.dtype == DAI8_BF16) {
              // 32 columns -> 64 bytes = chunks 4*sub .. 4*sub+3 of the row
#pragma unroll
              for (int g = 0; g < 2; ++g) {
                uint32_t w[8];
#pragma unroll
                for (int i = 0; i < 8; ++i)
                  w[i] = pack_bf16x2(__fmul_rn(__int2float_rn(va[g][2 * i]), scale),
                                     __fmul_rn(__int2float_rn(va[g][2 * i + 1]), scale));
                const int c0 = sub * 4 + g * 2;
                *reinterpret_cast<uint4*>(row + (((c0) ^ (lane & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                *reinterpret_cast<uint4*>(row + (((c0 + 1) ^ (lane & 7)) << 4)) = make_uint4(w[4], w[5], w[6], w[7]);
              }
            } else {
#pragma unroll
              for (int g = 0; g < 2; ++g)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  uint4 o;
                  if (prm.out.dtype == DAI8_F32) {
                    o.x = __float_as_uint(__fmul_rn(__int2float_rn(va[g][4 * i]), scale));
                    o.y = __float_as_uint(__fmul_rn(__int2float_rn(va[g][4 * i + 1]), scale));
                    o.z = __float_as_uint(__fmul_rn(__int2float_rn(va[g][4 * i + 2]), scale));
                    o.w = __float_as_uint(__fmul_rn(__int2float_rn(va[g][4 * i + 3]), scale));
                  } else {
                    o = make_uint4((uint32_t)va[g][4 * i], (uint32_t)va[g][4 * i + 1], (uint32_t)va[g][4 * i + 2], (uint32_t)va[g][4 * i + 3]);
                  }
                  *reinterpret_cast<uint4*>(row + (((g * 4 + i) ^ (lane & 7)) << 4)) = o;
                }
            }
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_store_tile_2d(&mapC, st, (n0 + col) * prm.out_elem_bytes, m0 + quarter * 32);
            bulk_commit();
          }
          ++n_store;
        }
      } else
      for (int cg2 = c_first; cg2 * 32 < prm.BN; cg2 += c_step) {
        const int col = cg2 * 32;
        if (n0 + col >= prm.Nout) break;
        const bool second = col + 16 < prm.BN && n0 + col + 16 < prm.Nout;
        int va[2][16];
        tmem_ld16(t_tmem + (uint32_t)col, va[0]);           // both loads in flight, one wait
        if (second) tmem_ld16(t_tmem + (uint32_t)(col + 16), va[1]);
        tmem_ld_wait();
#pragma unroll
        for (int g = 0; g < 2; ++g) {
          if (g == 1 && !second) break;
          const int (&v)[16] = va[g];
          const int j0 = n0 + col + g * 16;
          if (vec_ok) {
            const int nv = min(16, prm.Nout - j0);     // valid columns of this group: a multiple of 8 (bf16) or 4
            if (prm.out.dtype == DAI8_F32) {
              float4* dst = reinterpret_cast<float4*>(static_cast<float*>(prm.out.ptr) + pix_base + j0);
#pragma unroll
              for (int i = 0; i < 4; ++i)
                if (4 * i < nv) dst[i] = make_float4(__fmul_rn(__int2float_rn(v[4 * i]), scale), __fmul_rn(__int2float_rn(v[4 * i + 1]), scale),
                                     __fmul_rn(__int2float_rn(v[4 * i + 2]), scale), __fmul_rn(__int2float_rn(v[4 * i + 3]), scale));
            } else if (prm.out.dtype == DAI8_BF16) {
              uint32_t w[8];
#pragma unroll
              for (int i = 0; i < 8; ++i)
                w[i] = pack_bf16x2(__fmul_rn(__int2float_rn(v[2 * i]), scale), __fmul_rn(__int2float_rn(v[2 * i + 1]), scale));
              uint4* dst = reinterpret_cast<uint4*>(static_cast<uint16_t*>(prm.out.ptr) + pix_base + j0);
              dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
              if (nv > 8) dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
            } else {
              int4* dst = reinterpret_cast<int4*>(static_cast<int*>(prm.out.ptr) + pix_base + j0);
#pragma unroll
              for (int i = 0; i < 4; ++i) if (4 * i < nv) dst[i] = make_int4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            }
          } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const int j = j0 + i;
              if (j < prm.Nout) {
                const size_t idx = nhwc ? pix_base + j : ((size_t)img * prm.Nout + j) * plane + opix;
                store_result(prm.out.ptr, prm.out.dtype, idx, v[i], scale);
              }
            }
          }
        }
      }
      // this warp has read its lanes of the buffer: hand it back to the MMA warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[buf]);
    }
    if (prm.tma_store && lane == 0) bulk_wait_read<0>();   // staging blocks must outlive their stores
  }

  // teardown: everything this CTA issued must have drained before tensor memory is released
  tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    // a wait expired: give in-flight copies and MMAs time to land before the CTA's resources go
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, (uint32_t)prm.tmem_cols);
  }
}

// ---------------------------------------------------------------------------------------------
// Host side: tensor maps and launch
// ---------------------------------------------------------------------------------------------
// Contraction bytes per chunk for a code tensor with `cp` channels (multiple of 16, >= 32).
int chunk_bytes_for(int cp) {
  if (cp % 128 == 0) return 128;
  if (cp % 64 == 0) return 64;
  if (cp >= 128) return 128;  // ragged tail chunk, zero-filled by the copy engine
  if (cp >= 64) return 64;
  return 32;
}

struct IgemmProblem {
  const int8_t* A;  // [N][Hi][Wi][Kc]
  const int8_t* B;  // [Brows][R*S][Kc]
  int N, Hi, Wi, Kc, Brows;
  int P, Q, Nout, R, S, sh, sw, lower_h, lower_w;
  int oH, oW, oh_step, oh_off, ow_step, ow_off;   // output placement, see IgemmParams
  // b_mn: B is the forward weight tensor [Bk][b_taps][Brows bytes] read as an MN-major operand
  int b_mn = 0, Bk = 0, b_taps = 0, b_tap_base = 0, b_tap_dr = 0, b_tap_ds = 0;
};

bool igemm_supported(const IgemmProblem& pb) {
  if (pb.Kc < 32) return false;
  if ((int64_t)pb.N * pb.P * pb.Q < kBM) return false;
  // small activation tensors stay on the direct kernels (im2col descriptors of tiny tensors are
  // not relied upon)
  if ((int64_t)pb.N * pb.Hi * pb.Wi * pb.Kc < 131072) return false;
  if (pb.sh > 8 || pb.sw > 8 || pb.R > 16 || pb.S > 16) return false;
  if (pb.lower_h < -16 || pb.lower_w < -16 || pb.lower_h > 0 || pb.lower_w > 0) return false;
  if (pb.Nout < 1) return false;
  return true;
}

dai8_status launch_igemm(const IgemmProblem& pb, const float* sa, const float* sb, const ConvOut& out,
                         cudaStream_t st) {
  if (!driver_api().ok()) return DAI8_ERR_CUDA;
  IgemmParams prm;
  prm.Mtot = pb.N * pb.P * pb.Q;
  prm.P = pb.P; prm.Q = pb.Q; prm.Nout = pb.Nout; prm.R = pb.R; prm.S = pb.S;
  prm.kc_bytes = chunk_bytes_for(pb.Kc);
  prm.chunks_per_tap = (pb.Kc + prm.kc_bytes - 1) / prm.kc_bytes;
  prm.G = 128 / prm.kc_bytes;
  const int total_chunks = pb.R * pb.S * prm.chunks_per_tap;
  if (prm.G > total_chunks) prm.G = total_chunks;
  prm.k_iters = (total_chunks + prm.G - 1) / prm.G;
  const int noutp = round_up(pb.Nout, 16);
  prm.BN = noutp < 256 ? noutp : 256;
  if (noutp > 256 && noutp % 256 != 0 && noutp % 128 == 0) prm.BN = 128;
  prm.b_mn = pb.b_mn; prm.b_tap_base = pb.b_tap_base; prm.b_tap_dr = pb.b_tap_dr; prm.b_tap_ds = pb.b_tap_ds;
  prm.b_bw = prm.BN % 128 == 0 ? 128 : (prm.BN % 64 == 0 ? 64 : 32);
  prm.b_nb = prm.BN / prm.b_bw;
  if (pb.b_mn && prm.BN % 32 != 0) return DAI8_ERR_UNSUPPORTED;
  prm.tmem_cols = 32;
  while (prm.tmem_cols < 2 * prm.BN) prm.tmem_cols *= 2;
  prm.m_tiles = (prm.Mtot + kBM - 1) / kBM;
  prm.n_tiles = (noutp + prm.BN - 1) / prm.BN;
  const int smem_budget = 227 * 1024 - 2048 - 1024;   // opt-in limit minus static and alignment slack
  const int a_chunk = kBM * prm.kc_bytes, b_chunk = prm.BN * prm.kc_bytes;
  const int b_res = (total_chunks * b_chunk + 1023) & ~1023;
  const int out_es = out.dtype == DAI8_BF16 ? 2 : 4;
  prm.out_elem_bytes = out_es;
  const bool identity_place = pb.oH == pb.P && pb.oW == pb.Q && pb.oh_step == 1 && pb.ow_step == 1 && pb.oh_off == 0 && pb.ow_off == 0;
  prm.tma_store = (identity_place && out.layout == DAI8_NHWC && (pb.Nout * out_es) % 16 == 0 && pb.Nout * out_es >= 128) ? 1 : 0;
  prm.b_resident = b_res <= 96 * 1024 ? 1 : 0;
  // streamed weights make the operand ring the bottleneck (bytes in flight per SM): those layers
  // give the epilogue's staging blocks to the ring and store straight from registers
  if (!prm.b_resident) prm.tma_store = 0;
  const int stage_out_bytes = prm.tma_store ? kEpiWarps * 2 * kOutBlockBytes : 0;
  const int stage_bytes = prm.G * (a_chunk + (prm.b_resident ? 0 : b_chunk));
  int stages = (smem_budget - stage_out_bytes - (prm.b_resident ? b_res : 0)) / stage_bytes;
  if (stages > 8) stages = 8;
  if (stages < 2) return DAI8_ERR_UNSUPPORTED;
  prm.stages = stages;
  prm.sh = pb.sh; prm.sw = pb.sw; prm.lower_h = pb.lower_h; prm.lower_w = pb.lower_w;
  prm.oH = pb.oH; prm.oW = pb.oW; prm.oh_step = pb.oh_step; prm.oh_off = pb.oh_off;
  prm.ow_step = pb.ow_step; prm.ow_off = pb.ow_off;
  prm.out = out; prm.sa = sa; prm.sb = sb;

  CUtensorMap mapA, mapB, mapC;
  memset(&mapC, 0, sizeof(mapC));
  if (prm.tma_store) {
    // output viewed as bytes: [pixels][Nout*es], stored in boxes of 32 rows x 128 bytes
    const cuuint64_t dims[2] = {(cuuint64_t)pb.Nout * out_es, (cuuint64_t)prm.Mtot};
    const cuuint64_t strides[1] = {(cuuint64_t)pb.Nout * out_es};
    const cuuint32_t box[2] = {128, 32};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = encode_tiled_cached(&mapC, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, out.ptr, dims, strides, box, estr, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
    if (r != CUDA_SUCCESS) return DAI8_ERR_CUDA;
  }
  {
    const cuuint64_t dims[4] = {(cuuint64_t)pb.Kc, (cuuint64_t)pb.Wi, (cuuint64_t)pb.Hi, (cuuint64_t)pb.N};
    const cuuint64_t strides[3] = {(cuuint64_t)pb.Kc, (cuuint64_t)pb.Wi * pb.Kc, (cuuint64_t)pb.Hi * pb.Wi * pb.Kc};
    // base pixel w ranges over [lower_w, Wi - 1 + upper_w]; there are Q of them at step sw
    const int lower[2] = {pb.lower_w, pb.lower_h};
    const int upper[2] = {pb.lower_w + (pb.Q - 1) * pb.sw - (pb.Wi - 1), pb.lower_h + (pb.P - 1) * pb.sh - (pb.Hi - 1)};
    const cuuint32_t estr[4] = {1, (cuuint32_t)pb.sw, (cuuint32_t)pb.sh, 1};
    CUresult r = encode_im2col_cached(&mapA, const_cast<int8_t*>(pb.A), dims, strides, lower, upper, (cuuint32_t)prm.kc_bytes, (cuuint32_t)kBM, estr, swizzle_for(prm.kc_bytes));
    if (r != CUDA_SUCCESS) return DAI8_ERR_CUDA;
  }
  if (pb.b_mn) {
    // weights as stored for the forward pass: [Bk = Cout][taps][Brows = Cinp]; a box is kc output
    // channels (the contraction) x b_bw input channels (N) of one tap
    const cuuint64_t dims[3] = {(cuuint64_t)pb.Brows, (cuuint64_t)pb.b_taps, (cuuint64_t)pb.Bk};
    const cuuint64_t strides[2] = {(cuuint64_t)pb.Brows, (cuuint64_t)pb.b_taps * pb.Brows};
    const cuuint32_t box[3] = {(cuuint32_t)prm.b_bw, 1, (cuuint32_t)prm.kc_bytes};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = encode_tiled_cached(&mapB, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<int8_t*>(pb.B), dims, strides, box, estr, swizzle_for(prm.b_bw), CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
    if (r != CUDA_SUCCESS) return DAI8_ERR_CUDA;
  } else {
    const cuuint64_t dims[3] = {(cuuint64_t)pb.Kc, (cuuint64_t)(pb.R * pb.S), (cuuint64_t)pb.Brows};
    const cuuint64_t strides[2] = {(cuuint64_t)pb.Kc, (cuuint64_t)pb.R * pb.S * pb.Kc};
    const cuuint32_t box[3] = {(cuuint32_t)prm.kc_bytes, 1, (cuuint32_t)prm.BN};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = encode_tiled_cached(&mapB, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<int8_t*>(pb.B), dims, strides, box, estr, swizzle_for(prm.kc_bytes), CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
    if (r != CUDA_SUCCESS) return DAI8_ERR_CUDA;
  }
  const size_t smem_bytes = (size_t)(prm.b_resident ? b_res : 0) + stage_out_bytes + (size_t)stages * stage_bytes + 1024;
  static std::atomic<int> attr_done[64];
  if (set_max_smem_once(attr_done, igemm_kmajor_kernel, 227 * 1024 - 2048) != cudaSuccess) return DAI8_ERR_CUDA;
  // one persistent CTA per SM; with resident weights a CTA keeps its output-channel tile
  const int num_tiles = prm.m_tiles * prm.n_tiles;
  int ctas = sm_count();
  if (prm.b_resident && prm.n_tiles > 1) ctas = ctas >= prm.n_tiles ? ctas / prm.n_tiles * prm.n_tiles : prm.n_tiles;
  if (ctas > num_tiles) ctas = num_tiles;
  note_kernel("igemm_kmajor_kernel");
  log_choice("igemm_kmajor_kernel: im2col, N=%d (%d tiles x %d), kc=%d, %d chunks in stages of %d, taps %dx%d stride %dx%d, weights %s, %d stages, %s, %d CTAs",
             prm.BN, prm.m_tiles, prm.n_tiles, prm.kc_bytes, total_chunks, prm.G, prm.R, prm.S, prm.sh, prm.sw,
             prm.b_resident ? "resident" : (prm.b_mn ? "streamed in place" : "streamed"), prm.stages,
             prm.tma_store ? "tile stores" : "register stores", ctas);
  DAI8_RETURN_IF_CUDA(launch_dependent(igemm_kmajor_kernel, dim3((unsigned)ctas), dim3(kThreadsPersist), smem_bytes, st, mapA, mapB, mapC, prm));
  note_launch();
  return DAI8_OK;
}

std::atomic<int> g_halo_disabled{0};

// The patch form of a stride-1, identity-placed problem, if conv_halo.cu takes it.
bool as_halo(const IgemmProblem& pb, HaloProblem& h) {
  if (g_halo_disabled.load(std::memory_order_relaxed)) return false;
  if (pb.sh != 1 || pb.sw != 1 || pb.R * pb.S <= 1) return false;
  if (pb.oH != pb.P || pb.oW != pb.Q || pb.oh_step != 1 || pb.ow_step != 1 || pb.oh_off != 0 || pb.ow_off != 0) return false;
  h.A = pb.A; h.B = pb.B; h.N = pb.N; h.H = pb.Hi; h.W = pb.Wi; h.Kc = pb.Kc; h.Brows = pb.Brows;
  h.P = pb.P; h.Q = pb.Q; h.Nout = pb.Nout; h.R = pb.R; h.S = pb.S; h.lower_h = pb.lower_h; h.lower_w = pb.lower_w;
  h.b_mn = pb.b_mn; h.Bk = pb.Bk; h.b_taps = pb.b_taps; h.b_tap_base = pb.b_tap_base; h.b_tap_dr = pb.b_tap_dr; h.b_tap_ds = pb.b_tap_ds;
  return true;
}

// Patch form where it applies, im2col form otherwise.
dai8_status launch_conv(const IgemmProblem& pb, const float* sa, const float* sb, const ConvOut& out, cudaStream_t st) {
  HaloProblem h;
  if (as_halo(pb, h) && halo_supported(h, out.dtype, out.layout)) return launch_halo(h, sa, sb, out, st);
  return launch_igemm(pb, sa, sb, out, st);
}

IgemmProblem fwd_problem(const int8_t* qX, const int8_t* qW, const ConvShape& cs) {
  IgemmProblem pb;
  pb.A = qX; pb.B = qW;
  pb.N = cs.N; pb.Hi = cs.H; pb.Wi = cs.W; pb.Kc = cs.Cinp; pb.Brows = cs.Cout;
  pb.P = cs.P; pb.Q = cs.Q; pb.Nout = cs.Cout; pb.R = cs.R; pb.S = cs.S;
  pb.sh = cs.sh; pb.sw = cs.sw; pb.lower_h = -cs.ph; pb.lower_w = -cs.pw;
  pb.oH = cs.P; pb.oW = cs.Q; pb.oh_step = 1; pb.oh_off = 0; pb.ow_step = 1; pb.ow_off = 0;
  return pb;
}

// Input gradient (Eq. 3) as stride-1 forward convolutions of q(G).  Output pixel (h, w) receives
// G[p, q] * W[r, s] for h = p*sh + r - ph, w = q*sw + s - pw.  Fixing the residues a = h mod sh,
// b = w mod sw fixes which taps contribute (r = r0 + sh*j with r0 = (a + ph) mod sh) and makes the
// rest dense: with h = a + sh*h', row p = h' + e - j, e = (a + ph - r0)/sh.  So each residue class
// is one implicit GEMM over q(G) with the class's taps in mirrored order, padding lower = e - (Tr-1),
// written to every sh-th row / sw-th column of dX.  Stride 1 is the single class a = b = 0 (the
// mirrored filter with padding R-1-pad); at stride 2 a 3x3 filter splits into 1, 2, 2 and 4 taps,
// so no multiply is spent on inserted zeros.  A class without taps (1x1 filter, stride 2) leaves
// zeros, written by a memset.
int plan_dgrad(const ConvShape& cs, DgradClasses& dc) {
  int n = 0;
  size_t off = 0;
  dc.any_empty = 0;
  for (int a = 0; a < cs.sh; ++a)
    for (int b = 0; b < cs.sw; ++b) {
      DgradClass& c = dc.cls[n++];
      c.a = a; c.b = b;
      c.r0 = (a + cs.ph) % cs.sh; c.s0 = (b + cs.pw) % cs.sw;
      c.Tr = c.r0 < cs.R ? (cs.R - c.r0 + cs.sh - 1) / cs.sh : 0;
      c.Ts = c.s0 < cs.S ? (cs.S - c.s0 + cs.sw - 1) / cs.sw : 0;
      c.Ha = a < cs.H ? (cs.H - a + cs.sh - 1) / cs.sh : 0;
      c.Wb = b < cs.W ? (cs.W - b + cs.sw - 1) / cs.sw : 0;
      c.lower_h = (a + cs.ph - c.r0) / cs.sh - (c.Tr - 1);
      c.lower_w = (b + cs.pw - c.s0) / cs.sw - (c.Ts - 1);
      c.w_off = (long long)off;
      if (c.Tr * c.Ts == 0 || c.Ha * c.Wb == 0) {
        if (c.Ha * c.Wb != 0) dc.any_empty = 1;
        c.Tr = c.Ts = 0;
      }
      off += (size_t)cs.Cinp * c.Tr * c.Ts * cs.Coutp;
    }
  dc.n = n;
  return n;
}

IgemmProblem dgrad_class_problem(const int8_t* gq, const int8_t* wT, const ConvShape& cs, const DgradClass& c) {
  IgemmProblem pb;
  pb.A = gq; pb.B = wT + c.w_off;
  pb.N = cs.N; pb.Hi = cs.P; pb.Wi = cs.Q; pb.Kc = cs.Coutp; pb.Brows = cs.Cinp;
  pb.P = c.Ha; pb.Q = c.Wb; pb.Nout = cs.Cin; pb.R = c.Tr; pb.S = c.Ts;
  pb.sh = 1; pb.sw = 1; pb.lower_h = c.lower_h; pb.lower_w = c.lower_w;
  pb.oH = cs.H; pb.oW = cs.W; pb.oh_step = cs.sh; pb.oh_off = c.a; pb.ow_step = cs.sw; pb.ow_off = c.b;
  return pb;
}

// ---------------------------------------------------------------------------------------------
// Weight gradient (Eq. 4): D[co][tap][ci] = sum over output pixels of vq[pix][co] * qX[pix+tap][ci].
// The contraction runs over pixels, so with NHWC codes both operands are "MN-major" (the channel
// index is contiguous, the contraction index strided): the paper's X -> X', G -> G' dimension
// transformation is just the major-ness bit of the MMA descriptors, no transposed copy is made.
// A CTA owns 128 output channels x (a group of taps) x (up to 256 input channels) in tensor memory
// and a slice of the pixels.  Every slice writes its own partial image with plain stores and the
// de-quantizing kernel adds the slices in a fixed order: a hundred-odd CTAs adding into one small
// image with atomics took longer to drain in L2 than the whole contraction.
// ---------------------------------------------------------------------------------------------
constexpr int kWgradSmem = 222 * 1024;   // operand ring of the weight-gradient kernel
constexpr int kKP = 128;  // pixels per pipeline stage (4 MMAs of K = 32); 256 where the stage is small

struct WgradParams {
  int npix, P, Q;
  int Cout, Cinp, R, S;
  int sh, sw, lower_h, lower_w;
  int bw;                // channels per B box: 32, 64 or 128 (selects the swizzle)
  int nb;                // B boxes per tap (1 or 2); MMA N = nb * bw
  int tg;                // taps per CTA
  int ci_tiles;
  int chunks_total, chunks_per_split;
  int stages, tmem_cols;
  int kp;                // pixels per pipeline stage: 128 or 256
  int* acc;              // [splits][Cout][R*S][Cinp]: one partial image per slice of the pixels
  size_t acc_stride;     // elements per partial image
};

__device__ __forceinline__ uint64_t mnmajor_desc(uint32_t saddr, int width_bytes, uint32_t lbo_bytes) {
  const uint64_t layout = width_bytes == 128 ? 2ull : (width_bytes == 64 ? 4ull : 6ull);
  const uint64_t sbo = (uint64_t)(8 * width_bytes) >> 4;  // eight contraction rows
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | (sbo << 32) | (1ull << 46) |
         (layout << 61);
}

__device__ __forceinline__ void tma_load_tile_2d_a(uint64_t map, uint32_t bar, uint32_t dst, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tma_load_tile_2d(const CUtensorMap* map, uint64_t* bar, void* dst, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
      : "memory");
}

__global__ void __launch_bounds__(kThreadsIgemm, 1)
wgrad_mnmajor_kernel(const __grid_constant__ CUtensorMap mapG, const __grid_constant__ CUtensorMap mapX,
                     const WgradParams prm) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t full_bar[8], empty_bar[8], acc_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ volatile uint32_t abort_flag;

  const int chunk_begin = blockIdx.x * prm.chunks_per_split;
  const int k_iters = min(prm.chunks_total, chunk_begin + prm.chunks_per_split) - chunk_begin;
  if (k_iters <= 0) return;  // uniform over the CTA

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int T = prm.R * prm.S;
  const int grp = blockIdx.y / prm.ci_tiles, cit = blockIdx.y - grp * prm.ci_tiles;
  const int Nw = prm.nb * prm.bw;
  const int ci0 = cit * Nw;
  const int co0 = blockIdx.z * kBM;
  const int tap_begin = grp * prm.tg;
  const int ntap = min(T, tap_begin + prm.tg) - tap_begin;
  const int a_bytes = prm.kp * 128;
  const int b_box_bytes = prm.kp * prm.bw;
  const int stage_bytes = a_bytes + prm.tg * prm.nb * b_box_bytes;

  if (threadIdx.x == 0) {
    abort_flag = 0u;
    for (int s = 0; s < prm.stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    mbar_init(&acc_bar, 1);
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(&tmem_base_slot, (uint32_t)prm.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  grid_dependency_release();
  grid_dependency_wait();   // everything above overlapped the tail of the previous kernel

  if (warp == 0) {
    // Copy-engine issue: the whole warp runs the loop, one elected lane issues a stage's loads from an
    // unrolled block (a bulk-tensor copy takes its many operands from uniform registers, which the
    // compiler fills cheaply only in warp-uniform code: issued from a loop under `lane == 0` a single
    // load cost the issuing thread about 300 cycles, and the loads, not the MMAs, bound the kernel).
    const bool leader = elect_one();
    if (leader) {
      tma_prefetch_desc(&mapG);
      tma_prefetch_desc(&mapX);
    }
    const uint64_t pg = reinterpret_cast<uint64_t>(&mapG), px = reinterpret_cast<uint64_t>(&mapX);
    const uint32_t ring_a = smem_u32(smem), full_a = smem_u32(&full_bar[0]);
    const uint32_t tx_bytes = (uint32_t)(a_bytes + ntap * prm.nb * b_box_bytes);
    int tap_r[8], tap_s[8];          // filter row and column of this CTA's taps (tg <= 8)
#pragma unroll
    for (int tl = 0; tl < 8; ++tl) {
      const int tap = tap_begin + tl;
      tap_r[tl] = tap / prm.S;
      tap_s[tl] = tap - tap_r[tl] * prm.S;
    }
    int s = 0;
    uint32_t phase = 0;
    bool first_pass = true, ok = true;
    for (int it = 0; it < k_iters; ++it) {
      if (!first_pass) ok = mbar_wait(&empty_bar[s], phase ^ 1u, &abort_flag, &g_device_status) && ok;
      const int pix0 = (chunk_begin + it) * prm.kp;
      const int q0 = pix0 % prm.Q;
      const int t = pix0 / prm.Q;
      const int p0 = t % prm.P, img = t / prm.P;
      const int cw = prm.lower_w + q0 * prm.sw, ch = prm.lower_h + p0 * prm.sh;
      if (leader && ok) {
        const uint32_t bar = full_a + 8u * (uint32_t)s;
        const uint32_t sa = ring_a + (uint32_t)(s * stage_bytes);
        const uint32_t sb = sa + (uint32_t)a_bytes;
        mbar_expect_tx_a(bar, tx_bytes);
        tma_load_tile_2d_a(pg, bar, sa, co0, pix0);
#pragma unroll
        for (int tl = 0; tl < 8; ++tl) {
          if (tl < ntap) {
            tma_load_im2col_4d_a(px, bar, sb + (uint32_t)(tl * prm.nb * b_box_bytes), ci0, cw, ch, img, (uint16_t)tap_s[tl],
                                 (uint16_t)tap_r[tl]);
            if (prm.nb > 1)
              tma_load_im2col_4d_a(px, bar, sb + (uint32_t)((tl * prm.nb + 1) * b_box_bytes), ci0 + prm.bw, cw, ch, img,
                                   (uint16_t)tap_s[tl], (uint16_t)tap_r[tl]);
          }
        }
      }
      if (++s == prm.stages) { s = 0; phase ^= 1u; first_pass = false; }
    }
  } else if (warp == 1) {
    // A and B MN-major (bits 15, 16), int32 accumulate, signed 8-bit operands, M = 128.  The
    // boxes of consecutive taps lie side by side in shared memory and in tensor memory, so one
    // MMA covers as many of them as fit N <= 256.  The whole warp runs the loop; one elected lane
    // issues a stage's instructions from an unrolled block (see issue_stage()).
    const bool leader = elect_one();
    const int nbox = ntap * prm.nb;              // boxes of bw channels in this CTA's stage
    const int per_mma = 256 / prm.bw;            // boxes per MMA
    const uint32_t idesc_full = idesc_i8_kmajor(per_mma * prm.bw) | (1u << 15) | (1u << 16);
    const int tail = nbox % per_mma;             // boxes of the last, narrower MMA group (0: none)
    const uint32_t idesc_tail = idesc_i8_kmajor((tail ? tail : per_mma) * prm.bw) | (1u << 15) | (1u << 16);
    const int groups = (nbox + per_mma - 1) / per_mma;
    const uint64_t a_kstep = (uint64_t)((32 * 128) >> 4), b_kstep = (uint64_t)((32 * prm.bw) >> 4);
    int s = 0;
    uint32_t phase = 0;
    for (int it = 0; it < k_iters; ++it) {
      mbar_wait(&full_bar[s], phase, &abort_flag, &g_device_status);
      tc_fence_after();
      const uint32_t sa = smem_u32(smem + (size_t)s * stage_bytes);
      const uint32_t sb = sa + a_bytes;
      if (leader) {
        const uint64_t ad = mnmajor_desc(sa, 128, (uint32_t)a_bytes);
        const uint32_t first = it > 0 ? 1u : 0u;
#pragma unroll 1
        for (int g = 0; g < groups; ++g) {
          const uint32_t idesc = (g == groups - 1) ? idesc_tail : idesc_full;
          const uint64_t bd = mnmajor_desc(sb + g * per_mma * b_box_bytes, prm.bw, (uint32_t)b_box_bytes);
          const uint32_t d = tmem_base + (uint32_t)(g * per_mma * prm.bw);
          if (prm.kp == 256) {
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) mma_i8(d, ad + a_kstep * kk, bd + b_kstep * kk, idesc, kk ? 1u : first);
          } else {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) mma_i8(d, ad + a_kstep * kk, bd + b_kstep * kk, idesc, kk ? 1u : first);
          }
        }
        tc_commit(&empty_bar[s]);
        if (it == k_iters - 1) tc_commit(&acc_bar);
      }
      if (++s == prm.stages) { s = 0; phase ^= 1u; }
    }
  } else {
    const int quarter = warp & 3;
    const bool ok = mbar_wait(&acc_bar, 0, &abort_flag, &g_device_status);
    tc_fence_after();
    if (ok) {
      // Tensor-memory lane = output channel: every lane holds 32 consecutive input channels of its
      // own row per pair of loads and writes them as eight 16-byte stores.
      int* part = prm.acc + (size_t)blockIdx.x * prm.acc_stride;   // this pixel slice's partial sums
      const int co = co0 + quarter * 32 + lane;
      for (int tl = 0; tl < ntap; ++tl) {
        const int tap = tap_begin + tl;
        for (int cg = 0; cg < Nw / 32; ++cg) {
          int v0[16], v1[16];
          const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(tl * Nw + cg * 32);
          tmem_ld16(taddr, v0);
          tmem_ld16(taddr + 16, v1);
          tmem_ld_wait();
          const int ci = ci0 + cg * 32;
          if (co < prm.Cout && ci < prm.Cinp) {            // Cinp is a multiple of 16
            int4* dst = reinterpret_cast<int4*>(part + ((size_t)co * T + tap) * prm.Cinp + ci);
#pragma unroll
            for (int i = 0; i < 4; ++i) dst[i] = make_int4(v0[4 * i], v0[4 * i + 1], v0[4 * i + 2], v0[4 * i + 3]);
            if (ci + 16 < prm.Cinp) {
#pragma unroll
              for (int i = 0; i < 4; ++i) dst[4 + i] = make_int4(v1[4 * i], v1[4 * i + 1], v1[4 * i + 2], v1[4 * i + 3]);
            }
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, (uint32_t)prm.tmem_cols);
  }
}

bool wgrad_supported(const ConvShape& cs) {
  if (cs.Cinp < 32) return false;
  if ((int64_t)cs.N * cs.P * cs.Q < kKP) return false;
  if ((int64_t)cs.N * cs.H * cs.W * cs.Cinp < 131072) return false;
  if (cs.sh > 8 || cs.sw > 8 || cs.R > 16 || cs.S > 16 || cs.ph > 16 || cs.pw > 16) return false;
  return true;
}

// Tiling of the weight gradient: fills everything of `prm` that depends on the geometry only and
// returns the number of pixel slices (partial images), or 0 if the kernel does not take the shape.
int plan_wgrad(const ConvShape& cs, WgradParams& prm, int* ngroups_out, int* co_tiles_out) {
  prm.npix = cs.N * cs.P * cs.Q;
  prm.P = cs.P; prm.Q = cs.Q; prm.Cout = cs.Cout; prm.Cinp = cs.Cinp; prm.R = cs.R; prm.S = cs.S;
  prm.sh = cs.sh; prm.sw = cs.sw; prm.lower_h = -cs.ph; prm.lower_w = -cs.pw;
  if (cs.Cinp >= 128) {
    prm.bw = 128;
    const int blocks128 = (cs.Cinp + 127) / 128;
    // two boxes (N = 256) share the gradient tile; pointwise filters have so little work per pixel
    // slice that more, narrower tiles (fewer slices, fewer partial images) are faster
    prm.nb = (blocks128 % 2 == 0 && cs.R * cs.S > 1) ? 2 : 1;
  } else {
    prm.bw = cs.Cinp > 32 ? 64 : 32;
    prm.nb = 1;
  }
  const int Nw = prm.nb * prm.bw;
  prm.ci_tiles = (cs.Cinp + Nw - 1) / Nw;
  const int T = cs.R * cs.S;
  const int b_tap_bytes = prm.nb * kKP * prm.bw;
  int tg_max = 512 / Nw;
  if (tg_max > 8) tg_max = 8;          // the producer's unrolled issue block handles up to eight taps
  // Many pixels per slice: fat stages (several taps share the gradient tile, two stages in flight)
  // are fastest, the MMA phase dominates.  Few pixels (28x28 and below at batch 64): the partial
  // images dominate, and fewer taps per CTA mean fewer pixel slices, i.e. fewer partial images, and
  // four lighter stages in flight.  Measured on the VGG-16 / ResNet-50 shapes.
  const int stage_cap = prm.npix >= 100000 ? 100 * 1024 : 56 * 1024;
  int tg_smem = (stage_cap - kKP * 128) / b_tap_bytes;
  if (tg_smem < 1) tg_smem = 1;
  if (tg_max > tg_smem) tg_max = tg_smem;
  if (tg_max < 1) return 0;
  const int ngroups = (T + tg_max - 1) / tg_max;
  prm.tg = (T + ngroups - 1) / ngroups;
  prm.tmem_cols = 32;
  while (prm.tmem_cols < prm.tg * Nw) prm.tmem_cols *= 2;
  // Per-load fixed costs dominate small stages: shapes whose 128-pixel stage is small advance 256
  // pixels per stage (halving the stage to 64 pixels where it is large made things slower).
  prm.kp = kKP;
  int stage_bytes = kKP * 128 + prm.tg * b_tap_bytes;
  if ((kWgradSmem) / (2 * stage_bytes) >= 3 && prm.npix >= 8 * 256) { prm.kp = 256; stage_bytes *= 2; }
  int stages = kWgradSmem / stage_bytes;
  if (stages > 8) stages = 8;
  prm.chunks_total = (prm.npix + prm.kp - 1) / prm.kp;
  const int co_tiles = (cs.Cout + kBM - 1) / kBM;
  const int tiles = ngroups * prm.ci_tiles * co_tiles;
  int ksplit = sm_count() / tiles;
  if (ksplit < 1) ksplit = 1;
  if (ksplit > prm.chunks_total) ksplit = prm.chunks_total;
  prm.chunks_per_split = (prm.chunks_total + ksplit - 1) / ksplit;
  ksplit = (prm.chunks_total + prm.chunks_per_split - 1) / prm.chunks_per_split;
  if (stages > prm.chunks_per_split) stages = prm.chunks_per_split;
  if (stages < 1) return 0;
  prm.stages = stages;
  prm.acc_stride = (size_t)cs.Coutp * T * cs.Cinp;
  *ngroups_out = ngroups;
  *co_tiles_out = co_tiles;
  return ksplit;
}

dai8_status launch_wgrad(const int8_t* qX, const int8_t* vq, const ConvShape& cs, int* acc, int* splits_out,
                         cudaStream_t st) {
  if (!driver_api().ok()) return DAI8_ERR_CUDA;
  WgradParams prm;
  int ngroups = 0, co_tiles = 0;
  const int ksplit = plan_wgrad(cs, prm, &ngroups, &co_tiles);
  if (ksplit < 1) return DAI8_ERR_UNSUPPORTED;
  prm.acc = acc;
  *splits_out = ksplit;
  const int stages = prm.stages;
  const int stage_bytes = prm.kp * 128 + prm.tg * prm.nb * prm.kp * prm.bw;

  CUtensorMap mapG, mapX;
  {
    const cuuint64_t dims[2] = {(cuuint64_t)cs.Coutp, (cuuint64_t)prm.npix};
    const cuuint64_t strides[1] = {(cuuint64_t)cs.Coutp};
    const cuuint32_t box[2] = {128, (cuuint32_t)prm.kp};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = encode_tiled_cached(&mapG, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(vq), dims, strides, box, estr, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
    if (r != CUDA_SUCCESS) return DAI8_ERR_CUDA;
  }
  {
    const cuuint64_t dims[4] = {(cuuint64_t)cs.Cinp, (cuuint64_t)cs.W, (cuuint64_t)cs.H, (cuuint64_t)cs.N};
    const cuuint64_t strides[3] = {(cuuint64_t)cs.Cinp, (cuuint64_t)cs.W * cs.Cinp, (cuuint64_t)cs.H * cs.W * cs.Cinp};
    const int lower[2] = {-cs.pw, -cs.ph};
    const int upper[2] = {-cs.pw + (cs.Q - 1) * cs.sw - (cs.W - 1), -cs.ph + (cs.P - 1) * cs.sh - (cs.H - 1)};
    const cuuint32_t estr[4] = {1, (cuuint32_t)cs.sw, (cuuint32_t)cs.sh, 1};
    CUresult r = encode_im2col_cached(&mapX, const_cast<int8_t*>(qX), dims, strides, lower, upper, (cuuint32_t)prm.bw, (cuuint32_t)prm.kp, estr, swizzle_for(prm.bw));
    if (r != CUDA_SUCCESS) return DAI8_ERR_CUDA;
  }
  const size_t smem_bytes = (size_t)stages * stage_bytes + 1024;
  static std::atomic<int> attr_done[64];
  if (set_max_smem_once(attr_done, wgrad_mnmajor_kernel, kWgradSmem + 1024) != cudaSuccess) return DAI8_ERR_CUDA;
  const dim3 grid((unsigned)ksplit, (unsigned)(ngroups * prm.ci_tiles), (unsigned)co_tiles);
  note_kernel("wgrad_mnmajor_kernel");
  log_choice("wgrad_mnmajor_kernel: %d pixel slices x %d tap groups of %d x %d channel tiles of %d x %d output-channel tiles, %d pixels per stage, %d stages",
             ksplit, ngroups, prm.tg, prm.ci_tiles, prm.nb * prm.bw, co_tiles, prm.kp, stages);
  DAI8_RETURN_IF_CUDA(launch_dependent(wgrad_mnmajor_kernel, grid, dim3(kThreadsIgemm), smem_bytes, st, mapG, mapX, prm));
  note_launch();
  return DAI8_OK;
}

}  // namespace

dai8_status expire_conv_wait(long long limit, int* report_dev, cudaStream_t st) {
  expire_conv_wait_kernel<<<1, 64, 0, st>>>(limit, report_dev);
  note_launch(1);
  DAI8_RETURN_IF_CUDA(cudaGetLastError());
  return DAI8_OK;
}

void set_halo_disabled(int disabled) { g_halo_disabled.store(disabled ? 1 : 0, std::memory_order_relaxed); }

bool umma_fwd_supported(const ConvShape& cs) { return igemm_supported(fwd_problem(nullptr, nullptr, cs)); }

bool umma_bwd_data_supported(const ConvShape& cs) {
  if (cs.sh > 4 || cs.sw > 4) return false;
  DgradClasses dc;
  plan_dgrad(cs, dc);
  for (int i = 0; i < dc.n; ++i)
    if (dc.cls[i].Tr > 0 && !igemm_supported(dgrad_class_problem(nullptr, nullptr, cs, dc.cls[i]))) return false;
  return true;
}

bool umma_bwd_filter_supported(const ConvShape& cs) { return umma_bwd_filter_splits(cs) > 0; }

dai8_status umma_fwd(const int8_t* qX, const int8_t* qW, const float* sX, const float* sW, const ConvShape& cs,
                     const ConvOut& out, cudaStream_t st) {
  return launch_conv(fwd_problem(qX, qW, cs), sX, sW, out, st);
}

dai8_status umma_bwd_data(const int8_t* gq, const int8_t* qW, int8_t* wT, const float* gmax, const float* sW,
                          const ConvShape& cs, const ConvOut& out, cudaStream_t st) {
  DgradClasses dc;
  plan_dgrad(cs, dc);
  if (dc.any_empty) {   // positions no tap reaches
    const size_t es = out.dtype == DAI8_BF16 ? 2 : 4;
    DAI8_RETURN_IF_CUDA(cudaMemsetAsync(out.ptr, 0, (size_t)cs.N * cs.H * cs.W * cs.Cin * es, st));
  }
  // With an output tile width that is a multiple of 32 channels the weights are read where they are,
  // as an MN-major operand (the contraction index Cout is the strided one in [Cout][taps][Cinp]);
  // otherwise they are first transposed into the class-ordered K-major buffer.
  const int noutp = round_up(cs.Cin, 16);
  int bn = noutp < 256 ? noutp : 256;
  if (noutp > 256 && noutp % 256 != 0 && noutp % 128 == 0) bn = 128;
  // Reading in place saves the transposing launch (a few microseconds, which decide the small layers
  // of ResNet-50 / MobileNetV2); the K-major copy makes the GEMM itself faster (measured 10-30 % on
  // the VGG-16 layers: 128->128 @112 177 -> 143 us), so large problems take the copy.
  const bool in_place = bn % 32 == 0 && (double)cs.N * cs.P * cs.Q * cs.Cout * cs.Cin * cs.R * cs.S < 2e10;
  dai8_status r = DAI8_OK;
  if (!in_place) {
    r = repack_weights_classes(qW, cs, dc, wT, st);
    if (r != DAI8_OK) return r;
  }
  for (int i = 0; i < dc.n; ++i) {
    const DgradClass& c = dc.cls[i];
    if (c.Tr == 0) continue;
    IgemmProblem pb = dgrad_class_problem(gq, wT, cs, c);
    if (in_place) {
      // class tap (tr, ts) is filter tap (r0 + sh*(Tr-1-tr), s0 + sw*(Ts-1-ts))
      pb.B = qW; pb.b_mn = 1; pb.Bk = cs.Cout; pb.b_taps = cs.R * cs.S;
      pb.b_tap_base = (c.r0 + cs.sh * (c.Tr - 1)) * cs.S + c.s0 + cs.sw * (c.Ts - 1);
      pb.b_tap_dr = cs.sh * cs.S;
      pb.b_tap_ds = cs.sw;
    }
    r = launch_conv(pb, gmax, sW, out, st);
    if (r != DAI8_OK) return r;
  }
  return DAI8_OK;
}

dai8_status umma_bwd_filter_acc(const int8_t* qX, const int8_t* vq, const ConvShape& cs, int* acc, int* splits,
                                cudaStream_t st) {
  return launch_wgrad(qX, vq, cs, acc, splits, st);
}

int umma_bwd_filter_splits(const ConvShape& cs) {
  if (!wgrad_supported(cs)) return 0;
  WgradParams prm;
  int ngroups = 0, co_tiles = 0;
  return plan_wgrad(cs, prm, &ngroups, &co_tiles);
}

}  // namespace dai8
