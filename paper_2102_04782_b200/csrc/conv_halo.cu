// Tensor-core convolution for filters with more than one tap at stride 1 (the 3x3 layers of VGG-16
// and ResNet-50; forward pass, Fig. 2, and input gradient, Eq. 3): implicit GEMM on
// tcgen05.mma.kind::i8 in which every activation is fetched from L2 about three times instead of
// once per filter tap.
//
// The im2col form of the copy engine (conv_umma.cu) delivers, for every tap, the 128 input pixels
// under that tap: a 3x3 filter reads every activation nine times, and the copy engine, which
// handles such loads pixel row by pixel row, becomes the bound (the MMA thread of those layers
// waits for operands most of the time).  Here an output tile is a patch of 16 rows x 8 columns of
// one image (or 8 x 16, or 4 x 32: whichever wastes least on the image extent), and its accumulator
// row m = TX*y + x.  For tap column s the copy engine brings ONE box of (TY + R - 1) rows x TX
// columns x kc channels, starting s columns to the right; in shared memory that box is pixel-linear,
// TX (a multiple of eight) pixels per image row, so the operand of tap (r, s) is the same box read
// from r image rows -- whole 8-row swizzle groups -- further down: a descriptor offset, no second
// copy.  S boxes per channel chunk serve all R*S taps.  Out-of-image positions (padding, ragged
// tiles) are zero-filled by the copy engine on the way in and clipped by it on the way out.
//
// Weights: K-major [rows][taps][channels] (forward, or the transposed copy of the input gradient) or
// MN-major in place (input gradient, see conv_umma.cu).  They stay resident in shared memory when
// they fit beside the activation ring, else they stream through a ring of their own, one
// (tap, chunk) piece at a time, fed by a second producer warp.
//
// Roles: warp 0 activation loads, warp 1 MMA issue and tensor memory, warp 10 weight loads, warps 2-9
// epilogue in two groups of four (one warp per tensor-memory lane quarter): group 0 drains the even
// tiles of the CTA, group 1 the odd ones, so two tiles are in the epilogue at a time.  Four
// accumulators in tensor memory for tiles of up to 128 channels (two for wider ones), released as
// soon as their last column has been read, before it is converted and stored.  Every wait is bounded.
#include <cstring>

#include "umma_ptx.cuh"

namespace dai8 {
namespace {

using namespace umma;

constexpr int kHaloEpiWarps = 8;
constexpr int kHaloThreads = 64 + 32 * kHaloEpiWarps + 32;   // + the weight-load warp
constexpr int kHaloOutBlock = 32 * 128;          // staging block of an epilogue warp: 32 pixels x 128 bytes
constexpr int kHaloMaxAStages = 6, kHaloMaxBStages = 8;

struct HaloParams {
  int P, Q;              // output extent (= the extent the tiles cover)
  int Nout;              // real output channels
  int R, S;
  int TX, TY;            // output patch of a tile: TY rows x TX columns = 128 pixels, TX in {8, 16, 32}
  int kc_bytes, chunks;  // contraction bytes per chunk (32, 64, 128) and chunks per tap
  int BN, tmem_cols, nbuf;   // accumulator width, tensor-memory columns, accumulators (2 or 4)
  int tiles_x, tiles_y, m_tiles, n_tiles;
  int lower_h, lower_w;  // input position under tap (0, 0) of output (0, 0)
  int a_stages, b_stages, b_resident;
  int b_mn, b_bw, b_nb, b_tap_base, b_tap_dr, b_tap_ds;   // MN-major weights read in place (see IgemmParams)
  int tma_store, stage_bufs, out_elem_bytes;
  ConvOut out;
  const float* sa;
  const float* sb;
  unsigned int* status;
};

__device__ __forceinline__ void tma_load_tile_4d_a(uint64_t map, uint32_t bar, uint32_t dst, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tma_store_tile_4d(const CUtensorMap* map, const void* src, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(src)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

// The MMAs of one (tile, channel chunk): R*S taps x KK instructions of K = 32, issued by ONE lane from
// straight-line code.  What one tcgen05.mma costs the issuing thread depends on the code around it far
// more than on the instruction: from a loop nest over taps with one elected-lane region per tap the
// 64-channel layers ran at 180 cycles per instruction; fully unrolled inside a single elected-lane
// region the same instructions take about 100 (the tensor core itself needs 48 at N = 64).  Hence the
// template over the filter size and the chunk width, with a loop version for other filters.
struct TapIssue {
  uint32_t d_tmem, a_base, row_step, copy_step, a_hi, b_step, b_kstep, b_hi, idesc;
};
template <int R, int S, int KK>
__device__ __forceinline__ void issue_taps_resident(const TapIssue& q, uint32_t b_base, uint32_t accumulate) {
#pragma unroll
  for (int r = 0; r < R; ++r) {
#pragma unroll
    for (int s = 0; s < S; ++s) {
      const uint32_t a_lo = q.a_base + (uint32_t)r * q.row_step + (uint32_t)s * q.copy_step;
      const uint32_t b_lo = b_base + (uint32_t)(r * S + s) * q.b_step;
#pragma unroll
      for (int kk = 0; kk < KK; ++kk)
        mma_i8_parts2(q.d_tmem, a_lo + 2u * kk, q.a_hi, b_lo + q.b_kstep * kk, q.b_hi, q.idesc, (r | s | kk) ? 1u : accumulate);
    }
  }
}
struct BRing {
  uint64_t* full;
  uint32_t empty_a, base_lo;
  int stages;
  volatile uint32_t* abort_flag;
  unsigned int* status;
};
// The same with the weights streamed: every tap waits for its piece and hands it back when its MMAs
// have read it.  Runs in the issuing lane only; stage and phase are that lane's ring position.
template <int R, int S, int KK>
__device__ __forceinline__ void issue_taps_streamed(const TapIssue& q, const BRing& ring, int& stage, uint32_t& phase,
                                                    uint32_t accumulate) {
#pragma unroll
  for (int r = 0; r < R; ++r) {
#pragma unroll
    for (int s = 0; s < S; ++s) {
      mbar_wait(&ring.full[stage], phase, ring.abort_flag, ring.status);
      tc_fence_after();
      const uint32_t a_lo = q.a_base + (uint32_t)r * q.row_step + (uint32_t)s * q.copy_step;
      const uint32_t b_lo = ring.base_lo + (uint32_t)stage * q.b_step;
#pragma unroll
      for (int kk = 0; kk < KK; ++kk)
        mma_i8_parts2(q.d_tmem, a_lo + 2u * kk, q.a_hi, b_lo + q.b_kstep * kk, q.b_hi, q.idesc, (r | s | kk) ? 1u : accumulate);
      tc_commit_a(ring.empty_a + 8u * (uint32_t)stage);   // frees the piece once these MMAs have read it
      if (++stage == ring.stages) { stage = 0; phase ^= 1u; }
    }
  }
}
// Any filter size and chunk width, with loops.
__device__ __forceinline__ void issue_taps_generic(const TapIssue& q, int R, int S, int KK, bool resident, uint32_t b_base,
                                                const BRing& ring, int& stage, uint32_t& phase, uint32_t accumulate) {
  for (int r = 0; r < R; ++r)
    for (int s = 0; s < S; ++s) {
      uint32_t b_lo;
      if (resident) {
        b_lo = b_base + (uint32_t)(r * S + s) * q.b_step;
      } else {
        mbar_wait(&ring.full[stage], phase, ring.abort_flag, ring.status);
        tc_fence_after();
        b_lo = ring.base_lo + (uint32_t)stage * q.b_step;
      }
      const uint32_t a_lo = q.a_base + (uint32_t)r * q.row_step + (uint32_t)s * q.copy_step;
      for (int kk = 0; kk < KK; ++kk) {
        mma_i8_parts2(q.d_tmem, a_lo + 2u * kk, q.a_hi, b_lo + q.b_kstep * kk, q.b_hi, q.idesc, accumulate);
        accumulate = 1;
      }
      if (!resident) {
        tc_commit_a(ring.empty_a + 8u * (uint32_t)stage);
        if (++stage == ring.stages) { stage = 0; phase ^= 1u; }
      }
    }
}

__global__ void __launch_bounds__(kHaloThreads, 1)
igemm_halo_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                  const __grid_constant__ CUtensorMap mapC, const HaloParams prm) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t a_full[kHaloMaxAStages], a_empty[kHaloMaxAStages], b_full[kHaloMaxBStages], b_empty[kHaloMaxBStages];
  __shared__ uint64_t acc_full[4], acc_empty[4], bres_full;
  __shared__ uint32_t tmem_base_slot;
  __shared__ volatile uint32_t abort_flag;

  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int T = prm.R * prm.S;
  const int kc = prm.kc_bytes;
  const int patch_rows = prm.TY + prm.R - 1;
  const int copy_bytes = patch_rows * prm.TX * kc;           // one box: whole 8-row swizzle groups
  const int a_stage_bytes = prm.S * copy_bytes;
  const int b_piece_bytes = prm.BN * kc;
  const int pieces_total = T * prm.chunks;
  // layout: [resident weights | weight ring] [epilogue staging] [activation ring]
  const int b_region = ((prm.b_resident ? pieces_total : prm.b_stages) * b_piece_bytes + 1023) & ~1023;
  uint8_t* b_base = smem;
  uint8_t* stage_out = smem + b_region;
  uint8_t* a_ring = stage_out + (prm.tma_store ? kHaloEpiWarps * prm.stage_bufs * kHaloOutBlock : 0);
  const int num_tiles = prm.m_tiles * prm.n_tiles;
  const int nbuf = prm.nbuf;

  if (threadIdx.x == 0) {
    abort_flag = 0u;
    for (int s = 0; s < prm.a_stages; ++s) { mbar_init(&a_full[s], 1); mbar_init(&a_empty[s], 1); }
    for (int s = 0; s < prm.b_stages; ++s) { mbar_init(&b_full[s], 1); mbar_init(&b_empty[s], 1); }
    for (int i = 0; i < 4; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], kHaloEpiWarps / 2); }
    mbar_init(&bres_full, 1);
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

  // tile t = m_tile * n_tiles + n_tile; m_tile = (img * tiles_y + ty) * tiles_x + tx
  const int tiles_per_img = prm.tiles_y * prm.tiles_x;

  // The three issuing roles below are loops that their whole warp runs: trip counts depend only on the
  // launch parameters, never on what a wait returns (a wait that gives up sets the abort flag, after
  // which every later wait returns at once and the kernel drains), so that control flow and addresses
  // stay warp-uniform (see elect_one()).
  if (warp == 0) {
    // ---- activation loads: per (tile, chunk) S boxes, one per tap column ------------------------------
    const bool leader = elect_one();
    if (leader) {
      tma_prefetch_desc(&mapA);
      if (prm.tma_store) tma_prefetch_desc(&mapC);
    }
    const uint64_t pa = reinterpret_cast<uint64_t>(&mapA);
    const uint32_t ring_a = smem_u32(a_ring), full_a = smem_u32(&a_full[0]);
    int stage = 0;
    uint32_t phase = 0;
    bool first_pass = true, ok = true;
    for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) {
      const int m_tile = t / prm.n_tiles;
      const int img = m_tile / tiles_per_img, rem = m_tile - img * tiles_per_img;
      const int ty = rem / prm.tiles_x, tx = rem - ty * prm.tiles_x;
      const int cy = ty * prm.TY + prm.lower_h, cx = tx * prm.TX + prm.lower_w;
      for (int c = 0; c < prm.chunks; ++c) {
        if (!first_pass) ok = mbar_wait(&a_empty[stage], phase ^ 1u, &abort_flag, prm.status) && ok;
        if (leader && ok) {
          const uint32_t bar = full_a + 8u * (uint32_t)stage;
          mbar_expect_tx_a(bar, (uint32_t)a_stage_bytes);
          uint32_t dst = ring_a + (uint32_t)(stage * a_stage_bytes);
          for (int s = 0; s < prm.S; ++s, dst += (uint32_t)copy_bytes)
            tma_load_tile_4d_a(pa, bar, dst, c * kc, cx + s, cy, img);
        }
        if (++stage == prm.a_stages) { stage = 0; phase ^= 1u; first_pass = false; }
      }
    }
  } else if (warp == 10) {
    // ---- weight loads: everything once (resident) or one (tap, chunk) piece at a time ------------------
    const bool leader = elect_one();
    if (leader) tma_prefetch_desc(&mapB);
    const uint64_t pb = reinterpret_cast<uint64_t>(&mapB);
    const bool b_mn = prm.b_mn != 0;
    auto load_piece = [&](uint32_t bar, uint32_t dst, int tap, int k0, int n0) {
      if (b_mn) {
        const int tr = tap / prm.S, ts = tap - tr * prm.S;
        const int ftap = prm.b_tap_base - tr * prm.b_tap_dr - ts * prm.b_tap_ds;
        for (int b = 0; b < prm.b_nb; ++b)
          tma_load_tile_3d_a(pb, bar, dst + (uint32_t)(b * kc * prm.b_bw), n0 + b * prm.b_bw, ftap, k0);
      } else {
        tma_load_tile_3d_a(pb, bar, dst, k0, tap, n0);
      }
    };
    if (prm.b_resident) {
      const int n0 = (blockIdx.x % prm.n_tiles) * prm.BN;     // gridDim.x is a multiple of n_tiles
      const uint32_t bar = smem_u32(&bres_full);
      if (leader) mbar_expect_tx_a(bar, (uint32_t)(pieces_total * b_piece_bytes));
      for (int c = 0; c < prm.chunks; ++c)
        for (int tap = 0; tap < T; ++tap)
          if (leader) load_piece(bar, smem_u32(b_base) + (uint32_t)((c * T + tap) * b_piece_bytes), tap, c * kc, n0);
    } else {
      const uint32_t ring_b = smem_u32(b_base), full_b = smem_u32(&b_full[0]);
      int stage = 0;
      uint32_t phase = 0;
      bool first_pass = true, ok = true;
      for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) {
        const int n0 = (t % prm.n_tiles) * prm.BN;
        for (int c = 0; c < prm.chunks; ++c)
          for (int tap = 0; tap < T; ++tap) {
            if (!first_pass) ok = mbar_wait(&b_empty[stage], phase ^ 1u, &abort_flag, prm.status) && ok;
            if (leader && ok) {
              const uint32_t bar = full_b + 8u * (uint32_t)stage;
              mbar_expect_tx_a(bar, (uint32_t)b_piece_bytes);
              load_piece(bar, ring_b + (uint32_t)(stage * b_piece_bytes), tap, c * kc, n0);
            }
            if (++stage == prm.b_stages) { stage = 0; phase ^= 1u; first_pass = false; }
          }
      }
    }
  } else if (warp == 1) {
    // ---- MMA issue ----------------------------------------------------------------------------------------
    // After a wait has given up, the remaining iterations still issue (on whatever shared memory
    // holds): their results are never stored, and nothing in the loop depends on a wait's outcome.
    const bool leader = elect_one();
    const bool b_mn = prm.b_mn != 0, resident = prm.b_resident != 0;
    const uint32_t idesc = idesc_i8_kmajor(prm.BN) | (b_mn ? (1u << 16) : 0u);
    const uint32_t a_hi = kmajor_desc_hi(kc);
    const uint32_t b_hi = b_mn ? kmajor_desc_hi(prm.b_bw) : kmajor_desc_hi(kc);
    const uint32_t b_lbo = b_mn ? ((uint32_t)(kc * prm.b_bw) >> 4) << 16 : (1u << 16);
    const uint32_t b_kstep = b_mn ? (uint32_t)(32 * prm.b_bw) >> 4 : 2u;
    const uint32_t a_ring_lo = kmajor_desc_lo(smem_u32(a_ring));
    const uint32_t b_base_lo = ((smem_u32(b_base) & 0x3FFFFu) >> 4) | b_lbo;
    const uint32_t a_stage_step = (uint32_t)a_stage_bytes >> 4, copy_step = (uint32_t)copy_bytes >> 4;
    const uint32_t row_step = (uint32_t)(prm.TX * kc) >> 4;      // one image row of the box = TX/8 swizzle groups
    const uint32_t b_step = (uint32_t)b_piece_bytes >> 4;
    const uint32_t a_empty_a = smem_u32(&a_empty[0]), b_empty_a = smem_u32(&b_empty[0]);
    const int kk_n = kc / 32;
    const bool k3 = prm.R == 3 && prm.S == 3;
    if (resident) mbar_wait(&bres_full, 0, &abort_flag, prm.status);
    TapIssue q;
    q.row_step = row_step; q.copy_step = copy_step; q.a_hi = a_hi; q.b_step = b_step; q.b_kstep = b_kstep; q.b_hi = b_hi; q.idesc = idesc;
    BRing ring;
    ring.full = b_full; ring.empty_a = b_empty_a; ring.base_lo = b_base_lo; ring.stages = prm.b_stages;
    ring.abort_flag = &abort_flag; ring.status = prm.status;
    int a_stage = 0, b_stage = 0, tile_i = 0, buf = 0, use = 0;   // use = tile_i / nbuf; b_stage, b_phase: the leader's
    uint32_t a_phase = 0, b_phase = 0;
    // Layers whose whole contraction is one stage of eighteen or fewer instructions per tile (3x3 taps,
    // weights resident): two tiles per trip.  All four waits come first, then both tiles are issued
    // back to back from one leader region, so the tensor pipe idles between tiles once per pair.
    // Only with four or more activation stages and accumulators: with fewer, waiting for two full stages
    // leaves the loads nothing to overlap with (measured: 57 -> 64 us on a three-stage layer).
    const bool pairs = k3 && resident && prm.chunks == 1 && prm.a_stages >= 4 && nbuf >= 4;
    for (int t = blockIdx.x; pairs && t < num_tiles; t += 2 * gridDim.x) {
      const bool two = t + (int)gridDim.x < num_tiles;
      const int buf0 = buf, use0 = use, st0 = a_stage;
      const uint32_t ph0 = a_phase;
      if (++buf == nbuf) { buf = 0; ++use; }
      if (++a_stage == prm.a_stages) { a_stage = 0; a_phase ^= 1u; }
      const int buf1 = buf, use1 = use, st1 = a_stage;
      const uint32_t ph1 = a_phase;
      if (two) {
        if (++buf == nbuf) { buf = 0; ++use; }
        if (++a_stage == prm.a_stages) { a_stage = 0; a_phase ^= 1u; }
      }
      if (use0 > 0) mbar_wait(&acc_empty[buf0], (uint32_t)(use0 - 1) & 1u, &abort_flag, prm.status);
      mbar_wait(&a_full[st0], ph0, &abort_flag, prm.status);
      if (two) {
        if (use1 > 0) mbar_wait(&acc_empty[buf1], (uint32_t)(use1 - 1) & 1u, &abort_flag, prm.status);
        mbar_wait(&a_full[st1], ph1, &abort_flag, prm.status);
      }
      tc_fence_after();
      if (leader) {
        q.d_tmem = tmem_base + (uint32_t)(buf0 * prm.BN);
        q.a_base = a_ring_lo + (uint32_t)st0 * a_stage_step;
        if (kk_n == 4) issue_taps_resident<3, 3, 4>(q, b_base_lo, 0u);
        else if (kk_n == 2) issue_taps_resident<3, 3, 2>(q, b_base_lo, 0u);
        else issue_taps_resident<3, 3, 1>(q, b_base_lo, 0u);
        tc_commit_a(a_empty_a + 8u * (uint32_t)st0);
        tc_commit(&acc_full[buf0]);
        if (two) {
          q.d_tmem = tmem_base + (uint32_t)(buf1 * prm.BN);
          q.a_base = a_ring_lo + (uint32_t)st1 * a_stage_step;
          if (kk_n == 4) issue_taps_resident<3, 3, 4>(q, b_base_lo, 0u);
          else if (kk_n == 2) issue_taps_resident<3, 3, 2>(q, b_base_lo, 0u);
          else issue_taps_resident<3, 3, 1>(q, b_base_lo, 0u);
          tc_commit_a(a_empty_a + 8u * (uint32_t)st1);
          tc_commit(&acc_full[buf1]);
        }
      }
    }
    for (int t = blockIdx.x; !pairs && t < num_tiles; t += gridDim.x, ++tile_i) {
      if (use > 0) mbar_wait(&acc_empty[buf], (uint32_t)(use - 1) & 1u, &abort_flag, prm.status);
      tc_fence_after();
      q.d_tmem = tmem_base + (uint32_t)(buf * prm.BN);
      for (int c = 0; c < prm.chunks; ++c) {
        mbar_wait(&a_full[a_stage], a_phase, &abort_flag, prm.status);
        tc_fence_after();
        q.a_base = a_ring_lo + (uint32_t)a_stage * a_stage_step;
        if (leader) {
          const uint32_t accumulate = c > 0 ? 1u : 0u;
          const uint32_t bres = b_base_lo + (uint32_t)(c * T) * b_step;
          if (k3 && resident) {
            if (kk_n == 4) issue_taps_resident<3, 3, 4>(q, bres, accumulate);
            else if (kk_n == 2) issue_taps_resident<3, 3, 2>(q, bres, accumulate);
            else issue_taps_resident<3, 3, 1>(q, bres, accumulate);
          } else if (k3) {
            if (kk_n == 4) issue_taps_streamed<3, 3, 4>(q, ring, b_stage, b_phase, accumulate);
            else if (kk_n == 2) issue_taps_streamed<3, 3, 2>(q, ring, b_stage, b_phase, accumulate);
            else issue_taps_streamed<3, 3, 1>(q, ring, b_stage, b_phase, accumulate);
          } else {
            issue_taps_generic(q, prm.R, prm.S, kk_n, resident, bres, ring, b_stage, b_phase, accumulate);
          }
          tc_commit_a(a_empty_a + 8u * (uint32_t)a_stage);
          if (c == prm.chunks - 1) tc_commit(&acc_full[buf]);
        }
        if (++a_stage == prm.a_stages) { a_stage = 0; a_phase ^= 1u; }
      }
      if (++buf == nbuf) { buf = 0; ++use; }
    }
  } else {
    // ---- epilogue: group g = (warp - 2) / 4 drains the CTA's tiles g, g + 2, g + 4, ...; its warp of
    // lane quarter q = warp % 4 reads tensor-memory lanes 32q..32q+31 = tile pixels 32q..32q+31, all columns
    const int quarter = warp & 3;
    const int group = (warp - 2) >> 2;
    const bool nhwc = prm.out.layout == DAI8_NHWC;
    const bool vec_ok = nhwc && (prm.Nout % (prm.out_elem_bytes == 2 ? 8 : 4)) == 0;
    const size_t plane = (size_t)prm.P * prm.Q;
    const float scale = prm.out.dtype == DAI8_I32 ? 0.f : dequant_scale(*prm.sa, *prm.sb);
    uint8_t* my_stage = stage_out + (size_t)(warp - 2) * prm.stage_bufs * kHaloOutBlock;
    const int rows_per_warp = 32 / prm.TX;                 // image rows of the patch one warp covers (1, 2 or 4)
    const int m_lane = quarter * 32 + lane;
    const int yy = m_lane / prm.TX, xx = m_lane - yy * prm.TX;
    int n_store = 0;
    for (int tile_i = group, t = blockIdx.x + group * gridDim.x; t < num_tiles; tile_i += 2, t += 2 * gridDim.x) {
      const int buf = tile_i % nbuf;
      if (!mbar_wait(&acc_full[buf], (uint32_t)(tile_i / nbuf) & 1u, &abort_flag, prm.status)) break;
      tc_fence_after();
      const int m_tile = t / prm.n_tiles;
      const int n0 = (t - m_tile * prm.n_tiles) * prm.BN;
      const int img = m_tile / tiles_per_img, rem = m_tile - img * tiles_per_img;
      const int ty = rem / prm.tiles_x, tx = rem - ty * prm.tiles_x;
      const int y = ty * prm.TY + yy, x = tx * prm.TX + xx;
      const bool inside = y < prm.P && x < prm.Q;
      const size_t opix = (size_t)y * prm.Q + (size_t)x;
      const size_t pix_base = nhwc ? ((size_t)img * plane + opix) * prm.Nout : 0;
      const uint32_t t_tmem = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * prm.BN);
      const int ncols = min(prm.BN, prm.Nout - n0);        // real columns of this tile
      bool released = false;
      auto release = [&]() {        // this warp has read its lanes of the accumulator: hand it back
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&acc_empty[buf]);
        released = true;
      };
      if (prm.tma_store) {
        // 32 pixels x 128 bytes of channels per tile store; the copy engine clips what lies outside the image
        const int cols_per_block = 128 / prm.out_elem_bytes;          // 32 (fp32, int32) or 64 (bf16)
        const int y_warp = ty * prm.TY + quarter * rows_per_warp;     // first image row of this warp's pixels
        const bool rows_inside = y_warp < prm.P;                      // uniform over the warp
        const int nblk = rows_inside ? (ncols + cols_per_block - 1) / cols_per_block : 0;
        for (int blk = 0; blk < nblk; ++blk) {
          const int col = blk * cols_per_block;
          int va[32], vb[32];
          tmem_ld32(t_tmem + (uint32_t)col, va);
          if (prm.out_elem_bytes == 2) tmem_ld32(t_tmem + (uint32_t)(col + 32), vb);
          tmem_ld_wait();
          if (blk == nblk - 1) release();
          uint8_t* st = my_stage + (size_t)(n_store % prm.stage_bufs) * kHaloOutBlock;
          if (n_store >= prm.stage_bufs) {          // the store that last used this block must have read it
            if (lane == 0) { if (prm.stage_bufs == 2) bulk_wait_read<1>(); else bulk_wait_read<0>(); }
            __syncwarp();
          }
          uint8_t* row = st + lane * 128;
          if (prm.out.dtype == DAI8_BF16) {
#pragma unroll
            for (int g = 0; g < 4; ++g) {       // chunk pairs (2g, 2g+1): columns 16g .. 16g+15
              uint32_t w[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const int j = 16 * g + 2 * i;
                const int lo = j < 32 ? va[j & 31] : vb[j & 31], hi = j < 32 ? va[(j + 1) & 31] : vb[(j + 1) & 31];
                w[i] = pack_bf16x2(__fmul_rn(__int2float_rn(lo), scale), __fmul_rn(__int2float_rn(hi), scale));
              }
              *reinterpret_cast<uint4*>(row + (((2 * g) ^ (lane & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
              *reinterpret_cast<uint4*>(row + (((2 * g + 1) ^ (lane & 7)) << 4)) = make_uint4(w[4], w[5], w[6], w[7]);
            }
          } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              uint4 o;
              if (prm.out.dtype == DAI8_F32) {
                o.x = __float_as_uint(__fmul_rn(__int2float_rn(va[4 * i]), scale));
                o.y = __float_as_uint(__fmul_rn(__int2float_rn(va[4 * i + 1]), scale));
                o.z = __float_as_uint(__fmul_rn(__int2float_rn(va[4 * i + 2]), scale));
                o.w = __float_as_uint(__fmul_rn(__int2float_rn(va[4 * i + 3]), scale));
              } else {
                o = make_uint4((uint32_t)va[4 * i], (uint32_t)va[4 * i + 1], (uint32_t)va[4 * i + 2], (uint32_t)va[4 * i + 3]);
              }
              *reinterpret_cast<uint4*>(row + ((i ^ (lane & 7)) << 4)) = o;
            }
          }
          fence_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_store_tile_4d(&mapC, st, (n0 + col) * prm.out_elem_bytes, tx * prm.TX, y_warp, img);
            bulk_commit();
          }
          ++n_store;
        }
      } else {
        const int ngrp = (ncols + 31) / 32;
        for (int cg = 0; cg < ngrp; ++cg) {
          const int col = cg * 32;
          int v[32];
          tmem_ld32(t_tmem + (uint32_t)col, v);
          tmem_ld_wait();
          if (cg == ngrp - 1) release();
          if (!inside) continue;
          const int j0 = n0 + col;
          const int nv = min(32, prm.Nout - j0);       // valid columns of this group
          if (vec_ok) {                                // nv is a multiple of 8 (bf16) or 4
            if (prm.out.dtype == DAI8_F32) {
              float4* dst = reinterpret_cast<float4*>(static_cast<float*>(prm.out.ptr) + pix_base + j0);
#pragma unroll
              for (int i = 0; i < 8; ++i)
                if (4 * i < nv) dst[i] = make_float4(__fmul_rn(__int2float_rn(v[4 * i]), scale), __fmul_rn(__int2float_rn(v[4 * i + 1]), scale),
                                     __fmul_rn(__int2float_rn(v[4 * i + 2]), scale), __fmul_rn(__int2float_rn(v[4 * i + 3]), scale));
            } else if (prm.out.dtype == DAI8_BF16) {
              uint4* dst = reinterpret_cast<uint4*>(static_cast<uint16_t*>(prm.out.ptr) + pix_base + j0);
#pragma unroll
              for (int i = 0; i < 4; ++i)
                if (8 * i < nv) {
                  uint32_t w[4];
#pragma unroll
                  for (int k = 0; k < 4; ++k)
                    w[k] = pack_bf16x2(__fmul_rn(__int2float_rn(v[8 * i + 2 * k]), scale), __fmul_rn(__int2float_rn(v[8 * i + 2 * k + 1]), scale));
                  dst[i] = make_uint4(w[0], w[1], w[2], w[3]);
                }
            } else {
              int4* dst = reinterpret_cast<int4*>(static_cast<int*>(prm.out.ptr) + pix_base + j0);
#pragma unroll
              for (int i = 0; i < 8; ++i) if (4 * i < nv) dst[i] = make_int4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const int j = j0 + i;
              if (j < prm.Nout) {
                const size_t idx = nhwc ? pix_base + j : ((size_t)img * prm.Nout + j) * plane + opix;
                store_result(prm.out.ptr, prm.out.dtype, idx, v[i], scale);
              }
            }
          }
        }
      }
      if (!released) release();      // a tile none of whose columns this warp had to read
    }
    if (prm.tma_store && lane == 0) bulk_wait_read<0>();   // the staging blocks must outlive their stores
  }

  // teardown: everything this CTA issued must have drained before tensor memory is released
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

// Contraction bytes per chunk for a code tensor with `cp` channels (multiple of 16, >= 32).
int halo_chunk_bytes(int cp) {
  if (cp % 128 == 0) return 128;
  if (cp % 64 == 0) return 64;
  if (cp >= 128) return 128;  // ragged tail chunk, zero-filled by the copy engine
  if (cp >= 64) return 64;
  return 32;
}

// Fills the geometry-dependent part of `prm`; false when the kernel does not take the problem.
bool plan_halo(const HaloProblem& pb, dai8_dtype out_dtype, dai8_layout out_layout, HaloParams& prm) {
  if (pb.R * pb.S <= 1 || pb.R > 7 || pb.S > 7) return false;
  if (pb.Kc < 32) return false;
  if ((int64_t)pb.N * pb.H * pb.W * pb.Kc < 131072) return false;
  if (pb.lower_h > 0 || pb.lower_w > 0 || pb.lower_h < -8 || pb.lower_w < -8) return false;
  prm.P = pb.P; prm.Q = pb.Q; prm.Nout = pb.Nout; prm.R = pb.R; prm.S = pb.S;
  // patch shape: the one that computes the fewest positions outside the image (ties: the squarest,
  // which has the smallest halo)
  double best = 1e30;
  for (int tx = 8; tx <= 32; tx *= 2) {
    const int ty = 128 / tx;
    const double w = (double)((pb.Q + tx - 1) / tx * tx) * ((pb.P + ty - 1) / ty * ty) / ((double)pb.P * pb.Q);
    if (w < best - 1e-9) { best = w; prm.TX = tx; prm.TY = ty; }
  }
  // ragged tiles compute positions outside the image: worth it only while that waste stays small
  if (best > 1.16) return false;
  prm.tiles_x = (pb.Q + prm.TX - 1) / prm.TX;
  prm.tiles_y = (pb.P + prm.TY - 1) / prm.TY;
  const int64_t m_tiles = (int64_t)pb.N * prm.tiles_y * prm.tiles_x;
  if (m_tiles > (1 << 30)) return false;
  prm.m_tiles = (int)m_tiles;
  prm.kc_bytes = halo_chunk_bytes(pb.Kc);
  prm.chunks = (pb.Kc + prm.kc_bytes - 1) / prm.kc_bytes;
  const int noutp = round_up(pb.Nout, 16);
  prm.BN = noutp < 256 ? noutp : 256;
  if (noutp > 256 && noutp % 256 != 0 && noutp % 128 == 0) prm.BN = 128;
  prm.n_tiles = (noutp + prm.BN - 1) / prm.BN;
  prm.b_mn = pb.b_mn; prm.b_tap_base = pb.b_tap_base; prm.b_tap_dr = pb.b_tap_dr; prm.b_tap_ds = pb.b_tap_ds;
  prm.b_bw = prm.BN % 128 == 0 ? 128 : (prm.BN % 64 == 0 ? 64 : 32);
  prm.b_nb = prm.BN / prm.b_bw;
  if (pb.b_mn && prm.BN % 32 != 0) return false;
  // accumulators: four while they fit the 512 tensor-memory columns, else two; the epilogue reads whole
  // groups of 64 columns, so the last accumulator is followed by room for its ragged group
  prm.nbuf = prm.BN <= 128 ? 4 : 2;
  prm.tmem_cols = 32;
  while (prm.tmem_cols < (prm.nbuf - 1) * prm.BN + round_up(prm.BN, 64)) prm.tmem_cols *= 2;
  if (prm.tmem_cols > 512) return false;
  prm.lower_h = pb.lower_h; prm.lower_w = pb.lower_w;
  const int out_es = out_dtype == DAI8_BF16 ? 2 : 4;
  prm.out_elem_bytes = out_es;
  const int budget = 227 * 1024 - 2048 - 1024;   // opt-in limit minus static and alignment slack
  const int a_stage = pb.S * (prm.TY + pb.R - 1) * prm.TX * prm.kc_bytes;
  const int b_piece = prm.BN * prm.kc_bytes;
  const int b_all = (pb.R * pb.S * prm.chunks * b_piece + 1023) & ~1023;
  const bool store_ok = out_layout == DAI8_NHWC && (pb.Nout * out_es) % 16 == 0 && pb.Nout * out_es >= 128;
  const int staging1 = kHaloEpiWarps * kHaloOutBlock;
  prm.b_resident = 0; prm.b_stages = 1; prm.tma_store = 0; prm.stage_bufs = 1;
  if (b_all + (store_ok ? staging1 : 0) + 2 * a_stage <= budget) {
    prm.b_resident = 1;
    prm.tma_store = store_ok ? 1 : 0;
    if (store_ok && b_all + 2 * staging1 + 3 * a_stage <= budget) prm.stage_bufs = 2;
    prm.a_stages = (budget - b_all - (store_ok ? prm.stage_bufs * staging1 : 0)) / a_stage;
  } else {
    // streamed weights: two activation stages, the rest of shared memory to the weight ring, stores
    // straight from registers (the staging blocks would cost a weight piece or two).  These layers are
    // bound by the weight traffic from L2, which grows with every wasted position: measured, the
    // wide patches of small images (28 x 28: 4 x 32) lose to the im2col form, 16 x 8 patches win.
    if (prm.TX != 8) return false;
    prm.a_stages = 2;
    prm.b_stages = (budget - 2 * a_stage) / b_piece;
    if (prm.b_stages < 2) return false;
    if (prm.b_stages > kHaloMaxBStages) {
      prm.b_stages = kHaloMaxBStages;
      prm.a_stages = (budget - ((prm.b_stages * b_piece + 1023) & ~1023)) / a_stage;
    }
  }
  if (prm.a_stages > kHaloMaxAStages) prm.a_stages = kHaloMaxAStages;
  if (prm.a_stages < 2) return false;
  return true;
}

}  // namespace

bool halo_supported(const HaloProblem& pb, dai8_dtype out_dtype, dai8_layout out_layout) {
  HaloParams prm;
  return plan_halo(pb, out_dtype, out_layout, prm);
}

dai8_status launch_halo(const HaloProblem& pb, const float* sa, const float* sb, const ConvOut& out, cudaStream_t st) {
  if (!driver_api().ok()) return DAI8_ERR_CUDA;
  HaloParams prm;
  if (!plan_halo(pb, out.dtype, out.layout, prm)) return DAI8_ERR_UNSUPPORTED;
  prm.out = out; prm.sa = sa; prm.sb = sb;
  prm.status = device_status_address();
  if (!prm.status) return DAI8_ERR_CUDA;
  const int out_es = prm.out_elem_bytes;

  CUtensorMap mapA, mapB, mapC;
  memset(&mapC, 0, sizeof(mapC));
  if (prm.tma_store) {
    // output as bytes [N][P][Q][Nout*es], stored in boxes of 32 pixels (32/TX rows x TX columns) x 128 bytes
    const cuuint64_t dims[4] = {(cuuint64_t)pb.Nout * out_es, (cuuint64_t)pb.Q, (cuuint64_t)pb.P, (cuuint64_t)pb.N};
    const cuuint64_t strides[3] = {(cuuint64_t)pb.Nout * out_es, (cuuint64_t)pb.Q * pb.Nout * out_es,
                                   (cuuint64_t)pb.P * pb.Q * pb.Nout * out_es};
    const cuuint32_t box[4] = {128, (cuuint32_t)prm.TX, (cuuint32_t)(32 / prm.TX), 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = encode_tiled_cached(&mapC, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, out.ptr, dims, strides, box, estr, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
    if (r != CUDA_SUCCESS) return DAI8_ERR_CUDA;
  }
  {
    // activations [N][H][W][Kc] in boxes of (TY + R - 1) rows x TX columns x kc channels
    const cuuint64_t dims[4] = {(cuuint64_t)pb.Kc, (cuuint64_t)pb.W, (cuuint64_t)pb.H, (cuuint64_t)pb.N};
    const cuuint64_t strides[3] = {(cuuint64_t)pb.Kc, (cuuint64_t)pb.W * pb.Kc, (cuuint64_t)pb.H * pb.W * pb.Kc};
    const cuuint32_t box[4] = {(cuuint32_t)prm.kc_bytes, (cuuint32_t)prm.TX, (cuuint32_t)(prm.TY + pb.R - 1), 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = encode_tiled_cached(&mapA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<int8_t*>(pb.A), dims, strides, box, estr, swizzle_for(prm.kc_bytes), CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
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
  const int a_stage = pb.S * (prm.TY + pb.R - 1) * prm.TX * prm.kc_bytes;
  const int b_piece = prm.BN * prm.kc_bytes;
  const size_t b_region = (size_t)(((prm.b_resident ? pb.R * pb.S * prm.chunks : prm.b_stages) * b_piece + 1023) & ~1023);
  const size_t smem_bytes = b_region + (prm.tma_store ? kHaloEpiWarps * prm.stage_bufs * kHaloOutBlock : 0) + (size_t)prm.a_stages * a_stage + 1024;
  static std::atomic<int> attr_done[64];
  if (set_max_smem_once(attr_done, igemm_halo_kernel, 227 * 1024 - 2048) != cudaSuccess) return DAI8_ERR_CUDA;
  const int num_tiles = prm.m_tiles * prm.n_tiles;
  int ctas = sm_count();
  if (prm.b_resident && prm.n_tiles > 1) ctas = ctas >= prm.n_tiles ? ctas / prm.n_tiles * prm.n_tiles : prm.n_tiles;
  if (ctas > num_tiles) ctas = num_tiles;
  note_kernel("igemm_halo_kernel");
  log_choice("igemm_halo_kernel: %d x %d patches, N=%d (%d tiles x %d), kc=%d x %d chunks, taps %dx%d, weights %s (%d pieces), A stages %d, %d accumulators, %s, %d CTAs",
             prm.TY, prm.TX, prm.BN, prm.m_tiles, prm.n_tiles, prm.kc_bytes, prm.chunks, prm.R, prm.S,
             prm.b_resident ? "resident" : (prm.b_mn ? "streamed in place" : "streamed"), prm.b_resident ? pb.R * pb.S * prm.chunks : prm.b_stages,
             prm.a_stages, prm.nbuf, prm.tma_store ? "tile stores" : "register stores", ctas);
  DAI8_RETURN_IF_CUDA(launch_dependent(igemm_halo_kernel, dim3((unsigned)ctas), dim3(kHaloThreads), smem_bytes, st, mapA, mapB,
                                       mapC, prm));
  note_launch();
  return DAI8_OK;
}

}  // namespace dai8
