// Tensor-core GEMM for sm_100a (tcgen05 + TMEM + TMA) behind the dense layers
// and the convolution filter gradient:
//
//   D[m][n] = sum_k A(m, k) * B(n, k),   bf16 operands, fp32 accumulation.
//
// Each operand can sit in memory either K-major (a row per m / n, k contiguous:
// activations [batch][features], weights [out][in]) or MN-major (a row per k,
// m / n contiguous: the same matrices used transposed, as the backward pass
// does).  A third form of B reads an NHWC activation through a 3x3 window
// (TMA im2col) with the pixel index as k: that is the filter gradient
//   dW[cout][tap][c] = sum_pixels dz[pixel][cout] * x[pixel shifted by tap][c].
// A fourth form does the same for the 8-channel copy of the 3-channel image
// (16-byte rows, no swizzle; the tile's 80 columns are 10 taps x 8 channels).  There the copy
// engine, at nine small boxes per K block, sets the pace, so a K block is 128 pixels instead of 64:
// A's second 64 x 64 box holds the next 64 pixels instead of output channels 64..127 (the layer has
// 64), which leaves accumulator rows 64..127 meaningless and unread.
//
// One CTA computes one 128 x BN tile over its share of K (grid.y splits K):
//   warp 0 TMA producer, warp 1 TMEM owner + single-thread MMA issuer, warps
//   2-5 epilogue (one tile row per thread, straight from tensor memory).
// With K split, tiles write raw fp32 partial sums and a second kernel adds the
// splits in a fixed order and applies bias / ReLU / mask (deterministic).
// All waits are time-limited (see tc_common.cuh).
//
// The filter gradient can also produce the bias gradient db[m] = sum_k A(m, k): a narrow extra MMA
// multiplies the A tile by a block of ones into 16 spare tensor-memory columns.  The CTAs that share
// an m tile (one per n tile) take turns, K block by K block, so that the extra issue time is spread
// evenly; each writes its part of the sum and the finishing kernel adds the parts in a fixed order.
#include "tc_common.cuh"
#include "tc_kernels.cuh"

namespace vgg {
namespace {

using namespace tc;

enum OperandMode { kKMajor = 0, kMnMajor = 1, kMnMajorIm2col = 2, kMnMajorIm2colC8 = 3 };

constexpr int BM = 128, BK = 64;
constexpr int A_BYTES = BM * BK * 2;
constexpr int GROUP_BYTES = 64 * BK * 2;  // one 64 x 64 box of an MN-major operand
constexpr int kThreads = 192;
constexpr int kMaxStages = 8;

struct GemmArgs {
  int M, N;          // valid rows and columns of D
  int k_blocks;      // ceil(K / 64)
  int kb_per_split;
  int n_tiles;
  int stages;
  int H, W, Cin;     // im2col form of B: column j of D is (tap = j / Cin, channel = j % Cin)
  float* partial;    // split-K: raw sums at partial[(split * M + m) * N + n]; else null
  float* out_f;      // direct epilogue outputs (either may be null), row stride ldc
  bf16* out_h;
  long ldc;
  const float* bias; // per column, or null
  const bf16* mask;  // same shape as the output, or null: keep where mask > 0
  int relu;
  int* dev_error;
  float* db_partial; // column sums of A at db_partial[((split * n_tiles) + n_tile) * M + m], or null
  int tma_store;     // fp32 output (partial or out_f, no bias / ReLU / mask) leaves through staging tiles and map_c
  // Gradient-descent step folded into the epilogue (tma_store path, no split): the tile is a weight
  // gradient that is never stored; out_f / map_c address the fp32 master weights, which become
  // w - lr * D, and sgd_copy receives their bf16 rounding.  lr is read from device memory.
  bf16* sgd_copy;
  const float* sgd_lr;
  // fp32 product from split operands (K-major A, fp16 terms): A holds [hi | lo] per row, a_wrap K blocks each; B
  // holds [hi | lo | hi] of the weights times kSplitWeightScale.  K blocks [0, 2 * a_wrap) read A's hi term (the
  // second group wraps back), the rest its lo term; the sum is scaled back before the bias is added.
  int a_wrap;
};
constexpr int kStoreStagingBytes = 2 * BM * 128;  // two tiles of 128 rows x 32 fp32

// PAIR: two CTAs (a cluster, tcgen05 cta_group::2) compute a 256 x BN tile with one MMA stream; each
// stages its own 128 rows of A and half of the B tile.
// WIDE (pairs only): a second accumulator of 128 columns beside the BN = 256 one, fed by the same A tile - the
// pair's tile is 256 x 384, and the A operand, half of what a pair loads per K block, is loaded once for both.
template <int BN, bool PAIR, bool WIDE = false>
__host__ __device__ constexpr int stage_bytes() {
  // BN = 80 is the 8-channel form, whose K blocks are 128 pixels: ten taps x 128 pixels x 16 bytes
  return BN == 80 ? A_BYTES + 10 * 2048 : A_BYTES + (PAIR ? (BN + (WIDE ? 128 : 0)) / 2 : BN) * BK * 2;
}

template <int BN, int AMODE, int BMODE, bool PAIR, bool WIDE = false>
__global__ void __launch_bounds__(kThreads)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_c, GemmArgs g) {
  static_assert(!PAIR || (AMODE == kMnMajor && BMODE == kMnMajorIm2col && BN % 128 == 0), "pairs: filter gradient only");
  static_assert(!WIDE || (PAIR && BN == 256), "the second accumulator goes with the 256-column pair tile");
  constexpr int BN2 = WIDE ? 128 : 0;   // columns of the second accumulator
  constexpr int BNT = BN + BN2;         // columns of the whole tile
  constexpr int STAGE = stage_bytes<BN, PAIR, WIDE>();
  constexpr int B_GROUPS1 = (PAIR ? BN / 2 : BN) / 64;  // 64-column groups of B this CTA stages for the first accumulator
  constexpr int B_GROUPS = B_GROUPS1 + BN2 / 128;       // ... and in all (one more for the second)
  // filter gradient: 32 spare columns after the tile where the column sums of A can accumulate.  The
  // dense layers need none, and with 256 columns instead of 512 two of their CTAs share an SM.
  constexpr int COLS = BNT + (BMODE == kMnMajorIm2col ? 32 : 0);
  constexpr int TMEM_COLS = COLS <= 64 ? 64 : (COLS <= 128 ? 128 : (COLS <= 256 ? 256 : 512));
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t store_smem = smem_base + g.stages * STAGE;  // 1024-byte aligned: stages are multiples of 1 KB
  const uint32_t bars = store_smem + (g.tma_store ? kStoreStagingBytes : 0);
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (kMaxStages + s); };
  const uint32_t acc_bar = bars + 8u * (2 * kMaxStages);
  const uint32_t drain_bar = bars + 8u * (2 * kMaxStages + 1);
  const uint32_t ones = bars + 256;  // 1 KB of bf16 1.0
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;  // position in the pair; rank 0 issues the MMAs
  const int tile_index = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int m_tile = (tile_index / g.n_tiles) * (PAIR ? 2 : 1) + (int)rank, n_tile = tile_index % g.n_tiles;
  const int m0 = m_tile * BM, n0 = n_tile * BNT;
  const int kb0 = blockIdx.y * g.kb_per_split;
  const int kb1 = min(g.k_blocks, kb0 + g.kb_per_split);
  // K blocks kb = n_tile (mod n_tiles) are the ones whose column sums this CTA adds
  int db_first = kb1;
  if (BMODE == kMnMajorIm2col && g.db_partial) {
    int r = n_tile - kb0 % g.n_tiles;
    if (r < 0) r += g.n_tiles;
    db_first = kb0 + r;
    if (threadIdx.x >= 64) {
      const uint32_t t = threadIdx.x - 64;  // 128 threads x 8 bytes
      asm volatile("st.shared.v2.b32 [%0], {%1, %1};" ::"r"(ones + 8u * t), "r"(0x3F803F80u) : "memory");
    }
    fence_async_smem();
  }

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < g.stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(acc_bar, 1);
    mbar_init(drain_bar, 1);
    mbar_fence_init();
    tma_prefetch_desc(&map_a);
    tma_prefetch_desc(&map_b);
  }
  if (warp == 1) {
    if (PAIR) {
      tmem_alloc_pair(smem_u32(&tmem_base_slot), TMEM_COLS);
      tmem_relinquish_pair();
    } else {
      tmem_alloc(smem_u32(&tmem_base_slot), TMEM_COLS);
      tmem_relinquish();
    }
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();  // the peer's barriers are initialised before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  if (warp == 0) {
    if (lane == 0) {
      uint32_t fills[kMaxStages];
#pragma unroll
      for (int s = 0; s < kMaxStages; ++s) fills[s] = 0;
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      // im2col forms: each 64-column group of the tile is (tap, 64 channels), fixed for the CTA; the
      // pixel a K block starts at advances by 64 per block (no divisions in the loop)
      int grp_c[B_GROUPS > 0 ? B_GROUPS : 1], grp_s[B_GROUPS > 0 ? B_GROUPS : 1], grp_r[B_GROUPS > 0 ? B_GROUPS : 1];
      int w0 = 0, h0 = 0, img = 0;
      if (BMODE == kMnMajorIm2col || BMODE == kMnMajorIm2colC8) {
        if (BMODE == kMnMajorIm2col) {
#pragma unroll
          for (int q = 0; q < B_GROUPS; ++q) {
            // first accumulator: this CTA's half of its BN columns; second: its 64 of the 128 columns that follow
            const int j = q < B_GROUPS1 ? n0 + 64 * ((int)rank * B_GROUPS1 + q) : n0 + BN + 64 * (int)rank, tap = j / g.Cin;
            grp_c[q] = j - tap * g.Cin; grp_r[q] = tap / 3; grp_s[q] = tap - 3 * (tap / 3);
          }
        }
        const long p0 = (long)kb0 * (BMODE == kMnMajorIm2colC8 ? 2 * BK : BK);
        w0 = (int)(p0 % g.W);
        const long t = p0 / g.W;
        h0 = (int)(t % g.H); img = (int)(t / g.H);
      }
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!mbar_wait(empty_bar(stage), phase ^ 1, &abort_flag, g.dev_error, kDevTimeoutStageFree)) { ok = false; break; }
        const uint32_t sa = smem_base + stage * STAGE, sb = sa + A_BYTES;
        if (PAIR) {
          // both CTAs' copies are counted on the issuing CTA's barrier, which announces all their bytes
          const uint32_t full = map_to_cta(full_bar(stage), 0);
          if (rank == 0) mbar_expect_tx(full_bar(stage), 2 * STAGE);
          tma_load_2d_pair(sa, &map_a, full, m0, kb * BK);
          tma_load_2d_pair(sa + GROUP_BYTES, &map_a, full, m0 + 64, kb * BK);
#pragma unroll
          for (int q = 0; q < B_GROUPS; ++q)
            tma_load_im2col_4d_pair(sb + q * GROUP_BYTES, &map_b, full, grp_c[q], w0 - 1, h0 - 1, img,
                                    (uint16_t)grp_s[q], (uint16_t)grp_r[q]);
          w0 += BK;
          while (w0 >= g.W) { w0 -= g.W; if (++h0 == g.H) { h0 = 0; ++img; } }
          ++fills[stage];
          if (++stage == g.stages) { stage = 0; phase ^= 1; }
          continue;
        }
        mbar_expect_tx(full_bar(stage), BMODE == kMnMajorIm2colC8 ? A_BYTES + 9 * 2048 : STAGE);
        if (AMODE == kKMajor) {
          tma_load_2d(sa, &map_a, full_bar(stage), (g.a_wrap && kb >= g.a_wrap ? kb - g.a_wrap : kb) * BK, m0);
        } else if (BMODE == kMnMajorIm2colC8) {
          tma_load_2d(sa, &map_a, full_bar(stage), m0, kb * 2 * BK);
          tma_load_2d(sa + GROUP_BYTES, &map_a, full_bar(stage), m0, kb * 2 * BK + BK);
        } else {
          tma_load_2d(sa, &map_a, full_bar(stage), m0, kb * BK);
          tma_load_2d(sa + GROUP_BYTES, &map_a, full_bar(stage), m0 + 64, kb * BK);
        }
        if (BMODE == kKMajor) {
          tma_load_2d(sb, &map_b, full_bar(stage), kb * BK, n0);
        } else if (BMODE == kMnMajor) {
#pragma unroll
          for (int q = 0; q < BN / 64; ++q) tma_load_2d(sb + q * GROUP_BYTES, &map_b, full_bar(stage), n0 + 64 * q, kb * BK);
        } else if (BMODE == kMnMajorIm2col) {
#pragma unroll
          for (int q = 0; q < BN / 64; ++q)
            tma_load_im2col_4d(sb + q * GROUP_BYTES, &map_b, full_bar(stage), grp_c[q], w0 - 1, h0 - 1, img,
                               (uint16_t)grp_s[q], (uint16_t)grp_r[q]);
        } else {
          // nine taps of the 8-channel image, 128 pixels x 16 bytes each; the tenth slot (columns
          // 72..79 of the tile, never stored) is left as it is
#pragma unroll
          for (int tap = 0; tap < 9; ++tap)
            tma_load_im2col_4d(sb + tap * 2048, &map_b, full_bar(stage), 0, w0 - 1, h0 - 1, img, (uint16_t)(tap % 3),
                               (uint16_t)(tap / 3));
        }
        if (BMODE == kMnMajorIm2col || BMODE == kMnMajorIm2colC8) {
          w0 += BMODE == kMnMajorIm2colC8 ? 2 * BK : BK;
          while (w0 >= g.W) { w0 -= g.W; if (++h0 == g.H) { h0 = 0; ++img; } }
        }
        ++fills[stage];
        if (++stage == g.stages) { stage = 0; phase ^= 1; }
      }
      if (!ok && rank != 0) {
        // the peer's copies report to the issuing CTA's barriers: allow them a millisecond to land
        const unsigned long long t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 1000000ull) {}
      } else if (!ok) {
        for (int s = 0; s < g.stages; ++s)
          if (fills[s]) {
            const unsigned long long t0 = global_timer_ns();
            while (!mbar_try_wait(full_bar(s), (fills[s] - 1) & 1) && global_timer_ns() - t0 < 100000000ull) {}
          }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(PAIR ? 2 * BM : BM, BN, AMODE != kKMajor, BMODE != kKMajor);
      constexpr uint32_t idesc_ones = umma_idesc_bf16(PAIR ? 2 * BM : BM, 16, AMODE != kKMajor, false);
      const uint64_t d_ones = smem_desc_plain(ones, 128, 256);  // every element is 1: the layout is immaterial
      int db_next = db_first;
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!mbar_wait(full_bar(stage), phase, &abort_flag, g.dev_error, kDevTimeoutTmaFull)) { ok = false; break; }
        tc_fence_after();
        const uint32_t sa = smem_base + stage * STAGE, sb = sa + A_BYTES;
        // K-major: 16 k = 32 bytes along the swizzled row.  MN-major: 16 k = 16 rows = 2048 bytes.
        // 8-channel form: 16 k = 16 rows of 16 bytes; 8-row groups 128 bytes apart, taps 2048 bytes apart;
        // eight K steps per block, A's two boxes being consecutive in shared memory.
        constexpr uint32_t a_step = AMODE == kKMajor ? 32 : 2048;
        constexpr uint32_t b_step = BMODE == kKMajor ? 32 : (BMODE == kMnMajorIm2colC8 ? 256 : 2048);
        const uint64_t da = AMODE == kKMajor ? smem_desc_sw128(sa, 16) : smem_desc_sw128(sa, GROUP_BYTES);
        const uint64_t db = BMODE == kKMajor          ? smem_desc_sw128(sb, 16)
                            : BMODE == kMnMajorIm2colC8 ? smem_desc_plain(sb, 128, 2048)
                                                        : smem_desc_sw128(sb, GROUP_BYTES);
        if (PAIR) {
          umma_bf16_pair(tmem_base, da, db, idesc, kb > kb0 ? 1u : 0u);
#pragma unroll
          for (int k = 1; k < BK / 16; ++k)
            umma_bf16_pair_acc(tmem_base, desc_advance(da, k * a_step), desc_advance(db, k * b_step), idesc);
          if (WIDE) {
            // the same A tile against this pair's other 128 columns (one 64-column group per CTA, behind
            // the first accumulator's groups in the stage)
            constexpr uint32_t idesc2 = umma_idesc_bf16(2 * BM, 128, AMODE != kKMajor, BMODE != kKMajor);
            const uint64_t db2 = smem_desc_sw128(sb + B_GROUPS1 * GROUP_BYTES, GROUP_BYTES);
            umma_bf16_pair(tmem_base + BN, da, db2, idesc2, kb > kb0 ? 1u : 0u);
#pragma unroll
            for (int k = 1; k < BK / 16; ++k)
              umma_bf16_pair_acc(tmem_base + BN, desc_advance(da, k * a_step), desc_advance(db2, k * b_step), idesc2);
          }
          if (kb == db_next) {
            umma_bf16_pair(tmem_base + BNT, da, d_ones, idesc_ones, kb != db_first ? 1u : 0u);
#pragma unroll
            for (int k = 1; k < BK / 16; ++k)
              umma_bf16_pair_acc(tmem_base + BNT, desc_advance(da, k * a_step), d_ones, idesc_ones);
            db_next += g.n_tiles;
          }
          umma_commit_pair(empty_bar(stage), 3);  // frees the stage in both CTAs
        } else {
          constexpr int k_steps = BMODE == kMnMajorIm2colC8 ? 2 * BK / 16 : BK / 16;
          // split operands are fp16 (the instruction takes the element type from the descriptor)
          const uint32_t id = g.a_wrap ? umma_idesc_f16(BM, BN, AMODE != kKMajor, BMODE != kKMajor) : idesc;
          umma_bf16(tmem_base, da, db, id, kb > kb0 ? 1u : 0u);
#pragma unroll
          for (int k = 1; k < k_steps; ++k)
            umma_bf16_acc(tmem_base, desc_advance(da, k * a_step), desc_advance(db, k * b_step), id);
          if (kb == db_next) {
            umma_bf16(tmem_base + BN, da, d_ones, idesc_ones, kb != db_first ? 1u : 0u);
#pragma unroll
            for (int k = 1; k < BK / 16; ++k) umma_bf16_acc(tmem_base + BN, desc_advance(da, k * a_step), d_ones, idesc_ones);
            db_next += g.n_tiles;
          }
          umma_commit(empty_bar(stage));
        }
        if (++stage == g.stages) { stage = 0; phase ^= 1; }
      }
      if (ok) {
        if (PAIR) umma_commit_pair(acc_bar, 3); else umma_commit(acc_bar);
      } else {
        if (PAIR) umma_commit_pair(drain_bar, 1); else umma_commit(drain_bar);
        const unsigned long long t0 = global_timer_ns();
        while (!mbar_try_wait(drain_bar, 0) && global_timer_ns() - t0 < 100000000ull) {}
      }
    }
  } else {
    const int quarter = warp & 3;
    const int m = m0 + quarter * 32 + lane;
    const bool row_ok = m < g.M;
    const bool got_acc = mbar_wait(acc_bar, 0, &abort_flag, g.dev_error, kDevTimeoutAccum);
    if (got_acc && g.tma_store) {
      // Raw fp32 tile, 32 columns (one 128-byte line per row) at a time through two alternating
      // 128-byte-swizzled staging tiles and TMA stores: whole lines instead of 128 threads each
      // writing 16-byte pieces of their own rows.  Rows and columns past the tensor are clipped.
      tc_fence_after();
      const bool issuer = threadIdx.x == 64;
      const int row = quarter * 32 + lane;
      const int row0 = (g.partial ? (int)blockIdx.y * g.M : 0) + m0;
      // folded update: this thread's 32 master weights of the next chunk are requested one chunk ahead
      const bool fold = g.sgd_copy != nullptr;
      const float lr = fold ? __ldg(g.sgd_lr) : 0.f;
      const long w_row = (long)m * g.ldc + n0;
      float4 w_next[8];
      auto fetch = [&](int cc) {
        if (row_ok && n0 + cc < g.N) {
#pragma unroll
          for (int q = 0; q < 8; ++q) w_next[q] = __ldg(reinterpret_cast<const float4*>(g.out_f + w_row + cc) + q);
        }
      };
      if (fold) fetch(0);
#pragma unroll 1
      for (int cc = 0; cc < BNT; cc += 32) {
        uint32_t v[32];
        tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)cc, v);
        tmem_ld_wait();
        if (fold) {
          float4 w[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) w[q] = w_next[q];
          if (cc + 32 < BNT) fetch(cc + 32);
          if (row_ok && n0 + cc < g.N) {
            uint32_t h[16];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              const float a0 = fmaf(-lr, __uint_as_float(v[4 * q]), w[q].x), a1 = fmaf(-lr, __uint_as_float(v[4 * q + 1]), w[q].y);
              const float a2 = fmaf(-lr, __uint_as_float(v[4 * q + 2]), w[q].z), a3 = fmaf(-lr, __uint_as_float(v[4 * q + 3]), w[q].w);
              v[4 * q] = __float_as_uint(a0); v[4 * q + 1] = __float_as_uint(a1);
              v[4 * q + 2] = __float_as_uint(a2); v[4 * q + 3] = __float_as_uint(a3);
              __nv_bfloat162 lo = __floats2bfloat162_rn(a0, a1), hi = __floats2bfloat162_rn(a2, a3);
              h[2 * q] = *reinterpret_cast<uint32_t*>(&lo); h[2 * q + 1] = *reinterpret_cast<uint32_t*>(&hi);
            }
            uint4* hp = reinterpret_cast<uint4*>(g.sgd_copy + w_row + cc);
#pragma unroll
            for (int q = 0; q < 4; ++q) hp[q] = make_uint4(h[4 * q], h[4 * q + 1], h[4 * q + 2], h[4 * q + 3]);
          }
        }
        const uint32_t tile = store_smem + (uint32_t)((cc >> 5) & 1) * (BM * 128);
        if (issuer) tma_store_wait_read<1>();  // the store before last has read this staging tile
        named_bar_sync(1, 128);
        uint8_t* dst = smem_raw + (tile - smem_u32(smem_raw)) + row * 128;
#pragma unroll
        for (int q = 0; q < 8; ++q)
          *reinterpret_cast<uint4*>(dst + ((q ^ (row & 7)) << 4)) = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
        fence_async_smem();
        named_bar_sync(1, 128);
        if (issuer && n0 + cc < g.N) {
          tma_store_2d(&map_c, tile, n0 + cc, row0);
          tma_store_commit();
        }
      }
      if (issuer) tma_store_wait_all();
    }
    if (got_acc && !g.tma_store) {
      tc_fence_after();
#pragma unroll 1
      for (int cc = 0; cc < BNT; cc += 32) {
        uint32_t v[32];
        tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)cc, v);
        tmem_ld_wait();
        const int n = n0 + cc;
        if (!row_ok || n >= g.N) continue;
        if (g.partial) {
          float* dst = g.partial + ((long)blockIdx.y * g.M + m) * g.N + n;
#pragma unroll
          for (int j = 0; j < 32; j += 4)
            if (n + j < g.N)
              *reinterpret_cast<float4*>(dst + j) = make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]),
                                                                __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
        } else {
          const long o = (long)m * g.ldc + n;
#pragma unroll
          for (int j = 0; j < 32; j += 8) {
            if (n + j >= g.N) break;
            float x[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              x[e] = __uint_as_float(v[j + e]);
              if (g.a_wrap) x[e] *= 1.f / kSplitWeightScale;
              if (g.bias) x[e] += __ldg(g.bias + n + j + e);
              if (g.relu) x[e] = fmaxf(x[e], 0.f);
            }
            if (g.mask) {
              const uint4 mk = __ldg(reinterpret_cast<const uint4*>(g.mask + o + j));
              const uint32_t mw[4] = {mk.x, mk.y, mk.z, mk.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const uint32_t lo = mw[e] & 0xFFFFu, hi = mw[e] >> 16;
                if (lo == 0 || (lo & 0x8000u)) x[2 * e] = 0.f;
                if (hi == 0 || (hi & 0x8000u)) x[2 * e + 1] = 0.f;
              }
            }
            if (g.out_f) {
              *reinterpret_cast<float4*>(g.out_f + o + j) = make_float4(x[0], x[1], x[2], x[3]);
              *reinterpret_cast<float4*>(g.out_f + o + j + 4) = make_float4(x[4], x[5], x[6], x[7]);
            }
            if (g.out_h) {
              __nv_bfloat162 h0 = __floats2bfloat162_rn(x[0], x[1]), h1 = __floats2bfloat162_rn(x[2], x[3]);
              __nv_bfloat162 h2 = __floats2bfloat162_rn(x[4], x[5]), h3 = __floats2bfloat162_rn(x[6], x[7]);
              *reinterpret_cast<uint4*>(g.out_h + o + j) =
                  make_uint4(*reinterpret_cast<uint32_t*>(&h0), *reinterpret_cast<uint32_t*>(&h1),
                             *reinterpret_cast<uint32_t*>(&h2), *reinterpret_cast<uint32_t*>(&h3));
            }
          }
        }
      }
    }
    if (got_acc) {
      if (BMODE == kMnMajorIm2col && g.db_partial) {
        uint32_t v[32];
        tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)BNT, v);
        tmem_ld_wait();
        if (row_ok)
          g.db_partial[((long)blockIdx.y * g.n_tiles + n_tile) * g.M + m] = db_first < kb1 ? __uint_as_float(v[0]) : 0.f;
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  // a pair meets before either CTA releases tensor memory or exits: until then the peer may still
  // signal this CTA's barriers, and the issuing CTA's MMAs read the peer's shared memory
  if (PAIR) cluster_sync_all();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    if (PAIR) tmem_dealloc_pair(tmem_base, TMEM_COLS); else tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// out = epilogue(sum over splits of partial[split]), four columns per thread
__global__ void splitk_finish_kernel(const float* __restrict__ partial, int splits, long MN, int N,
                                     const float* __restrict__ bias, int relu, const bf16* __restrict__ mask,
                                     bf16* out_h, float* out_f, const float* __restrict__ db_partial, int db_parts,
                                     int M, float* db, float scale) {
  const long t = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (db && t < M) {
    float s = 0.f;
    for (int z = 0; z < db_parts; ++z) s += db_partial[(long)z * M + t];
    db[t] = s;
  }
  const long i = t * 4;
  if (i >= MN) return;
  // independent loads, issued several at a time; the additions stay in split order
  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
  int z = 0;
  for (; z + 4 <= splits; z += 4) {
    float4 p[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) p[u] = *reinterpret_cast<const float4*>(partial + (long)(z + u) * MN + i);
#pragma unroll
    for (int u = 0; u < 4; ++u) { s.x += p[u].x; s.y += p[u].y; s.z += p[u].z; s.w += p[u].w; }
  }
  for (; z < splits; ++z) {
    const float4 p = *reinterpret_cast<const float4*>(partial + (long)z * MN + i);
    s.x += p.x; s.y += p.y; s.z += p.z; s.w += p.w;
  }
  float x[4] = {s.x, s.y, s.z, s.w};
  const int n = (int)(i % N);
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    x[e] *= scale;  // 1 except for sums of split operands
    if (bias) x[e] += bias[n + e];
    if (relu) x[e] = fmaxf(x[e], 0.f);
    if (mask && !(__bfloat162float(mask[i + e]) > 0.f)) x[e] = 0.f;
  }
  if (out_f) *reinterpret_cast<float4*>(out_f + i) = make_float4(x[0], x[1], x[2], x[3]);
  if (out_h) {
    __nv_bfloat162 h0 = __floats2bfloat162_rn(x[0], x[1]), h1 = __floats2bfloat162_rn(x[2], x[3]);
    *reinterpret_cast<uint2*>(out_h + i) = make_uint2(*reinterpret_cast<uint32_t*>(&h0), *reinterpret_cast<uint32_t*>(&h1));
  }
}

int sm_count() {
  static int sms = 0;
  if (!sms) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (sms <= 0) sms = 148;
  }
  return sms;
}

// K split: as many CTAs as fit in one wave (one CTA per SM: a second, partial wave would leave most
// SMs idle for its whole duration), never an empty split.
void plan_split(int mn_tiles, int k_blocks, int* splits, int* kb_per_split, int ctas_per_tile = 1) {
  int want = sm_count() / ctas_per_tile / mn_tiles;
  if (want < 1) want = 1;
  if (want > k_blocks) want = k_blocks;
  int per = (k_blocks + want - 1) / want;
  *kb_per_split = per;
  *splits = (k_blocks + per - 1) / per;
}

// m_tiles counts tiles of 128 rows, or of 256 rows (CTA pairs) with PAIR
template <int BN, int AMODE, int BMODE, bool PAIR = false, bool WIDE = false>
cudaError_t launch_gemm_tc(const CUtensorMap& ma, const CUtensorMap& mb, GemmArgs g, int m_tiles, int splits,
                           cudaStream_t st) {
  constexpr int STAGE = stage_bytes<BN, PAIR, WIDE>();
  constexpr int kExtra = 1024 + 256 + 1024;  // alignment slack, barriers, block of ones
  // Raw fp32 output (split-K partial sums, or a result without bias / ReLU / mask) leaves by TMA store
  // where whole 128-row boxes cannot run into rows that belong to someone else: a single result
  // matrix (the copy engine clips at its end), or partial sums stacked per split with M a multiple
  // of 128, or M = 64 (box of 64 rows).
  float* target = g.partial ? g.partial : g.out_f;
  const bool plain = !g.bias && !g.relu && !g.mask && !g.out_h && target != nullptr;
  const long out_rows = g.partial ? (long)splits * g.M : g.M;
  const int out_cols = g.partial ? g.N : (int)g.ldc;
  CUtensorMap mc = ma;  // unused unless tma_store
  g.tma_store = 0;
  if (plain && out_cols % 4 == 0 && (!g.partial || g.M % BM == 0 || g.M == 64) &&
      make_tiled_map_2d_f32(&mc, target, (uint64_t)out_rows, (uint64_t)out_cols, g.M == 64 ? 64 : BM))
    g.tma_store = 1;
  if (g.sgd_copy && !g.tma_store) return cudaErrorInvalidValue;  // the folded update lives in that epilogue only
  constexpr int kBudget = 227 * 1024 - 3072 - kStoreStagingBytes;
  constexpr int max_stages = kBudget / STAGE > kMaxStages ? kMaxStages : kBudget / STAGE;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<BN, AMODE, BMODE, PAIR, WIDE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         max_stages * STAGE + kExtra + kStoreStagingBytes);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  g.stages = g.kb_per_split < max_stages ? g.kb_per_split : max_stages;
  const size_t smem = (size_t)g.stages * STAGE + kExtra + (g.tma_store ? kStoreStagingBytes : 0);
  if (PAIR) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * m_tiles * g.n_tiles, splits);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<BN, AMODE, BMODE, PAIR, WIDE>, ma, mb, mc, g);
  }
  dim3 grid(m_tiles * g.n_tiles, splits);
  gemm_tc_kernel<BN, AMODE, BMODE, PAIR, WIDE><<<grid, kThreads, smem, st>>>(ma, mb, mc, g);
  return cudaGetLastError();
}

cudaError_t finish(const GemmArgs& g, int splits, const float* bias, bool relu, const bf16* mask, bf16* out_h,
                   float* out_f, cudaStream_t st, float* db = nullptr) {
  const long MN = (long)g.M * g.N;
  splitk_finish_kernel<<<(unsigned)((MN / 4 + 255) / 256), 256, 0, st>>>(g.partial, splits, MN, g.N, bias, relu ? 1 : 0,
                                                                          mask, out_h, out_f, g.db_partial,
                                                                          splits * g.n_tiles, g.M, db,
                                                                          g.a_wrap ? 1.f / kSplitWeightScale : 1.f);
  return cudaGetLastError();
}

__global__ void db_finish_kernel(const float* __restrict__ db_partial, int parts, int M, float* db) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= M) return;
  float s = 0.f;
  for (int z = 0; z < parts; ++z) s += db_partial[(long)z * M + t];
  db[t] = s;
}

}  // namespace

// ---- dense layers ------------------------------------------------------------

bool tc_dense_supported(int M, int In, int Out) {
  return M >= 1 && In % 8 == 0 && Out % 8 == 0 && In >= 64 && Out >= 64;
}

size_t tc_dense_scratch_elems(int M, int In, int Out) {
  // forward and input-gradient both split K; bound both
  size_t worst = 0;
  const int shapes[2][2] = {{Out, In}, {In, Out}};  // {N, K}
  for (auto& s : shapes) {
    int splits, per;
    plan_split(((M + BM - 1) / BM) * ((s[0] + 127) / 128), (s[1] + BK - 1) / BK, &splits, &per);
    size_t e = (size_t)splits * M * s[0];
    if (e > worst) worst = e;
  }
  return worst;
}

// Y = [relu](X W^T + b): X [M][In], W [Out][In]
cudaError_t tc_dense_forward(const bf16* X, const bf16* Wt, const float* bias, bf16* out_h, float* out_f,
                             float* partial, int M, int In, int Out, bool relu, int* dev_error, cudaStream_t st) {
  CUtensorMap ma, mb;
  if (!make_tiled_map_2d(&ma, X, (uint64_t)M, (uint64_t)In, BM)) return cudaErrorInvalidValue;
  if (!make_tiled_map_2d(&mb, Wt, (uint64_t)Out, (uint64_t)In, 128)) return cudaErrorInvalidValue;
  GemmArgs g{};
  g.M = M; g.N = Out; g.k_blocks = (In + BK - 1) / BK; g.n_tiles = (Out + 127) / 128;
  g.dev_error = dev_error; g.ldc = Out;
  const int m_tiles = (M + BM - 1) / BM;
  int splits;
  plan_split(m_tiles * g.n_tiles, g.k_blocks, &splits, &g.kb_per_split);
  if (splits == 1) {
    g.bias = bias; g.relu = relu; g.out_h = out_h; g.out_f = out_f;
    return launch_gemm_tc<128, kKMajor, kKMajor>(ma, mb, g, m_tiles, 1, st);
  }
  g.partial = partial;
  cudaError_t e = launch_gemm_tc<128, kKMajor, kKMajor>(ma, mb, g, m_tiles, splits, st);
  if (e != cudaSuccess) return e;
  return finish(g, splits, bias, relu, nullptr, out_h, out_f, st);
}

constexpr int kSplitChunkBlocks = 8;
// fp32 Y = [relu](X W^T + b) from split operands: X [M][2 * In] = [x_hi | x_lo], Ws [Out][3 * In] =
// [w_hi | w_lo | w_hi] (fp16 terms); three products x_hi w_hi + x_hi w_lo + x_lo w_hi in one fp32 accumulator
cudaError_t tc_dense_forward_split(const half16* X, const half16* Ws, const float* bias, float* out_f, float* partial,
                                   int M, int In, int Out, bool relu, int* dev_error, cudaStream_t st) {
  if (In % BK != 0) return cudaErrorInvalidValue;
  CUtensorMap ma, mb;
  if (!make_tiled_map_2d(&ma, X, (uint64_t)M, (uint64_t)2 * In, BM)) return cudaErrorInvalidValue;
  if (!make_tiled_map_2d(&mb, Ws, (uint64_t)Out, (uint64_t)3 * In, 128)) return cudaErrorInvalidValue;
  GemmArgs g{};
  g.M = M; g.N = Out; g.k_blocks = 3 * In / BK; g.n_tiles = (Out + 127) / 128; g.a_wrap = In / BK;
  g.dev_error = dev_error; g.ldc = Out;
  const int m_tiles = (M + BM - 1) / BM;
  // The tensor core's fp32 accumulation truncates, an error that grows with the length of the chain: K is cut
  // into splits of kSplitChunkBlocks blocks (32 MMAs) whatever the tile count, and the finishing kernel adds
  // the partial sums with round-to-nearest fp32 additions.
  g.kb_per_split = kSplitChunkBlocks;
  const int splits = (g.k_blocks + kSplitChunkBlocks - 1) / kSplitChunkBlocks;
  g.partial = partial;
  cudaError_t e = launch_gemm_tc<128, kKMajor, kKMajor>(ma, mb, g, m_tiles, splits, st);
  if (e != cudaSuccess) return e;
  return finish(g, splits, bias, relu, nullptr, nullptr, out_f, st);
}

size_t tc_dense_split_scratch_elems(int M, int In, int Out) {
  return (size_t)((3 * In / BK + kSplitChunkBlocks - 1) / kSplitChunkBlocks) * M * Out;
}

// dX = (dY W) [* (mask > 0)]: dY [M][Out], W [Out][In]
cudaError_t tc_dense_dx(const bf16* dY, const bf16* Wt, const bf16* mask, bf16* dX, float* partial, int M, int In,
                        int Out, int* dev_error, cudaStream_t st) {
  CUtensorMap ma, mb;
  if (!make_tiled_map_2d(&ma, dY, (uint64_t)M, (uint64_t)Out, BM)) return cudaErrorInvalidValue;
  if (!make_tiled_map_2d(&mb, Wt, (uint64_t)Out, (uint64_t)In, 64)) return cudaErrorInvalidValue;
  GemmArgs g{};
  g.M = M; g.N = In; g.k_blocks = (Out + BK - 1) / BK; g.n_tiles = (In + 127) / 128;
  g.dev_error = dev_error; g.ldc = In;
  const int m_tiles = (M + BM - 1) / BM;
  int splits;
  plan_split(m_tiles * g.n_tiles, g.k_blocks, &splits, &g.kb_per_split);
  if (splits == 1) {
    g.mask = mask; g.out_h = dX;
    return launch_gemm_tc<128, kKMajor, kMnMajor>(ma, mb, g, m_tiles, 1, st);
  }
  g.partial = partial;
  cudaError_t e = launch_gemm_tc<128, kKMajor, kMnMajor>(ma, mb, g, m_tiles, splits, st);
  if (e != cudaSuccess) return e;
  return finish(g, splits, nullptr, false, mask, dX, nullptr, st);
}

// dW = dY^T X: dY [M][Out], X [M][In] -> dW fp32 [Out][In]
cudaError_t tc_dense_dw(const bf16* dY, const bf16* X, float* dW, int M, int In, int Out, int* dev_error,
                        cudaStream_t st, bf16* sgd_copy, const float* sgd_lr) {
  if ((sgd_copy != nullptr) && (sgd_lr == nullptr || In % 32 != 0)) return cudaErrorInvalidValue;
  CUtensorMap ma, mb;
  if (!make_tiled_map_2d(&ma, dY, (uint64_t)M, (uint64_t)Out, 64)) return cudaErrorInvalidValue;
  if (!make_tiled_map_2d(&mb, X, (uint64_t)M, (uint64_t)In, 64)) return cudaErrorInvalidValue;
  GemmArgs g{};
  g.M = Out; g.N = In; g.k_blocks = (M + BK - 1) / BK; g.kb_per_split = g.k_blocks;
  g.dev_error = dev_error; g.ldc = In; g.out_f = dW;
  g.sgd_copy = sgd_copy; g.sgd_lr = sgd_lr;
  const int m_tiles = (Out + BM - 1) / BM;
  // 128-column tiles: two of these one-tile CTAs fit an SM (98 KB of shared memory, 128 tensor-memory
  // columns each), so one's prologue and loads hide behind the other's 64 KB store
  g.n_tiles = (In + 127) / 128;
  return launch_gemm_tc<128, kMnMajor, kMnMajor>(ma, mb, g, m_tiles, 1, st);
}

// ---- convolution filter gradient ----------------------------------------------

namespace {
// 9*Cin columns in tiles of whole 64-channel groups: 256 or 128 wide, and 192 (three taps) for 64 channels
// 192 columns (three 64-channel groups) divide 9*Cin for every Cin that is a multiple of 64; with 128
// input channels they measured faster than 128-column tiles, CTA pairs included (0.43 -> 0.34 ms on layer 4)
int wgrad_bn(int Cin) { return Cin % 256 == 0 ? 256 : 192; }
// CTA pairs take 256 output channels and 384 columns per tile (two accumulators, 256 and 128 columns wide, fed by
// one dz tile); 9 * Cin divides into such tiles when Cin is a multiple of 128
bool wgrad_pair(ConvShape s, bool pairs) { return pairs && s.Cout % 256 == 0 && s.Cin % 128 == 0; }
// m_tiles: tiles of 128 output channels, or of 256 with CTA pairs
void wgrad_plan(ConvShape s, bool pairs, int* m_tiles, int* n_tiles, int* k_blocks, int* splits, int* per) {
  const long P = (long)s.N * s.H * s.W;
  const bool pair = wgrad_pair(s, pairs);
  *m_tiles = pair ? s.Cout / 256 : (s.Cout + BM - 1) / BM;
  *n_tiles = pair ? 9 * s.Cin / 384 : 9 * s.Cin / wgrad_bn(s.Cin);
  *k_blocks = (int)((P + BK - 1) / BK);
  plan_split(*m_tiles * *n_tiles, *k_blocks, splits, per, pair ? 2 : 1);
}
}  // namespace

bool tc_wgrad_supported(ConvShape s) {
  return s.Cin % 64 == 0 && s.Cout % 64 == 0 && s.H >= 2 && s.W >= 2 && (long)s.N * s.H * s.W < (1L << 31) - 256;
}

size_t tc_wgrad_scratch_elems(ConvShape s, bool pairs) {
  if (!tc_wgrad_supported(s)) return 0;
  int mt, nt, kb, splits, per;
  wgrad_plan(s, pairs, &mt, &nt, &kb, &splits, &per);
  return (size_t)splits * s.Cout * 9 * s.Cin + (size_t)splits * nt * s.Cout;
}

int tc_wgrad_launches(ConvShape s, bool with_db, bool pairs) {
  int mt, nt, kb, splits, per;
  wgrad_plan(s, pairs, &mt, &nt, &kb, &splits, &per);
  return splits > 1 || with_db ? 2 : 1;
}

// dW[k][tap][c] = sum_pixels dz[pixel][k] * x[pixel + tap][c]   (fp32 out, [Cout][9*Cin]);
// db[k] = sum_pixels dz[pixel][k] when db is not null
cudaError_t tc_conv3x3_wgrad(const bf16* x, const bf16* dz, float* dW, float* db, float* partial, ConvShape s,
                             int* dev_error, cudaStream_t st, bool pairs) {
  if (!tc_wgrad_supported(s)) return cudaErrorInvalidValue;
  const long P = (long)s.N * s.H * s.W;
  const int BN = wgrad_bn(s.Cin);
  CUtensorMap ma, mb;
  if (!make_tiled_map_2d(&ma, dz, (uint64_t)P, (uint64_t)s.Cout, 64)) return cudaErrorInvalidValue;
  if (!make_im2col_map(&mb, x, s.N, s.H, s.W, s.Cin, 64)) return cudaErrorInvalidValue;
  GemmArgs g{};
  int m_tiles, splits;
  wgrad_plan(s, pairs, &m_tiles, &g.n_tiles, &g.k_blocks, &splits, &g.kb_per_split);
  g.M = s.Cout; g.N = 9 * s.Cin; g.H = s.H; g.W = s.W; g.Cin = s.Cin;
  g.dev_error = dev_error; g.ldc = g.N;
  if (splits == 1) g.out_f = dW; else g.partial = partial;
  if (db) g.db_partial = partial + (splits == 1 ? 0 : (size_t)splits * s.Cout * 9 * s.Cin);
  cudaError_t e;
  const bool pair = wgrad_pair(s, pairs);
  if (pair) e = launch_gemm_tc<256, kMnMajor, kMnMajorIm2col, true, true>(ma, mb, g, m_tiles, splits, st);
  else if (BN == 256) e = launch_gemm_tc<256, kMnMajor, kMnMajorIm2col>(ma, mb, g, m_tiles, splits, st);
  else e = launch_gemm_tc<192, kMnMajor, kMnMajorIm2col>(ma, mb, g, m_tiles, splits, st);
  if (e != cudaSuccess) return e;
  if (splits == 1) {
    if (!db) return e;
    db_finish_kernel<<<(s.Cout + 255) / 256, 256, 0, st>>>(g.db_partial, g.n_tiles, s.Cout, db);
    return cudaGetLastError();
  }
  return finish(g, splits, nullptr, false, nullptr, nullptr, dW, st, db);
}

// ---- filter gradient of the first layer (3 channels, read from the 8-channel copy) ----

namespace {
// dW[k][tap][c] = sum over splits of partial[split][k][tap * 8 + c], c < 3.  Channel 3 of the
// 8-channel image is the constant 1, so column (centre tap, channel 3) is sum_pixels dz[pixel][k]:
// the bias gradient.
// One warp per output: lanes take the splits round-robin and a butterfly adds the lanes (a fixed order).
__global__ void wgrad_c8_finish_kernel(const float* __restrict__ partial, int splits, int Cout, float* dW, float* db) {
  const int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  const int n_dw = Cout * 27;
  if (i >= n_dw + Cout) return;  // whole warps leave together
  long col;
  float* dst;
  if (i < n_dw) {
    const int c = i % 3, tap = (i / 3) % 9, k = i / 27;
    col = (long)k * 80 + tap * 8 + c;
    dst = dW + i;
  } else {
    col = (long)(i - n_dw) * 80 + 4 * 8 + 3;
    dst = db ? db + (i - n_dw) : nullptr;
  }
  float s = 0.f;
  for (int z = lane; z < splits; z += 32) s += partial[(long)z * Cout * 80 + col];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0 && dst) *dst = s;
}
void wgrad_c8_plan(ConvShape s, int* k_blocks, int* splits, int* per) {
  const long P = (long)s.N * s.H * s.W;
  *k_blocks = (int)((P + 2 * BK - 1) / (2 * BK));  // K blocks of 128 pixels
  plan_split(1, *k_blocks, splits, per);
}
}  // namespace

size_t tc_first_wgrad_scratch_elems(ConvShape s) {
  int kb, splits, per;
  wgrad_c8_plan(s, &kb, &splits, &per);
  return (size_t)splits * s.Cout * 80;
}

cudaError_t tc_first_wgrad(const bf16* x8, const bf16* dz, float* dW, float* db, float* partial, ConvShape s, int* dev_error,
                           cudaStream_t st) {
  const long P = (long)s.N * s.H * s.W;
  CUtensorMap ma, mb;
  if (!make_tiled_map_2d(&ma, dz, (uint64_t)P, (uint64_t)s.Cout, 64)) return cudaErrorInvalidValue;
  if (!make_im2col_map_c8(&mb, x8, s.N, s.H, s.W, 128)) return cudaErrorInvalidValue;
  GemmArgs g{};
  int splits;
  wgrad_c8_plan(s, &g.k_blocks, &splits, &g.kb_per_split);
  g.M = s.Cout; g.N = 80; g.n_tiles = 1; g.H = s.H; g.W = s.W; g.Cin = 8;
  g.dev_error = dev_error; g.ldc = 80; g.partial = partial;
  cudaError_t e = launch_gemm_tc<80, kMnMajor, kMnMajorIm2colC8>(ma, mb, g, 1, splits, st);
  if (e != cudaSuccess) return e;
  wgrad_c8_finish_kernel<<<(s.Cout * 28 * 32 + 255) / 256, 256, 0, st>>>(partial, splits, s.Cout, dW, db);
  return cudaGetLastError();
}

}  // namespace vgg
