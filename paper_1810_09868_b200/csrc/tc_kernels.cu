// Tensor-core 3x3 convolution for sm_100a: an implicit GEMM on tcgen05 with the
// accumulator in tensor memory, fed by TMA.
//
//   D[pixel][cout] = sum over (r, s, c) of  X[pixel shifted by (r-1, s-1)][c] * Wt[cout][r][s][c]
//
// GEMM view: M = N*H*W output pixels, N = Cout, K = 9*Cin walked as nine filter
// taps times Cin/64 channel blocks.  One CTA computes a 128 (pixels) x BN
// (output channels) tile:
//   warp 0  : TMA producer.  Per K block it issues one im2col load (128 pixels
//             x 64 channels of the NHWC input at tap (r, s); zero padding comes
//             from the hardware's out-of-bounds fill) and one tiled load of the
//             BN x 64 filter slice, into a ring of shared-memory stages.
//   warp 1  : allocates tensor memory; one thread issues tcgen05.mma
//             (128 x BN x 16 per instruction, four per K block) and commits each
//             stage back to the producer and each finished tile to the epilogue.
//   warps 2-5: epilogue.  Each thread owns one pixel row of the tile: it reads
//             the fp32 accumulator from tensor memory 32 columns at a time, adds
//             the bias, applies ReLU and/or the ReLU mask of the layer below,
//             rounds to bf16 and stores to the NHWC output.
// Where the image is a whole number of 16 x 8 pixel patches (the 224x224 and
// 112x112 layers) a tile is such a patch and its input comes from plain tiled
// TMA boxes shifted by the tap, which the copy engine delivers several times
// faster than im2col boxes; elsewhere a tile is 128 consecutive pixels (it may
// span rows and images) fetched in im2col mode.
// The accumulator is double buffered (2 x BN columns of tensor memory) so the
// epilogue of one tile overlaps the main loop of the next; CTAs are persistent
// and walk the tile list with a fixed stride.  Every wait has a time limit.
#include "tc_kernels.cuh"

#include <mutex>

#include <cuda_fp16.h>

#include "tc_common.cuh"

namespace vgg {

// ---- tensor-map plumbing ------------------------------------------------------

const TensorMapApi& tensor_map_api() {
  static TensorMapApi api;
  static std::once_flag once;
  std::call_once(once, [] {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn) return;
    api.encode_tiled = reinterpret_cast<decltype(api.encode_tiled)>(fn);
    fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn) return;
    api.encode_im2col = reinterpret_cast<decltype(api.encode_im2col)>(fn);
    api.ok = true;
  });
  return api;
}

static bool tiled_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_cols,
                      uint32_t box_rows, CUtensorMapSwizzle swizzle) {
  const TensorMapApi& api = tensor_map_api();
  if (!api.ok) return false;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return api.encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_tiled_map_2d(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  return tiled_map(map, base, rows, cols, 64, box_rows, CU_TENSOR_MAP_SWIZZLE_128B);
}

bool make_tiled_map_2d_f32(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  const TensorMapApi& api = tensor_map_api();
  if (!api.ok) return false;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 4};
  cuuint32_t box[2] = {32, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return api.encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_tiled_map_2d_c8(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  return tiled_map(map, base, rows, cols, 8, box_rows, CU_TENSOR_MAP_SWIZZLE_NONE);
}

bool make_patch_map(CUtensorMap* map, const void* base, int N, int H, int W, int C, uint32_t box_w, uint32_t box_h) {
  const TensorMapApi& api = tensor_map_api();
  if (!api.ok) return false;
  cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
  cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)W * C * 2, (cuuint64_t)H * W * C * 2};
  cuuint32_t box[4] = {64, box_w, box_h, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return api.encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_window_map(CUtensorMap* map, const void* base, int N, int H, int W, int C, int a, int b, uint32_t box_w,
                     uint32_t box_h) {
  const TensorMapApi& api = tensor_map_api();
  if (!api.ok || (H & 1) || (W & 1)) return false;
  const char* first = static_cast<const char*>(base) + ((size_t)a * W + b) * C * 2;
  cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W / 2, (cuuint64_t)H / 2, (cuuint64_t)N};
  cuuint64_t strides[3] = {(cuuint64_t)2 * C * 2, (cuuint64_t)2 * W * C * 2, (cuuint64_t)H * W * C * 2};
  cuuint32_t box[4] = {64, box_w, box_h, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return api.encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<char*>(first), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_filter_row_map(CUtensorMap* map, const void* base, int Cout, int Cin, uint32_t box_cout) {
  const TensorMapApi& api = tensor_map_api();
  if (!api.ok) return false;
  cuuint64_t dims[3] = {(cuuint64_t)Cin, (cuuint64_t)Cout, 9};
  cuuint64_t strides[2] = {(cuuint64_t)Cin * 2, (cuuint64_t)Cout * Cin * 2};
  cuuint32_t box[3] = {64, box_cout, 3};
  cuuint32_t estr[3] = {1, 1, 1};
  return api.encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_patch_map_c8(CUtensorMap* map, const void* base, int N, int H, int W, uint32_t box_w, uint32_t box_h) {
  const TensorMapApi& api = tensor_map_api();
  if (!api.ok) return false;
  cuuint64_t dims[4] = {8, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
  cuuint64_t strides[3] = {16, (cuuint64_t)W * 16, (cuuint64_t)H * W * 16};
  cuuint32_t box[4] = {8, box_w, box_h, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return api.encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_im2col_map_c8(CUtensorMap* map, const void* base, int N, int H, int W, uint32_t pixels) {
  const TensorMapApi& api = tensor_map_api();
  if (!api.ok) return false;
  cuuint64_t dims[4] = {8, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
  cuuint64_t strides[3] = {16, (cuuint64_t)W * 16, (cuuint64_t)H * W * 16};
  int lower[2] = {-1, -1};
  int upper[2] = {-1, -1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return api.encode_im2col(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, lower,
                           upper, 8, pixels, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_im2col_map(CUtensorMap* map, const void* base, int N, int H, int W, int C, uint32_t pixels) {
  const TensorMapApi& api = tensor_map_api();
  if (!api.ok) return false;
  cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
  cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)W * C * 2, (cuuint64_t)H * W * C * 2};
  // 3x3 window, padding 1: the window's first tap sits one pixel up/left of the
  // output pixel, and the last tap (first + 2) must still be allowed to reach
  // one pixel past the far edge.
  int lower[2] = {-1, -1};
  int upper[2] = {-1, -1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return api.encode_im2col(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, lower,
                           upper, 64, pixels, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {

using namespace tc;

constexpr int BM = 128;             // pixels per tile (TMEM lanes)
constexpr int BK = 64;              // channels per K block (one 128-byte swizzle row)
constexpr int A_BYTES = BM * BK * 2;
constexpr int kSmemLimit = 227 * 1024;
constexpr int kSplitChunk = 8;      // SPLIT: K blocks (of 64) per accumulation chain in tensor memory: 32 MMAs

// EPI: epilogue groups of four warps, each with its own staging tile and BN / EPI of the tile's columns
template <int BN, int EPI = 1>
struct ConvTile {
  static constexpr int B_BYTES = BN * BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int OUT_BYTES = BM * 64 * 2;  // staging tile of the TMA store: 128 rows x 64 channels
  // leaves room for the staging tiles, barriers, bias and alignment
  static constexpr int STAGES = (kSmemLimit - 4608 - EPI * OUT_BYTES) / STAGE_BYTES > 8 ? 8 : (kSmemLimit - 4608 - EPI * OUT_BYTES) / STAGE_BYTES;
  static constexpr int TMEM_COLS = 2 * BN;  // 128, 256 or 512: powers of two
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI * OUT_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};
// SPLIT with 256-column tiles: two epilogue groups of 128 columns each (the running sums of a tile row live in
// registers: 128 per thread is what fits), 320 threads
template <int BN, bool SPLIT> __host__ __device__ constexpr int conv_epi_groups() { return SPLIT && BN == 256 ? 2 : 1; }
template <int BN, bool SPLIT> __host__ __device__ constexpr int conv_threads() { return 64 + 128 * conv_epi_groups<BN, SPLIT>(); }

struct ConvArgs {
  int pixels;     // N*H*W
  int H, W;
  int cin_blocks; // Cin / 64
  int Cout;
  int m_tiles, n_tiles;
  int relu;
  int patch;      // 1: tiles are 16 x 8 pixel patches loaded with tiled boxes
  int tiles_w, tiles_h;
  const float* bias;
  const bf16* mask;
  bf16* out;
  int* dev_error;
  int split_blocks;  // SPLIT: 64-channel blocks of one term of the input (logical Cin / 64)
};

constexpr int PW = 16, PH = 8;  // patch of a tile in patch mode (PW * PH = BM)

// SPLIT: fp32 convolution as three fp16 products.  Every fp32 value v travels as two fp16 terms, hi = fp16(v) and
// lo = fp16(v - hi), stored per pixel as [hi of all channels | lo of all channels].  The K loop runs over three
// groups of channel blocks per tap: x_hi * w_hi, x_hi * w_lo, x_lo * w_hi (the filter copy holds [w_hi | w_lo | w_hi]
// per tap, of the weights times kSplitWeightScale; the input's channel block wraps back by one term after the
// first group), all into the same fp32 accumulator; the epilogue scales the sum back, adds the bias, applies
// the ReLU, splits the result again and stores the two terms.  A result beyond fp16's range is reported in
// *dev_error (kDevSplitRange).
template <int BN, bool SPLIT>
__global__ void __launch_bounds__((conv_threads<BN, SPLIT>()), 1)
conv3x3_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                  const __grid_constant__ CUtensorMap map_y, ConvArgs a) {
  constexpr int EPI = conv_epi_groups<BN, SPLIT>();
  constexpr int CW = BN / EPI;  // columns of an epilogue group
  using T = ConvTile<BN, EPI>;
  extern __shared__ uint8_t smem_raw[];
  // stage buffers need 1024-byte alignment for the 128-byte swizzle pattern
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t out_smem = smem_base + T::STAGES * T::STAGE_BYTES;  // 1024-byte aligned
  const uint32_t bars = out_smem + EPI * T::OUT_BYTES;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (T::STAGES + s); };
  auto acc_full_bar = [&](int b) { return bars + 8u * (2 * T::STAGES + b); };
  auto acc_empty_bar = [&](int b) { return bars + 8u * (2 * T::STAGES + 2 + b); };
  const uint32_t drain_bar = bars + 8u * (2 * T::STAGES + 4);
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  __shared__ __align__(16) float bias_s[512];  // the layer's bias (zeros when it has none)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int k_blocks = 9 * a.cin_blocks;
  const int total_tiles = a.m_tiles * a.n_tiles;

  for (int i = threadIdx.x; i < a.Cout; i += (int)blockDim.x) bias_s[i] = a.bias ? a.bias[i] : 0.f;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < T::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full_bar(b), 1); mbar_init(acc_empty_bar(b), 128 * EPI); }
    mbar_init(drain_bar, 1);
    mbar_fence_init();
    tma_prefetch_desc(&map_x);
    tma_prefetch_desc(&map_w);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_slot), T::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      uint32_t fills[T::STAGES];
#pragma unroll
      for (int s = 0; s < T::STAGES; ++s) fills[s] = 0;
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const int m_tile = tile / a.n_tiles, n_tile = tile - m_tile * a.n_tiles;
        int w0, h0, n0;
        if (a.patch) {
          const int tw = m_tile % a.tiles_w, t = m_tile / a.tiles_w;
          w0 = tw * PW; h0 = (t % a.tiles_h) * PH; n0 = t / a.tiles_h;
        } else {
          const int p0 = m_tile * BM;
          w0 = p0 % a.W;
          const int t = p0 / a.W;
          h0 = t % a.H; n0 = t / a.H;
        }
        int kb = 0;
        for (int r = 0; r < 3 && ok; ++r)
          for (int s = 0; s < 3 && ok; ++s)
            for (int cb = 0; cb < a.cin_blocks; ++cb, ++kb) {
              if (!mbar_wait(empty_bar(stage), phase ^ 1, &abort_flag, a.dev_error, kDevTimeoutStageFree)) { ok = false; break; }
              const uint32_t sa = smem_base + stage * T::STAGE_BYTES, sb = sa + A_BYTES;
              mbar_expect_tx(full_bar(stage), T::STAGE_BYTES);
              // SPLIT: blocks [0, n) and [n, 2n) read x_hi, blocks [2n, 3n) read x_lo, which sits n blocks after x_hi
              const int xb = SPLIT && cb >= a.split_blocks ? cb - a.split_blocks : cb;
              if (a.patch)
                tma_load_4d(sa, &map_x, full_bar(stage), xb * BK, w0 + s - 1, h0 + r - 1, n0);
              else
                tma_load_im2col_4d(sa, &map_x, full_bar(stage), xb * BK, w0 - 1, h0 - 1, n0, (uint16_t)s, (uint16_t)r);
              tma_load_2d(sb, &map_w, full_bar(stage), kb * BK, n_tile * BN);
              ++fills[stage];
              if (++stage == T::STAGES) { stage = 0; phase ^= 1; }
            }
      }
      if (!ok) {
        // let every copy already in flight land before the CTA may exit
        for (int s = 0; s < T::STAGES; ++s)
          if (fills[s]) {
            const unsigned long long t0 = global_timer_ns();
            while (!mbar_try_wait(full_bar(s), (fills[s] - 1) & 1) && global_timer_ns() - t0 < 100000000ull) {}
          }
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer -------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc = SPLIT ? umma_idesc_f16(BM, BN, 0, 0) : umma_idesc_bf16(BM, BN, 0, 0);
      int stage = 0;
      uint32_t phase = 0;
      int local = 0;
      bool ok = true;
      // one accumulator hand-off per tile, or (SPLIT) per chunk of kSplitChunk K blocks of a tile
      const int chunk = SPLIT ? kSplitChunk : k_blocks;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        for (int kb0 = 0; kb0 < k_blocks && ok; kb0 += chunk, ++local) {
          const int buf = local & 1;
          const uint32_t use = (uint32_t)(local >> 1);  // how many times this buffer was used before
          if (!mbar_wait(acc_empty_bar(buf), (use & 1) ^ 1, &abort_flag, a.dev_error, kDevTimeoutTmemFree)) { ok = false; break; }
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
          const int kb1 = kb0 + chunk < k_blocks ? kb0 + chunk : k_blocks;
          for (int kb = kb0; kb < kb1; ++kb) {
            if (!mbar_wait(full_bar(stage), phase, &abort_flag, a.dev_error, kDevTimeoutTmaFull)) { ok = false; break; }
            tc_fence_after();
            const uint32_t sa = smem_base + stage * T::STAGE_BYTES, sb = sa + A_BYTES;
            // the issue loop is the critical path of the tensor pipe: one descriptor pair per stage,
            // advanced by 32 bytes (16 K elements) with a single add per MMA
            const uint64_t da = smem_desc_sw128(sa, 16), db = smem_desc_sw128(sb, 16);
            umma_bf16(d_tmem, da, db, idesc, kb != kb0 ? 1u : 0u);
#pragma unroll
            for (int k = 1; k < BK / 16; ++k)
              umma_bf16_acc(d_tmem, desc_advance(da, k * 32), desc_advance(db, k * 32), idesc);
            umma_commit(empty_bar(stage));  // frees the stage once these MMAs have read it
            if (++stage == T::STAGES) { stage = 0; phase ^= 1; }
          }
          if (ok) umma_commit(acc_full_bar(buf));
        }
      }
      if (!ok) {
        // wait for the MMAs already issued before shared and tensor memory go away
        umma_commit(drain_bar);
        const unsigned long long t0 = global_timer_ns();
        while (!mbar_try_wait(drain_bar, 0) && global_timer_ns() - t0 < 100000000ull) {}
      }
    }
  } else {
    // -------------------------------- epilogue --------------------------------
    const int quarter = warp & 3;  // the TMEM lane quarter this warp may read
    const int row = quarter * 32 + lane;
    const int grp = EPI == 1 ? 0 : (warp - 2) >> 2;  // epilogue group: columns [grp * CW, (grp + 1) * CW) of the tile
    const int col_base = grp * CW;
    const int bar_id = 1 + grp;
    const uint32_t my_out = out_smem + grp * T::OUT_BYTES;
    int local = 0;
    // The tile leaves 64 channels at a time through a 128-byte-swizzled staging tile and one TMA
    // store (whole 128-byte lines), not as per-thread pieces of rows.  The group's first thread owns its store groups.
    const bool issuer = threadIdx.x == 64 + 128 * grp;
    uint8_t* stage_row = smem_raw + (my_out - smem_u32(smem_raw)) + row * 128;
    bool alive = true;
    for (int tile = blockIdx.x; tile < total_tiles && alive; tile += gridDim.x, ++local) {
      const int m_tile = tile / a.n_tiles, n_tile = tile - m_tile * a.n_tiles;
      // SPLIT: the tensor core's fp32 accumulation truncates, an error that grows with the length of the chain
      // (1.6e-5 after the 864 MMAs of a 512-channel layer).  The K loop therefore hands over its accumulator every
      // kSplitChunk K blocks, and the chunks are added here, in registers, with round-to-nearest fp32 additions.
      float run[SPLIT ? CW : 1];
      if (SPLIT) {
#pragma unroll
        for (int j = 0; j < CW; ++j) run[j] = 0.f;
        for (int kb0 = kSplitChunk; kb0 < k_blocks && alive; kb0 += kSplitChunk, ++local) {
          const int cbuf = local & 1;
          const bool cgot = mbar_wait(acc_full_bar(cbuf), (uint32_t)(local >> 1) & 1, &abort_flag, a.dev_error, kDevTimeoutAccum);
          if (named_bar_or(bar_id, 128, !cgot)) { alive = false; break; }
          tc_fence_after();
#pragma unroll
          for (int cc = 0; cc < CW; cc += 32) {
            uint32_t v[32];
            tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(cbuf * BN + col_base + cc), v);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) run[cc + j] += __uint_as_float(v[j]);
          }
          tc_fence_before();
          mbar_arrive(acc_empty_bar(cbuf));
        }
        if (!alive) break;
      }
      const int buf = local & 1;
      const uint32_t use = (uint32_t)(local >> 1);
      const bool got = mbar_wait(acc_full_bar(buf), use & 1, &abort_flag, a.dev_error, kDevTimeoutAccum);
      if (named_bar_or(bar_id, 128, !got)) break;  // the group's four warps leave together
      tc_fence_after();
      long pixel;
      int tw = 0, th = 0, img = 0;
      if (a.patch) {
        tw = m_tile % a.tiles_w;
        const int t = m_tile / a.tiles_w;
        th = t % a.tiles_h; img = t / a.tiles_h;
        pixel = ((long)img * a.H + th * PH + row / PW) * a.W + tw * PW + row % PW;
      } else {
        pixel = (long)m_tile * BM + row;
      }
      const bool valid = pixel < a.pixels;
      const int c_base = n_tile * BN + col_base;  // first output channel of this group's columns
      const bf16* mask_row = (a.mask && valid) ? a.mask + pixel * a.Cout + c_base : nullptr;
#pragma unroll(SPLIT ? CW / 64 : 1)
      for (int c64 = 0; c64 < CW; c64 += 64) {
        if (issuer) tma_store_wait_read<0>();  // the previous store has read the staging tile
        named_bar_sync(bar_id, 128);
        uint32_t lo_packed[SPLIT ? 32 : 1];
        bool out_of_range = false;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const int cc = c64 + half * 32;
          uint32_t v[32];
          tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN + col_base + cc), v);
          tmem_ld_wait();
          uint32_t packed[16];
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            float x0 = __uint_as_float(v[j]), x1 = __uint_as_float(v[j + 1]);
            if (SPLIT) {
              x0 = (x0 + run[cc + j]) * (1.f / kSplitWeightScale);
              x1 = (x1 + run[cc + j + 1]) * (1.f / kSplitWeightScale);
            }
            x0 += bias_s[c_base + cc + j]; x1 += bias_s[c_base + cc + j + 1];
            if (a.relu) { x0 = fmaxf(x0, 0.f); x1 = fmaxf(x1, 0.f); }
            if (SPLIT) {
              // first term fp16(x); second term: what that rounding left (exact in fp32), rounded to fp16
              out_of_range |= fmaxf(fabsf(x0), fabsf(x1)) > 65504.f;
              __half2 h = __floats2half2_rn(x0, x1);
              __half2 l = __floats2half2_rn(x0 - __low2float(h), x1 - __high2float(h));
              packed[j >> 1] = *reinterpret_cast<uint32_t*>(&h);
              lo_packed[half * 16 + (j >> 1)] = *reinterpret_cast<uint32_t*>(&l);
            } else {
              __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
              packed[j >> 1] = *reinterpret_cast<uint32_t*>(&h);
            }
          }
          if (!SPLIT && mask_row) {
            const uint4* mp = reinterpret_cast<const uint4*>(mask_row + cc);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const uint4 m = __ldg(mp + q);
              const uint32_t mw[4] = {m.x, m.y, m.z, m.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                // a bf16 is > 0 iff its sign bit is clear and it is not zero
                const uint32_t lo = mw[e] & 0xFFFFu, hi = mw[e] >> 16;
                uint32_t keep = 0;
                if (lo != 0 && !(lo & 0x8000u)) keep |= 0x0000FFFFu;
                if (hi != 0 && !(hi & 0x8000u)) keep |= 0xFFFF0000u;
                packed[q * 4 + e] &= keep;
              }
            }
          }
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int chunk = half * 4 + q;  // 16-byte chunk of the 128-byte staging row
            *reinterpret_cast<uint4*>(stage_row + ((chunk ^ (row & 7)) << 4)) =
                make_uint4(packed[q * 4], packed[q * 4 + 1], packed[q * 4 + 2], packed[q * 4 + 3]);
          }
        }
        fence_async_smem();
        named_bar_sync(bar_id, 128);
        if (issuer) {
          // rows past the end of the tensor (last tile) are clipped by the copy engine
          if (a.patch) tma_store_4d(&map_y, my_out, c_base + c64, tw * PW, th * PH, img);
          else tma_store_2d(&map_y, my_out, c_base + c64, m_tile * BM);
          tma_store_commit();
        }
        if (SPLIT) {
          if (out_of_range && valid) atomicCAS(a.dev_error, 0, (int)kDevSplitRange);
          // the second terms of the same 64 channels, Cout channels further on in the pixel's row
          if (issuer) tma_store_wait_read<0>();
          named_bar_sync(bar_id, 128);
#pragma unroll
          for (int chunk = 0; chunk < 8; ++chunk)
            *reinterpret_cast<uint4*>(stage_row + ((chunk ^ (row & 7)) << 4)) =
                make_uint4(lo_packed[chunk * 4], lo_packed[chunk * 4 + 1], lo_packed[chunk * 4 + 2], lo_packed[chunk * 4 + 3]);
          fence_async_smem();
          named_bar_sync(bar_id, 128);
          if (issuer) {
            if (a.patch) tma_store_4d(&map_y, my_out, a.Cout + c_base + c64, tw * PW, th * PH, img);
            else tma_store_2d(&map_y, my_out, a.Cout + c_base + c64, m_tile * BM);
            tma_store_commit();
          }
        }
      }
      tc_fence_before();
      mbar_arrive(acc_empty_bar(buf));
    }
    if (issuer) tma_store_wait_all();  // shared memory must outlive the stores that read it
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, T::TMEM_COLS);
  }
}

template <int BN, bool SPLIT = false>
cudaError_t launch_conv(const CUtensorMap& mx, const CUtensorMap& mw, const CUtensorMap& my, ConvArgs a,
                        cudaStream_t st) {
  using T = ConvTile<BN, conv_epi_groups<BN, SPLIT>()>;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(conv3x3_tc_kernel<BN, SPLIT>, cudaFuncAttributeMaxDynamicSharedMemorySize, T::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int tiles = a.m_tiles * a.n_tiles;
  const int grid = tiles < sms ? tiles : sms;
  conv3x3_tc_kernel<BN, SPLIT><<<grid, conv_threads<BN, SPLIT>(), T::SMEM_BYTES, st>>>(mx, mw, my, a);
  return cudaGetLastError();
}

int pick_bn(int Cout) { return Cout % 256 == 0 ? 256 : (Cout % 128 == 0 ? 128 : 64); }

}  // namespace

bool tc_conv3x3_supported(ConvShape s) {
  return s.Cin % 64 == 0 && s.Cout % 64 == 0 && s.Cout <= 512 && s.H >= 2 && s.W >= 2 && s.N >= 1 &&
         (long)s.N * s.H * s.W < (1L << 31) - 256;
}

cudaError_t tc_conv3x3(const bf16* in, const bf16* wt, const float* bias, const bf16* mask, bf16* out, ConvShape s,
                       bool relu, int* dev_error, cudaStream_t st) {
  if (!tc_conv3x3_supported(s)) return cudaErrorInvalidValue;
  const int BN = pick_bn(s.Cout);
  CUtensorMap mx, mw;
  const bool patch = s.W % PW == 0 && s.H % PH == 0;
  if (patch) {
    if (!make_patch_map(&mx, in, s.N, s.H, s.W, s.Cin, PW, PH)) return cudaErrorInvalidValue;
  } else if (!make_im2col_map(&mx, in, s.N, s.H, s.W, s.Cin, BM)) {
    return cudaErrorInvalidValue;
  }
  if (!make_tiled_map_2d(&mw, wt, (uint64_t)s.Cout, (uint64_t)9 * s.Cin, (uint32_t)BN)) return cudaErrorInvalidValue;
  CUtensorMap my;
  if (patch) {
    if (!make_patch_map(&my, out, s.N, s.H, s.W, s.Cout, PW, PH)) return cudaErrorInvalidValue;
  } else if (!make_tiled_map_2d(&my, out, (uint64_t)s.N * s.H * s.W, (uint64_t)s.Cout, BM)) {
    return cudaErrorInvalidValue;
  }
  ConvArgs a;
  a.patch = patch ? 1 : 0;
  a.tiles_w = s.W / PW; a.tiles_h = s.H / PH;
  a.pixels = s.N * s.H * s.W;
  a.H = s.H; a.W = s.W;
  a.cin_blocks = s.Cin / 64;
  a.Cout = s.Cout;
  a.m_tiles = (a.pixels + BM - 1) / BM;
  a.n_tiles = s.Cout / BN;
  a.relu = relu ? 1 : 0;
  a.bias = bias; a.mask = mask; a.out = out; a.dev_error = dev_error;
  a.split_blocks = 0;
  switch (BN) {
    case 256: return launch_conv<256>(mx, mw, my, a, st);
    case 128: return launch_conv<128>(mx, mw, my, a, st);
    default: return launch_conv<64>(mx, mw, my, a, st);
  }
}

// fp32 convolution from split operands (see the kernel): in [N][H][W][2 * Cin] and out [N][H][W][2 * Cout] hold
// [hi | lo] per pixel, wt_split [Cout][9][3 * Cin] holds [w_hi | w_lo | w_hi] per tap; s has the logical channels.
// (The tensor maps only move 16-bit words: the bf16 ones serve fp16 data.)
cudaError_t tc_conv3x3_split(const half16* in, const half16* wt_split, const float* bias, half16* out, ConvShape s,
                             bool relu, int* dev_error, cudaStream_t st) {
  if (!tc_conv3x3_supported(s)) return cudaErrorInvalidValue;
  // the epilogue keeps a tile row's running sums in registers, 128 per thread: 256-column tiles take two groups of warps
  const int BN = s.Cout % 256 == 0 ? 256 : s.Cout % 128 == 0 ? 128 : 64;
  CUtensorMap mx, mw, my;
  const bool patch = s.W % PW == 0 && s.H % PH == 0;
  if (patch) {
    if (!make_patch_map(&mx, in, s.N, s.H, s.W, 2 * s.Cin, PW, PH)) return cudaErrorInvalidValue;
    if (!make_patch_map(&my, out, s.N, s.H, s.W, 2 * s.Cout, PW, PH)) return cudaErrorInvalidValue;
  } else {
    if (!make_im2col_map(&mx, in, s.N, s.H, s.W, 2 * s.Cin, BM)) return cudaErrorInvalidValue;
    if (!make_tiled_map_2d(&my, out, (uint64_t)s.N * s.H * s.W, (uint64_t)2 * s.Cout, BM)) return cudaErrorInvalidValue;
  }
  if (!make_tiled_map_2d(&mw, wt_split, (uint64_t)s.Cout, (uint64_t)27 * s.Cin, (uint32_t)BN)) return cudaErrorInvalidValue;
  ConvArgs a;
  a.patch = patch ? 1 : 0;
  a.tiles_w = s.W / PW; a.tiles_h = s.H / PH;
  a.pixels = s.N * s.H * s.W;
  a.H = s.H; a.W = s.W;
  a.cin_blocks = 3 * s.Cin / 64;
  a.split_blocks = s.Cin / 64;
  a.Cout = s.Cout;
  a.m_tiles = (a.pixels + BM - 1) / BM;
  a.n_tiles = s.Cout / BN;
  a.relu = relu ? 1 : 0;
  a.bias = bias; a.mask = nullptr; a.out = reinterpret_cast<bf16*>(out); a.dev_error = dev_error;
  return BN == 256 ? launch_conv<256, true>(mx, mw, my, a, st)
         : BN == 128 ? launch_conv<128, true>(mx, mw, my, a, st) : launch_conv<64, true>(mx, mw, my, a, st);
}

namespace {
__global__ void wait_selftest_kernel(int* dev_error, long long limit_cycles) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    tc::mbar_init(tc::smem_u32(&bar), 1);
    tc::mbar_fence_init();
  }
  __syncthreads();
  // phase 0 of a freshly initialised barrier completes only when its one expected arrival comes; none does
  if (threadIdx.x == 0)
    tc::mbar_wait(tc::smem_u32(&bar), 0, &abort_flag, dev_error, kDevTimeoutTest, limit_cycles);
  __syncthreads();
}
}  // namespace

cudaError_t tc_wait_selftest(int* dev_error, long long limit_cycles, cudaStream_t st) {
  wait_selftest_kernel<<<1, 32, 0, st>>>(dev_error, limit_cycles);
  return cudaGetLastError();
}

}  // namespace vgg
