// First convolution layer (3 input channels) on tensor cores.
//
// With 3 channels a pixel is 6 bytes, below TMA's 16-byte granule, so the image
// is first copied into an 8-channel tensor (channel 3 one, channels 4..7 zero;
// the filter is zero there, and the constant channel lets the filter-gradient
// GEMM produce the bias gradient as one more column).  The layer is
// then the implicit GEMM  D[pixel][cout] = sum_{tap, c<8} X8[pixel + tap][c] * W8[cout][tap][c]
// with K = 10 taps x 8 channels = 80 (tap 9 is zero padding so that K is a
// multiple of the MMA depth 16).  One K step of an MMA is two taps: each tap is
// its own TMA im2col box of 128 pixels x 8 channels (16-byte rows, no swizzle),
// i.e. exactly the 8x16-byte core-matrix layout tcgen05 reads without swizzle.
// Where the image is a whole number of 8 x 16 pixel patches, a tile is such a
// patch and its 10 x 18 input patch (with halo) arrives as ONE tiled box of 180
// 16-byte rows instead of nine boxes of 128; tap (r, s) then starts r*10 + s
// rows into that buffer, 8-row groups are 10 rows apart, and the two taps of a
// K step are 1 row (or, across a row change, 8 rows) apart.
// The layer is bound by writing its output (128 bytes per pixel), not by math.
//
// Roles and pipeline are those of the general convolution kernel: warp 0 TMA
// producer, warp 1 MMA issuer and TMEM owner, then epilogue warps; double-buffered
// accumulator; persistent CTAs; time-limited waits.  The main loop is five MMAs
// per tile, so the epilogue sets the pace: three groups of eight epilogue warps take
// tiles in turn (each group its own accumulator buffer, staging tile and named
// barrier), so that one tile's chain of wait, tensor-memory load, conversion, staging
// and store overlaps the next tile's; within a group two warps per TMEM lane quarter
// each convert and store 32 of the 64 output channels of their rows.
#include "tc_common.cuh"
#include "tc_kernels.cuh"

namespace vgg {
namespace {

using namespace tc;

constexpr int BM = 128, BN = 64;
constexpr int TAP_BYTES = BM * 16;        // 128 pixels x 8 channels
constexpr int STAGE_BYTES = 10 * TAP_BYTES;
constexpr int STAGES = 8;
constexpr int W_TAP_BYTES = BN * 16;      // 64 output channels x 8 channels
constexpr int W_BYTES = 10 * W_TAP_BYTES;
constexpr int OUT_TILE_BYTES = BM * BN * 2;  // 16 KB staging tile for the TMA store, two of them
constexpr int kGroups = 3;     // epilogue groups, each with its own accumulator buffer and staging tile
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + kGroups * OUT_TILE_BYTES + W_BYTES + 1024 + 256;
constexpr int kGroupThreads = 256;
constexpr int kThreads = 64 + kGroups * kGroupThreads;  // producer, MMA issuer, the groups of eight epilogue warps
constexpr int kTmemCols = 256;  // kGroups accumulators of 64 columns, rounded up to a power of two

constexpr int PW = 8, PH = 16, IW = PW + 2, IH = PH + 2;  // patch mode: output patch and input patch with halo
constexpr int PATCH_BYTES = IW * IH * 16;                 // 2880
constexpr int PATCH_ROWS_READ = 184;                      // the padding tap reads up to row 181

struct FirstArgs {
  int pixels, H, W, m_tiles, relu;
  int patch, tiles_w, tiles_h;
  const float* bias;
  bf16* out;
  int* dev_error;
};

__global__ void __launch_bounds__(kThreads, 1)
conv3x3_c8_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                     const __grid_constant__ CUtensorMap map_y, FirstArgs a) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t out_smem = smem_base + STAGES * STAGE_BYTES;  // 1024-byte aligned (20 KB stages)
  const uint32_t w_smem = out_smem + kGroups * OUT_TILE_BYTES;
  const uint32_t bars = w_smem + W_BYTES;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
  auto acc_full_bar = [&](int b) { return bars + 8u * (2 * STAGES + b); };
  auto acc_empty_bar = [&](int b) { return bars + 8u * (2 * STAGES + kGroups + b); };
  const uint32_t w_bar = bars + 8u * (2 * STAGES + 2 * kGroups);
  const uint32_t drain_bar = bars + 8u * (2 * STAGES + 2 * kGroups + 1);
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  __shared__ __align__(16) float bias_s[512];  // the layer's bias (zeros when it has none)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // the padding tap of every stage is multiplied by zero weights: it must hold finite numbers
  {
    uint8_t* base = smem_raw + (smem_base - smem_u32(smem_raw));
    for (int i = threadIdx.x; i < STAGES * (TAP_BYTES / 16); i += kThreads) {
      const int s = i / (TAP_BYTES / 16), q = i % (TAP_BYTES / 16);
      *reinterpret_cast<uint4*>(base + s * STAGE_BYTES + 9 * TAP_BYTES + q * 16) = make_uint4(0, 0, 0, 0);
    }
    // patch mode: rows 180..183 of every stage lie behind the copied patch and are read (times zero)
    for (int i = threadIdx.x; i < STAGES * (PATCH_ROWS_READ - IW * IH); i += kThreads) {
      const int s = i / (PATCH_ROWS_READ - IW * IH), q = i % (PATCH_ROWS_READ - IW * IH);
      *reinterpret_cast<uint4*>(base + s * STAGE_BYTES + PATCH_BYTES + q * 16) = make_uint4(0, 0, 0, 0);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  for (int i = threadIdx.x; i < BN; i += kThreads) bias_s[i] = a.bias ? a.bias[i] : 0.f;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < kGroups; ++b) { mbar_init(acc_full_bar(b), 1); mbar_init(acc_empty_bar(b), kGroupThreads); }
    mbar_init(w_bar, 1);
    mbar_init(drain_bar, 1);
    mbar_fence_init();
    tma_prefetch_desc(&map_x);
    tma_prefetch_desc(&map_w);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_slot), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  if (warp == 0) {
    if (lane == 0) {
      uint32_t fills[STAGES];
#pragma unroll
      for (int s = 0; s < STAGES; ++s) fills[s] = 0;
      mbar_expect_tx(w_bar, W_BYTES);
      for (int t = 0; t < 10; ++t) tma_load_2d(w_smem + t * W_TAP_BYTES, &map_w, w_bar, t * 8, 0);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < a.m_tiles; tile += gridDim.x) {
        if (!mbar_wait(empty_bar(stage), phase ^ 1, &abort_flag, a.dev_error, kDevTimeoutStageFree)) { ok = false; break; }
        const uint32_t sa = smem_base + stage * STAGE_BYTES;
        if (a.patch) {
          const int tw = tile % a.tiles_w, t = tile / a.tiles_w;
          mbar_expect_tx(full_bar(stage), PATCH_BYTES);
          tma_load_4d(sa, &map_x, full_bar(stage), 0, tw * PW - 1, (t % a.tiles_h) * PH - 1, t / a.tiles_h);
        } else {
          const int p0 = tile * BM;
          const int w0 = p0 % a.W, t = p0 / a.W;
          const int h0 = t % a.H, n0 = t / a.H;
          mbar_expect_tx(full_bar(stage), 9 * TAP_BYTES);
#pragma unroll
          for (int tap = 0; tap < 9; ++tap)
            tma_load_im2col_4d(sa + tap * TAP_BYTES, &map_x, full_bar(stage), 0, w0 - 1, h0 - 1, n0, (uint16_t)(tap % 3),
                               (uint16_t)(tap / 3));
        }
        ++fills[stage];
        if (++stage == STAGES) { stage = 0; phase ^= 1; }
      }
      if (!ok) {
        for (int s = 0; s < STAGES; ++s)
          if (fills[s]) {
            const unsigned long long t0 = global_timer_ns();
            while (!mbar_try_wait(full_bar(s), (fills[s] - 1) & 1) && global_timer_ns() - t0 < 100000000ull) {}
          }
      }
      // the filter load is always waited for by the MMA issuer or here
      {
        const unsigned long long t0 = global_timer_ns();
        while (!mbar_try_wait(w_bar, 0) && global_timer_ns() - t0 < 100000000ull) {}
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(BM, BN, 0, 0);
      int stage = 0;
      uint32_t phase = 0;
      int local = 0;
      bool ok = mbar_wait(w_bar, 0, &abort_flag, a.dev_error, kDevTimeoutTmaFull);
      for (int tile = blockIdx.x; tile < a.m_tiles && ok; tile += gridDim.x, ++local) {
        const int buf = local % kGroups;
        const uint32_t use = (uint32_t)(local / kGroups);
        if (!mbar_wait(acc_empty_bar(buf), (use & 1) ^ 1, &abort_flag, a.dev_error, kDevTimeoutTmemFree)) { ok = false; break; }
        if (!mbar_wait(full_bar(stage), phase, &abort_flag, a.dev_error, kDevTimeoutTmaFull)) { ok = false; break; }
        tc_fence_after();
        const uint32_t sa = smem_base + stage * STAGE_BYTES;
#pragma unroll
        for (int j = 0; j < 5; ++j) {
          // K step j = taps 2j and 2j+1: the two 8-element K chunks are one tap buffer apart,
          // 8-row groups are 128 bytes apart
          // (patch mode: tap 2j starts (r*10 + s) rows in; the next tap is one row on, or eight when the
          // pair straddles a filter row (j == 1: taps (0,2) and (1,0)); patch rows are 10 rows apart)
          const int t0 = 2 * j, r0 = t0 / 3, s0 = t0 - 3 * r0;
          const uint64_t da = a.patch ? smem_desc_plain(sa + (r0 * IW + s0) * 16, j == 1 ? (IW - 2) * 16 : 16, IW * 16)
                                      : smem_desc_plain(sa + 2 * j * TAP_BYTES, TAP_BYTES, 128);
          const uint64_t db = smem_desc_plain(w_smem + 2 * j * W_TAP_BYTES, W_TAP_BYTES, 128);
          umma_bf16(tmem_base + (uint32_t)(buf * BN), da, db, idesc, j != 0 ? 1u : 0u);
        }
        umma_commit(empty_bar(stage));
        umma_commit(acc_full_bar(buf));
        if (++stage == STAGES) { stage = 0; phase ^= 1; }
      }
      if (!ok) {
        umma_commit(drain_bar);
        const unsigned long long t0 = global_timer_ns();
        while (!mbar_try_wait(drain_bar, 0) && global_timer_ns() - t0 < 100000000ull) {}
      }
    }
  } else {
    const int group = (warp - 2) >> 3;            // which of the accumulator buffers / staging tiles
    const int quarter = warp & 3;                 // the TMEM lane quarter this warp may read
    const int row = quarter * 32 + lane;
    const int cc = (((warp - 2) >> 2) & 1) * 32;  // this warp's 32 of the 64 output channels
    const int bar_id = 1 + group;
    const bool issuer = threadIdx.x == 64 + group * kGroupThreads;  // owns the group's store groups
    const uint32_t stage_out = out_smem + (uint32_t)group * OUT_TILE_BYTES;
    uint32_t use = 0;  // tiles this group has taken
    for (int tile = blockIdx.x + group * gridDim.x; tile < a.m_tiles; tile += kGroups * gridDim.x, ++use) {
      const bool got = mbar_wait(acc_full_bar(group), use & 1, &abort_flag, a.dev_error, kDevTimeoutAccum);
      // the group's previous store must have read the staging tile before anyone refills it; the
      // barrier doubles as the vote that lets the group's warps leave together if any wait failed
      if (issuer) tma_store_wait_read<0>();
      if (named_bar_or(bar_id, kGroupThreads, !got)) break;
      tc_fence_after();
      uint32_t v[32];
      tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(group * BN + cc), v);
      tmem_ld_wait();
      // the accumulator is in registers: the MMA issuer may have the buffer back
      tc_fence_before();
      mbar_arrive(acc_empty_bar(group));
      uint32_t packed[16];
#pragma unroll
      for (int j = 0; j < 32; j += 2) {
        float x0 = __uint_as_float(v[j]), x1 = __uint_as_float(v[j + 1]);
        x0 += bias_s[cc + j]; x1 += bias_s[cc + j + 1];
        if (a.relu) { x0 = fmaxf(x0, 0.f); x1 = fmaxf(x1, 0.f); }
        __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
        packed[j >> 1] = *reinterpret_cast<uint32_t*>(&h);
      }
      if (a.patch) {
        // the tile leaves through shared memory and one TMA store (whole 128-byte lines) instead of
        // 256 threads writing 64-byte pieces of their own rows
        uint8_t* dst = smem_raw + (stage_out - smem_u32(smem_raw)) + row * 128;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int chunk = (cc >> 3) + q;  // 16-byte chunk of the 128-byte row, 128-byte swizzled
          *reinterpret_cast<uint4*>(dst + ((chunk ^ (row & 7)) << 4)) =
              make_uint4(packed[q * 4], packed[q * 4 + 1], packed[q * 4 + 2], packed[q * 4 + 3]);
        }
        fence_async_smem();
        named_bar_sync(bar_id, kGroupThreads);
        if (issuer) {
          const int tw = tile % a.tiles_w, t = tile / a.tiles_w;
          tma_store_4d(&map_y, stage_out, 0, tw * PW, (t % a.tiles_h) * PH, t / a.tiles_h);
          tma_store_commit();
        }
      } else {
        const long pixel = (long)tile * BM + row;
        if (pixel < a.pixels) {
          uint4* op = reinterpret_cast<uint4*>(a.out + pixel * BN + cc);
#pragma unroll
          for (int q = 0; q < 4; ++q)
            op[q] = make_uint4(packed[q * 4], packed[q * 4 + 1], packed[q * 4 + 2], packed[q * 4 + 3]);
        }
      }
    }
    if (issuer) tma_store_wait_all();  // shared memory must outlive the stores that read it
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// x8[p][0..2] = x[p][0..2], x8[p][3] = 1, x8[p][4..7] = 0
__global__ void pad_to8_kernel(const bf16* __restrict__ x, bf16* __restrict__ x8, long P) {
  long p = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= P) return;
  const unsigned short* s = reinterpret_cast<const unsigned short*>(x) + p * 3;
  const uint32_t a = s[0], b = s[1], c = s[2];
  reinterpret_cast<uint4*>(x8)[p] = make_uint4(a | (b << 16), c | (0x3F80u << 16), 0u, 0u);  // 0x3F80 = bf16 1.0
}

// w8[k][tap][c] = w[k][tap][c] for tap < 9 and c < 3, else 0
__global__ void first_filter_kernel(const float* __restrict__ w, bf16* __restrict__ w8, int Cout) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= Cout * 80) return;
  int c = i % 8, tap = (i / 8) % 10, k = i / 80;
  float v = (tap < 9 && c < 3) ? w[(k * 9 + tap) * 3 + c] : 0.f;
  w8[i] = __float2bfloat16_rn(v);
}

}  // namespace

bool tc_first_conv_supported(ConvShape s) {
  return s.Cin == 3 && s.Cout == 64 && s.H >= 2 && s.W >= 2 && (long)s.N * s.H * s.W < (1L << 31) - 256;
}

cudaError_t tc_pad_to8(const bf16* x, bf16* x8, long pixels, cudaStream_t st) {
  pad_to8_kernel<<<(unsigned)((pixels + 255) / 256), 256, 0, st>>>(x, x8, pixels);
  return cudaGetLastError();
}

cudaError_t tc_make_first_filter(const float* w, bf16* w8, cudaStream_t st) {
  first_filter_kernel<<<(64 * 80 + 255) / 256, 256, 0, st>>>(w, w8, 64);
  return cudaGetLastError();
}

cudaError_t tc_first_conv(const bf16* x8, const bf16* w8, const float* bias, bf16* out, ConvShape s, bool relu,
                          int* dev_error, cudaStream_t st) {
  if (!tc_first_conv_supported(s)) return cudaErrorInvalidValue;
  CUtensorMap mx, mw;
  const bool patch = s.W % PW == 0 && s.H % PH == 0;
  if (patch) {
    if (!make_patch_map_c8(&mx, x8, s.N, s.H, s.W, IW, IH)) return cudaErrorInvalidValue;
  } else if (!make_im2col_map_c8(&mx, x8, s.N, s.H, s.W, BM)) {
    return cudaErrorInvalidValue;
  }
  if (!make_tiled_map_2d_c8(&mw, w8, 64, 80, 64)) return cudaErrorInvalidValue;
  CUtensorMap my = mw;  // only read in patch mode
  if (patch && !make_patch_map(&my, out, s.N, s.H, s.W, 64, PW, PH)) return cudaErrorInvalidValue;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(conv3x3_c8_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  FirstArgs a;
  a.pixels = s.N * s.H * s.W; a.H = s.H; a.W = s.W;
  a.patch = patch ? 1 : 0;
  a.tiles_w = s.W / PW; a.tiles_h = s.H / PH;
  a.m_tiles = patch ? s.N * a.tiles_w * a.tiles_h : (a.pixels + BM - 1) / BM;
  a.relu = relu ? 1 : 0; a.bias = bias; a.out = out; a.dev_error = dev_error;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int grid = a.m_tiles < sms ? a.m_tiles : sms;
  conv3x3_c8_tc_kernel<<<grid, kThreads, SMEM_BYTES, st>>>(mx, mw, my, a);
  return cudaGetLastError();
}

}  // namespace vgg
