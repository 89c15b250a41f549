// Filter (and bias) gradient of a 3x3 convolution with few channels, from tiled patches.
//
//   dW[k][r][s][c] = sum over output pixels o of  dz[o][k] * x[o + (r-1, s-1)][c]
//
// The general filter-gradient GEMM (tc_gemm.cu) reads x through the copy engine's im2col mode, one
// 64-pixel box per tap and 64 channels; on the layers with 64 or 128 channels that mode's rate, not
// the tensor pipe, sets the pace, and with 64 output channels half of every 128-row MMA is padding.
// Here the sum runs over positions q = o + (0, s) instead of output pixels:
//
//   dW[k][r][s][c] = sum over q of  P_r[q][c] * Z_s[q][k],   P_r[q] = x[q + (r-1, -1)],  Z_s[q] = dz[q - (0, s)]
//
// so that for a K block of 8 x 8 positions both operands are shifted views of two small patches that
// plain tiled TMA boxes deliver: x rows h0-1 .. h0+8, columns w0-1 .. w0+6 (10 x 8 pixels), and dz rows
// h0 .. h0+7, columns w0-2 .. w0+7 (8 x 10 pixels), zero outside the image.  Both are MN-major operands
// (a row per position, 64 channels contiguous, 128-byte swizzled):
//   A = [P_0 | P_1]: two 64-channel groups one patch row (8 pixels, 1024 bytes) apart,
//   B = [Z_2 | Z_1 | Z_0]: three 64-channel groups one pixel (128 bytes) apart, patch rows 1280 bytes apart,
// one MMA 128 x 192 x 16 covers six taps for 16 positions; a second one has P_2 in its first 64 rows
// and a block of ones in the other 64, whose result rows are the column sums of Z: the bias gradient
// (group Z_0) for free.  Positions run over W + 2 columns per image row (the two extra columns pair
// the last output pixels with their right-hand taps).  One CTA per (64 input channels, 64 output
// channels) and share of the positions; fp32 partial sums, added in split order by a second kernel
// that also transposes them into dW's layout.  Warp roles and bounded waits as in tc_gemm.cu.
#include "tc_common.cuh"
#include "tc_kernels.cuh"

namespace vgg {
namespace {

using namespace tc;

constexpr int QW = 8, QH = 8;                 // positions of a K block
constexpr int X_BYTES = (QH + 2) * QW * 128;  // 10 x 8 pixel patch of x: 10240
constexpr int Z_BYTES = QH * (QW + 2) * 128;  // 8 x 10 pixel patch of dz: 10240
constexpr int STAGE = X_BYTES + Z_BYTES;
constexpr int ONES_BYTES = 2048;              // two 8-row groups of bf16 1.0
constexpr int kStages = 8;
constexpr int kThreads = 192;
constexpr int kSmem = kStages * STAGE + ONES_BYTES + 1024 + 256;
constexpr int D2_COL = 256;                   // tensor-memory column of the second accumulator
// floats one CTA writes: D1 [128][192], the first 64 rows of D2 [64][192], one row of column sums [192]
constexpr int kPartialFloats = 128 * 192 + 64 * 192 + 192;

struct PatchArgs {
  int H, W, tiles_w, tiles_h;
  int q_tiles;        // N * tiles_h * tiles_w
  int per_split;      // K blocks per CTA
  int k_blocks_out;   // Cout / 64
  float* partial;     // [split][tile][kPartialFloats]
  int* dev_error;
};

__global__ void __launch_bounds__(kThreads)
wgrad_patch_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_z, PatchArgs g) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t ones = smem_base + kStages * STAGE;
  const uint32_t bars = ones + ONES_BYTES;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (kStages + s); };
  const uint32_t acc_bar = bars + 8u * (2 * kStages);
  const uint32_t drain_bar = bars + 8u * (2 * kStages + 1);
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x;                     // (input-channel block, output-channel block)
  const int cb = tile / g.k_blocks_out, kb = tile - cb * g.k_blocks_out;
  const int q0 = blockIdx.y * g.per_split;
  const int q1 = min(g.q_tiles, q0 + g.per_split);

  if (threadIdx.x >= 64) {
    const uint32_t t = threadIdx.x - 64;  // 128 threads x 16 bytes
    asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(ones + 16u * t), "r"(0x3F803F80u) : "memory");
    fence_async_smem();
  }
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    mbar_init(acc_bar, 1);
    mbar_init(drain_bar, 1);
    mbar_fence_init();
    tma_prefetch_desc(&map_x);
    tma_prefetch_desc(&map_z);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_slot), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  if (warp == 0) {
    if (lane == 0) {
      uint32_t fills[kStages];
#pragma unroll
      for (int s = 0; s < kStages; ++s) fills[s] = 0;
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int tw = q0 % g.tiles_w, t = q0 / g.tiles_w;
      int th = t % g.tiles_h, img = t / g.tiles_h;
      for (int q = q0; q < q1; ++q) {
        if (!mbar_wait(empty_bar(stage), phase ^ 1, &abort_flag, g.dev_error, kDevTimeoutStageFree)) { ok = false; break; }
        const uint32_t sx = smem_base + stage * STAGE, sz = sx + X_BYTES;
        mbar_expect_tx(full_bar(stage), STAGE);
        tma_load_4d(sx, &map_x, full_bar(stage), cb * 64, tw * QW - 1, th * QH - 1, img);
        tma_load_4d(sz, &map_z, full_bar(stage), kb * 64, tw * QW - 2, th * QH, img);
        ++fills[stage];
        if (++stage == kStages) { stage = 0; phase ^= 1; }
        if (++tw == g.tiles_w) { tw = 0; if (++th == g.tiles_h) { th = 0; ++img; } }
      }
      if (!ok)
        for (int s = 0; s < kStages; ++s)
          if (fills[s]) {
            const unsigned long long t0 = global_timer_ns();
            while (!mbar_try_wait(full_bar(s), (fills[s] - 1) & 1) && global_timer_ns() - t0 < 100000000ull) {}
          }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(128, 192, 1, 1);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int q = q0; q < q1; ++q) {
        if (!mbar_wait(full_bar(stage), phase, &abort_flag, g.dev_error, kDevTimeoutTmaFull)) { ok = false; break; }
        tc_fence_after();
        const uint32_t sx = smem_base + stage * STAGE, sz = sx + X_BYTES;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          // 16 positions = position rows 2ks, 2ks+1 (8 each).  x patch rows are 8 pixels (1024 bytes),
          // dz patch rows 10 pixels (1280 bytes).
          const uint32_t a0 = sx + (uint32_t)(2 * ks) * 1024u;       // P_0; P_1 one patch row (1024 B) further
          const uint32_t a2 = sx + (uint32_t)(2 * ks + 2) * 1024u;   // P_2; the block of ones as its second group
          const uint32_t b0 = sz + (uint32_t)(2 * ks) * 1280u;       // Z_2; Z_1, Z_0 one pixel (128 B) further each
          const uint64_t db = smem_desc_sw128_full(b0, 128, 1280);
          umma_bf16(tmem_base, smem_desc_sw128_full(a0, 1024, 1024), db, idesc, (q > q0 || ks > 0) ? 1u : 0u);
          umma_bf16(tmem_base + D2_COL, smem_desc_sw128_full(a2, ones - a2, 1024), db, idesc, (q > q0 || ks > 0) ? 1u : 0u);
        }
        umma_commit(empty_bar(stage));
        if (++stage == kStages) { stage = 0; phase ^= 1; }
      }
      if (ok) {
        umma_commit(acc_bar);
      } else {
        umma_commit(drain_bar);
        const unsigned long long t0 = global_timer_ns();
        while (!mbar_try_wait(drain_bar, 0) && global_timer_ns() - t0 < 100000000ull) {}
      }
    }
  } else {
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    if (mbar_wait(acc_bar, 0, &abort_flag, g.dev_error, kDevTimeoutAccum)) {
      tc_fence_after();
      float* out = g.partial + ((size_t)blockIdx.y * gridDim.x + tile) * kPartialFloats;
      const bool empty = q0 >= q1;  // a split without positions contributes zeros
#pragma unroll 1
      for (int half = 0; half < 2; ++half) {
        // D1: all 128 rows.  D2: rows 0..63 (P_2) and row 64 (the column sums).
        const bool keep = half == 0 || row <= 64;
        float* dst = half == 0 ? out + row * 192 : out + 128 * 192 + row * 192;  // row 64 of D2 lands right after its 64 rows
#pragma unroll 1
        for (int cc = 0; cc < 192; cc += 32) {
          uint32_t v[32];
          tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(half * D2_COL + cc), v);
          tmem_ld_wait();
          if (!keep) continue;
#pragma unroll
          for (int j = 0; j < 32; j += 4)
            *reinterpret_cast<float4*>(dst + cc + j) =
                empty ? make_float4(0.f, 0.f, 0.f, 0.f)
                      : make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]), __uint_as_float(v[j + 2]),
                                    __uint_as_float(v[j + 3]));
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// dW[k][r][s][c] = sum over splits of the tile (c / 64, k / 64)'s partial sums; db[k] likewise from the
// tiles of input-channel block 0.  A block is 32 outputs (k fastest, so that a warp's reads are
// contiguous) x 8 groups of splits: with up to 148 splits and only 9 * Cin * Cout outputs one thread per
// output would add its splits as a chain of dependent loads.  Each group adds its range of splits in
// order, the groups are added in order through shared memory: a fixed order, whatever the launch.
constexpr int kFinishGroups = 8;
__global__ void wgrad_patch_finish_kernel(const float* __restrict__ partial, int splits, int tiles, int Cin, int Cout,
                                          float* __restrict__ dW, float* __restrict__ db) {
  __shared__ float part[kFinishGroups][33];
  const int g = threadIdx.y;
  const long i = (long)blockIdx.x * 32 + threadIdx.x;
  const long total = 9L * Cin * Cout;
  const int per = (splits + kFinishGroups - 1) / kFinishGroups;
  const int z0 = g * per, z1 = min(splits, z0 + per);
  if (db && g == 0 && i < Cout) {
    const int kb = (int)(i / 64), kl = (int)(i % 64);  // tile (cb = 0, kb), column sums row, group Z_0
    float s = 0.f;
    for (int z = 0; z < splits; ++z)
      s += partial[((size_t)z * tiles + kb) * kPartialFloats + 128 * 192 + 64 * 192 + 128 + kl];
    db[i] = s;
  }
  float sum = 0.f;
  long out = -1;
  if (i < total) {
    const int k = (int)(i % Cout);
    long t = i / Cout;
    const int c = (int)(t % Cin); t /= Cin;
    const int s9 = (int)(t % 3), r = (int)(t / 3);
    const int kb = k / 64, kl = k % 64, cb = c / 64, cl = c % 64;
    const int tile = cb * (Cout / 64) + kb;
    const int col = (2 - s9) * 64 + kl;
    const size_t off = r < 2 ? (size_t)(r * 64 + cl) * 192 + col : (size_t)128 * 192 + (size_t)cl * 192 + col;
    out = ((long)k * 9 + r * 3 + s9) * Cin + c;
    const float* src = partial + (size_t)tile * kPartialFloats + off;
    const size_t stride = (size_t)tiles * kPartialFloats;
    int z = z0;
    for (; z + 4 <= z1; z += 4) {  // independent loads, issued together; the additions stay in split order
      float v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) v[u] = src[(size_t)(z + u) * stride];
#pragma unroll
      for (int u = 0; u < 4; ++u) sum += v[u];
    }
    for (; z < z1; ++z) sum += src[(size_t)z * stride];
  }
  part[g][threadIdx.x] = sum;
  __syncthreads();
  if (g == 0 && out >= 0) {
    float tot = part[0][threadIdx.x];
#pragma unroll
    for (int q = 1; q < kFinishGroups; ++q) tot += part[q][threadIdx.x];
    dW[out] = tot;
  }
}

int patch_sm_count() {
  static int sms = 0;
  if (!sms) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (sms <= 0) sms = 148;
  }
  return sms;
}

void patch_plan(ConvShape s, int* tiles, int* q_tiles, int* splits, int* per) {
  *tiles = (s.Cin / 64) * (s.Cout / 64);
  const int tiles_w = (s.W + 2 + QW - 1) / QW, tiles_h = s.H / QH;
  *q_tiles = s.N * tiles_h * tiles_w;
  int want = patch_sm_count() / *tiles;  // one wave of CTAs
  if (want < 1) want = 1;
  if (want > *q_tiles) want = *q_tiles;
  *per = (*q_tiles + want - 1) / want;
  *splits = (*q_tiles + *per - 1) / *per;
}

}  // namespace

// Up to four 64 x 64 channel blocks (layers 2 to 4 of the network): measured at batch 100, layer 2 (one
// block) 0.60 -> 0.34 ms, layers 3 and 4 (two and four blocks) a few per cent, layer 5 (eight) slower than
// the im2col GEMM, whose wider tiles re-read less.
bool tc_wgrad_patch_supported(ConvShape s) {
  return s.Cin % 64 == 0 && s.Cout % 64 == 0 && (s.Cin / 64) * (s.Cout / 64) <= 4 && s.H % QH == 0 && s.W >= 16 && s.H >= 16 &&
         s.N >= 1 && (long)s.N * s.H * (s.W + 2 + QW) < (1L << 31);
}

size_t tc_wgrad_patch_scratch_elems(ConvShape s) {
  if (!tc_wgrad_patch_supported(s)) return 0;
  int tiles, qt, splits, per;
  patch_plan(s, &tiles, &qt, &splits, &per);
  return (size_t)splits * tiles * kPartialFloats;
}

cudaError_t tc_conv3x3_wgrad_patch(const bf16* x, const bf16* dz, float* dW, float* db, float* partial, ConvShape s,
                                   int* dev_error, cudaStream_t st) {
  if (!tc_wgrad_patch_supported(s)) return cudaErrorInvalidValue;
  CUtensorMap mx, mz;
  if (!make_patch_map(&mx, x, s.N, s.H, s.W, s.Cin, QW, QH + 2)) return cudaErrorInvalidValue;
  if (!make_patch_map(&mz, dz, s.N, s.H, s.W, s.Cout, QW + 2, QH)) return cudaErrorInvalidValue;
  PatchArgs g;
  int tiles, splits;
  patch_plan(s, &tiles, &g.q_tiles, &splits, &g.per_split);
  g.H = s.H; g.W = s.W;
  g.tiles_w = (s.W + 2 + QW - 1) / QW; g.tiles_h = s.H / QH;
  g.k_blocks_out = s.Cout / 64;
  g.partial = partial; g.dev_error = dev_error;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(wgrad_patch_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  wgrad_patch_tc_kernel<<<dim3(tiles, splits), kThreads, kSmem, st>>>(mx, mz, g);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const long total = 9L * s.Cin * s.Cout;
  wgrad_patch_finish_kernel<<<(unsigned)((total + 31) / 32), dim3(32, kFinishGroups), 0, st>>>(partial, splits, tiles, s.Cin, s.Cout, dW,
                                                                                                   db);
  return cudaGetLastError();
}

}  // namespace vgg
