// The first two convolutions (3 -> 64 -> 64 channels, each with bias and ReLU) as ONE kernel, for passes
// that keep neither layer's full-resolution output: conv1_1's activation, the largest tensor of the
// network, is never written to memory.
//
// The second convolution is the row-shift kernel of tc_conv_rowshift.cu (a tile is 8 x 14 output pixels, its
// accumulator 128 rows x 192 columns, three taps per MMA, the epilogue adds the three column-shifted partial
// sums).  What changes is where its 10 x 16 x 64 input patch comes from.  Instead of a TMA copy of conv1_1's
// stored output, the patch is computed in place:
//   * the 12 x 18 pixel patch of the (8-channel copy of the) image behind it arrives by TMA, 3.4 KB;
//   * ten small MMAs (128 x 64 x 16, two filter taps of 8 channels each per MMA, operands without swizzle
//     as in tc_conv_first.cu) compute conv1_1 on the patch's left and right halves (8 columns x 10 rows
//     each, so that an 8-row group of the A operand is 8 consecutive pixels of one image row and groups are
//     one image row apart) into the 2 x 64 tensor-memory columns the two main accumulators leave free;
//   * six "builder" warps read those accumulators, add the bias, apply the ReLU, put zeros where the patch
//     position lies outside the image (the second convolution's padding), round to bf16 and write the rows
//     into the patch slot in the 128-byte-swizzled layout the main MMAs read.
// The single MMA-issuing thread alternates: first-layer MMAs of tile t + 1, main MMAs of tile t.
//
// Warps: 0 image-patch producer, 1 MMA issuer and tensor-memory owner, 2 filter loader, 4-19 epilogue (two
// groups of eight taking alternate tiles, as in the row-shift kernel), 20-22 and 24-26 builders (one patch half each).  All waits are
// time-limited (tc_common.cuh).
#include "tc_common.cuh"
#include "tc_kernels.cuh"

namespace vgg {
namespace {

using namespace tc;

constexpr int BM = 128, BK = 64, BN3 = 192;
constexpr int TH = 8, TW = 14;                    // output pixels of a tile
constexpr int AW = 16, IH = TH + 2;               // patch of conv1_1's output: 10 rows x 16 columns
constexpr int A_BYTES = IH * AW * 128;            // 20480
constexpr int B_BYTES = 3 * 64 * BK * 2;          // one filter row of the second layer: three taps x 64 x 64
constexpr int FILTER_BYTES = 3 * B_BYTES;
constexpr int OUT_BYTES = TH * TW * 128;          // staging tile of the TMA store
constexpr int IMG_W = AW + 2, IMG_H = IH + 2;     // image pixels behind a patch: 18 columns x 12 rows
constexpr int IMG_BYTES = IMG_H * IMG_W * 16;     // what the copy engine writes (16-byte pixels)
constexpr int IMG_SLOT = 5248;                    // the MMAs' 16 row groups reach image row 17 (never copied: kept zero)
constexpr int W8_TAP_BYTES = 64 * 16;             // first-layer filter, one tap: 64 output x 8 input channels
constexpr int W8_BYTES = 10 * W8_TAP_BYTES;
constexpr int NA = 4, NI = 3;                     // patch slots, image slots
constexpr int kThreads = 864, kGroupThreads = 256, kBuilderThreads = 192;  // builders: warps 20-22 and 24-26
constexpr int ACC_STRIDE = 256;                   // main accumulators at columns 0 and 256
constexpr int C1_LEFT = 192, C1_RIGHT = 448;      // first-layer accumulators in the columns they leave free
constexpr int SMEM_BYTES = NA * A_BYTES + FILTER_BYTES + 2 * OUT_BYTES + W8_BYTES + NI * IMG_SLOT + 512 + 1024;

struct F12Args {
  int N, H, W;
  int tiles_w, tiles_h, tiles;
  const float* bias1;
  const float* bias2;
  bf16* out;     // the second layer's full-resolution output, or null
  bf16* pooled;  // its 2x2 max-pool, or null
  int* dev_error;
};

__global__ void __launch_bounds__(kThreads, 1)
conv12_fused_tc_kernel(const __grid_constant__ CUtensorMap map_img, const __grid_constant__ CUtensorMap map_w,
                       const __grid_constant__ CUtensorMap map_w8, const __grid_constant__ CUtensorMap map_y, F12Args a) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t b_base = smem_base + NA * A_BYTES;
  const uint32_t out_smem = b_base + FILTER_BYTES;
  const uint32_t w8_smem = out_smem + 2 * OUT_BYTES;
  const uint32_t img_smem = w8_smem + W8_BYTES;
  const uint32_t bars = img_smem + NI * IMG_SLOT;
  auto a_full = [&](int s) { return bars + 8u * s; };
  auto a_empty = [&](int s) { return bars + 8u * (NA + s); };
  auto img_full = [&](int s) { return bars + 8u * (2 * NA + s); };
  auto img_empty = [&](int s) { return bars + 8u * (2 * NA + NI + s); };
  auto acc_full = [&](int b) { return bars + 8u * (2 * NA + 2 * NI + b); };
  auto acc_empty = [&](int b) { return bars + 8u * (2 * NA + 2 * NI + 2 + b); };
  const uint32_t c1_full = bars + 8u * (2 * NA + 2 * NI + 4);
  const uint32_t c1_empty = bars + 8u * (2 * NA + 2 * NI + 5);
  const uint32_t w_bar = bars + 8u * (2 * NA + 2 * NI + 6);
  const uint32_t drain_bar = bars + 8u * (2 * NA + 2 * NI + 7);
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  __shared__ __align__(16) float bias1_s[64];
  __shared__ __align__(16) float bias2_s[64];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // image rows 12..17 of every slot lie behind the copied patch; the MMAs read them into accumulator rows
  // nobody uses, and the padding tap of row 11 reads the first of them times zero: keep them finite
  {
    uint8_t* base = smem_raw + (img_smem - smem_u32(smem_raw));
    constexpr int kTail16 = (IMG_SLOT - IMG_BYTES) / 16;
    for (int i = threadIdx.x; i < NI * kTail16; i += kThreads)
      *reinterpret_cast<uint4*>(base + (i / kTail16) * IMG_SLOT + IMG_BYTES + (i % kTail16) * 16) = make_uint4(0, 0, 0, 0);
    fence_async_smem();
  }
  if (threadIdx.x < 64) {
    bias1_s[threadIdx.x] = a.bias1 ? a.bias1[threadIdx.x] : 0.f;
    bias2_s[threadIdx.x] = a.bias2 ? a.bias2[threadIdx.x] : 0.f;
  }
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < NA; ++s) { mbar_init(a_full(s), 1); mbar_init(a_empty(s), 1); }
    for (int s = 0; s < NI; ++s) { mbar_init(img_full(s), 1); mbar_init(img_empty(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), kGroupThreads); }
    mbar_init(c1_full, 1);
    mbar_init(c1_empty, kBuilderThreads);
    mbar_init(w_bar, 1);
    mbar_init(drain_bar, 1);
    mbar_fence_init();
    tma_prefetch_desc(&map_img);
    tma_prefetch_desc(&map_w);
    tma_prefetch_desc(&map_w8);
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
    // ---------------- image-patch producer ----------------
    if (lane == 0) {
      uint32_t fills[NI];
#pragma unroll
      for (int s = 0; s < NI; ++s) fills[s] = 0;
      int slot = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < a.tiles && ok; tile += gridDim.x) {
        const int tw = tile % a.tiles_w, t = tile / a.tiles_w;
        const int w0 = tw * TW, h0 = (t % a.tiles_h) * TH, img = t / a.tiles_h;
        if (!mbar_wait(img_empty(slot), phase ^ 1, &abort_flag, a.dev_error, kDevTimeoutStageFree)) { ok = false; break; }
        mbar_expect_tx(img_full(slot), IMG_BYTES);
        // conv1_1's output patch starts one pixel up/left of the tile, its own input one more; outside the image: zeros
        tma_load_4d(img_smem + slot * IMG_SLOT, &map_img, img_full(slot), 0, w0 - 2, h0 - 2, img);
        ++fills[slot];
        if (++slot == NI) { slot = 0; phase ^= 1; }
      }
      if (!ok)
        for (int s = 0; s < NI; ++s)
          if (fills[s]) {
            const unsigned long long t0 = global_timer_ns();
            while (!mbar_try_wait(img_full(s), (fills[s] - 1) & 1) && global_timer_ns() - t0 < 100000000ull) {}
          }
    }
  } else if (warp == 2) {
    // ---------------- filters: both layers', loaded once ----------------
    if (lane == 0) {
      mbar_expect_tx(w_bar, (uint32_t)(FILTER_BYTES + W8_BYTES));
      for (int r = 0; r < 3; ++r) tma_load_3d(b_base + r * B_BYTES, &map_w, w_bar, 0, 0, 3 * r);
      for (int t = 0; t < 10; ++t) tma_load_2d(w8_smem + t * W8_TAP_BYTES, &map_w8, w_bar, t * 8, 0);
      const unsigned long long t0 = global_timer_ns();  // never leave with the copy in flight
      while (!mbar_try_wait(w_bar, 0) && global_timer_ns() - t0 < 100000000ull) {}
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(BM, BN3, 0, 0);
      constexpr uint32_t idesc1 = umma_idesc_bf16(BM, 64, 0, 0);
      int aslot = 0, islot = 0;
      uint32_t aphase = 0, iphase = 0;
      bool ok = mbar_wait(w_bar, 0, &abort_flag, a.dev_error, kDevTimeoutTmaFull);
      // first layer on the image patch of this CTA's p-th tile: left and right half of the 10 x 16 patch
      auto first_layer = [&](int p) {
        if (!mbar_wait(img_full(islot), iphase, &abort_flag, a.dev_error, kDevTimeoutTmaFull)) return false;
        if (!mbar_wait(c1_empty, (uint32_t)((p & 1) ^ 1), &abort_flag, a.dev_error, kDevTimeoutTmemFree)) return false;
        tc_fence_after();
        const uint32_t si = img_smem + islot * IMG_SLOT;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const uint32_t d = tmem_base + (uint32_t)(half ? C1_RIGHT : C1_LEFT);
#pragma unroll
          for (int j = 0; j < 5; ++j) {
            // K step j = taps 2j and 2j + 1, 8 channels (16 bytes) each.  Tap (r, s) of patch pixel (i, c) reads
            // image pixel (i + r, c + s): an 8-row group of A is 8 consecutive pixels of a row (128 bytes),
            // groups are one image row (18 pixels) apart; the second tap of a step is one pixel on, or, for
            // the step that straddles a filter row (taps (0,2) and (1,0)), 16 pixels on
            const int t0 = 2 * j, r0 = t0 / 3, s0 = t0 - 3 * r0;
            const uint64_t da = smem_desc_plain(si + (uint32_t)((r0 * IMG_W + s0 + 8 * half) * 16), j == 1 ? (IMG_W - 2) * 16 : 16,
                                                IMG_W * 16);
            const uint64_t db = smem_desc_plain(w8_smem + 2 * j * W8_TAP_BYTES, W8_TAP_BYTES, 128);
            umma_bf16(d, da, db, idesc1, j != 0 ? 1u : 0u);
          }
        }
        umma_commit(img_empty(islot));
        umma_commit(c1_full);
        if (++islot == NI) { islot = 0; iphase ^= 1; }
        return true;
      };
      int local = 0;
      if (ok && (int)blockIdx.x < a.tiles) ok = first_layer(0);
      for (int tile = blockIdx.x; tile < a.tiles && ok; tile += gridDim.x, ++local) {
        if (tile + (int)gridDim.x < a.tiles && !first_layer(local + 1)) { ok = false; break; }
        const int buf = local & 1;
        const uint32_t use = (uint32_t)(local >> 1);
        if (!mbar_wait(acc_empty(buf), (use & 1) ^ 1, &abort_flag, a.dev_error, kDevTimeoutTmemFree)) { ok = false; break; }
        if (!mbar_wait(a_full(aslot), aphase, &abort_flag, a.dev_error, kDevTimeoutTmaFull)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * ACC_STRIDE);
        const uint32_t sa = smem_base + aslot * A_BYTES;
#pragma unroll
        for (int r = 0; r < 3; ++r) {
          // filter row r: accumulator row (ph, j) reads patch row (ph + r) * 16 + j
          const uint64_t da = smem_desc_sw128(sa + (uint32_t)r * (AW * 128u), 16);
          const uint64_t db = smem_desc_sw128(b_base + r * B_BYTES, 16);
          umma_bf16(d_tmem, da, db, idesc, r != 0 ? 1u : 0u);
#pragma unroll
          for (int k = 1; k < BK / 16; ++k)
            umma_bf16_acc(d_tmem, desc_advance(da, k * 32), desc_advance(db, k * 32), idesc);
        }
        umma_commit(a_empty(aslot));
        umma_commit(acc_full(buf));
        if (++aslot == NA) { aslot = 0; aphase ^= 1; }
      }
      if (!ok) {
        umma_commit(drain_bar);
        const unsigned long long t0 = global_timer_ns();
        while (!mbar_try_wait(drain_bar, 0) && global_timer_ns() - t0 < 100000000ull) {}
      }
    }
  } else if (warp >= 20 && (warp & 3) != 3) {
    // ---------------- builders: first-layer accumulators -> the second layer's input patch ----------------
    // warps 20-22 take the left half of the patch, warps 24-26 the right half
    const int half = (warp - 20) >> 2;
    const int quarter = warp & 3;                 // 0, 1, 2: the tensor-memory lanes this warp may read
    const int row = quarter * 32 + lane;          // accumulator row = (patch row i, column cc of the half): 80 are real
    const int i = row >> 3, cc = row & 7;
    const bool real = row < IH * 8;
    const bool elected = threadIdx.x == 20 * 32;
    int slot = 0;
    uint32_t phase = 0;
    int p = 0;
    for (int tile = blockIdx.x; tile < a.tiles; tile += gridDim.x, ++p) {
      bool got = mbar_wait(a_empty(slot), phase ^ 1, &abort_flag, a.dev_error, kDevTimeoutStageFree);
      got = got && mbar_wait(c1_full, (uint32_t)(p & 1), &abort_flag, a.dev_error, kDevTimeoutAccum);
      if (named_bar_or(3, kBuilderThreads, !got)) break;  // the three warps leave together
      tc_fence_after();
      const int tw = tile % a.tiles_w, t = tile / a.tiles_w;
      const int w0 = tw * TW, h0 = (t % a.tiles_h) * TH;
      const int gh = h0 - 1 + i;
      uint8_t* slot_ptr = smem_raw + (smem_base + slot * A_BYTES - smem_u32(smem_raw));
      {
        const int col = cc + 8 * half;            // patch column
        const int gw = w0 - 1 + col;
        const bool inside = gh >= 0 && gh < a.H && gw >= 0 && gw < a.W;  // else: the second convolution's zero padding
        const int pr = i * AW + col;              // patch row (one pixel, 128 bytes)
        uint8_t* dst = slot_ptr + pr * 128;
        // both loads in flight before the one wait
        uint32_t va[32], vb[32];
        const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(half ? C1_RIGHT : C1_LEFT);
        tmem_ld_32x32(t_addr, va);
        tmem_ld_32x32(t_addr + 32u, vb);
        tmem_ld_wait();
        // the thread's last read of the accumulators: the issuer may start the next tile's first layer
        tc_fence_before();
        mbar_arrive(c1_empty);
        if (real) {
#pragma unroll
          for (int c32 = 0; c32 < 64; c32 += 32) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              uint32_t h[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const int ch = c32 + 8 * q + 2 * e;
                const uint32_t r0 = c32 ? vb[8 * q + 2 * e] : va[8 * q + 2 * e], r1 = c32 ? vb[8 * q + 2 * e + 1] : va[8 * q + 2 * e + 1];
                const float x0 = inside ? fmaxf(__uint_as_float(r0) + bias1_s[ch], 0.f) : 0.f;
                const float x1 = inside ? fmaxf(__uint_as_float(r1) + bias1_s[ch + 1], 0.f) : 0.f;
                __nv_bfloat162 hh = __floats2bfloat162_rn(x0, x1);
                h[e] = *reinterpret_cast<uint32_t*>(&hh);
              }
              const int chunk = (c32 >> 3) + q;   // 16-byte chunk of the 128-byte row, 128-byte swizzled
              *reinterpret_cast<uint4*>(dst + ((chunk ^ (pr & 7)) << 4)) = make_uint4(h[0], h[1], h[2], h[3]);
            }
          }
        }
      }
      fence_async_smem();  // the patch was written by ordinary stores, the MMAs read it through the async proxy
      named_bar_sync(3, kBuilderThreads);
      if (elected) mbar_arrive(a_full(slot));
      if (++slot == NA) { slot = 0; phase ^= 1; }
    }
  } else if (warp >= 4 && warp < 20) {
    // ---------------- epilogue of the second layer (as in the row-shift kernel) ----------------
    const int group = (warp - 4) >> 3;
    const int quarter = warp & 3;
    const int c_first = (((warp - 4) >> 2) & 1) * 32;
    const int ph = quarter * 2 + (lane >> 4);
    const int j = lane & 15;
    const bool col_ok = j < TW;
    const int rr = ph * TW + j;
    const bool issuer = threadIdx.x == 128 + group * kGroupThreads;
    const int bar_id = 1 + group;
    uint8_t* stage_row = smem_raw + (out_smem - smem_u32(smem_raw)) + group * OUT_BYTES + rr * 128;
    const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(group * ACC_STRIDE);
    const bool pool_lane = lane < 16 && (j & 1) == 0 && col_ok;
    uint32_t use = 0;
    for (int tile = blockIdx.x + group * gridDim.x; tile < a.tiles; tile += 2 * gridDim.x, ++use) {
      const bool got = mbar_wait(acc_full(group), use & 1, &abort_flag, a.dev_error, kDevTimeoutAccum);
      if (named_bar_or(bar_id, kGroupThreads, !got)) break;
      tc_fence_after();
      const int tw = tile % a.tiles_w, t = tile / a.tiles_w;
      const int w0 = tw * TW, h0 = (t % a.tiles_h) * TH, img = t / a.tiles_h;
      if (a.out) {
        if (issuer) tma_store_wait_read<0>();  // the group's previous store has read the staging tile
        named_bar_sync(bar_id, kGroupThreads);
      }
      bf16* pool_row = a.pooled ? a.pooled + (((long)img * (a.H / 2) + (h0 + ph) / 2) * (a.W / 2) + (w0 + j) / 2) * 64
                                : nullptr;
#pragma unroll
      for (int c16 = c_first; c16 < c_first + 32; c16 += 16) {
        uint32_t v0[16], v1[16], v2[16];
        tmem_ld_32x16(t_row + (uint32_t)c16, v0);
        tmem_ld_32x16(t_row + (uint32_t)(64 + c16), v1);
        tmem_ld_32x16(t_row + (uint32_t)(128 + c16), v2);
        tmem_ld_wait();
        uint32_t packed[8];
#pragma unroll
        for (int i = 0; i < 16; i += 2) {
          // out(ph, j) = D(ph, j)[s = 0] + D(ph, j + 1)[s = 1] + D(ph, j + 2)[s = 2]
          float x0 = __uint_as_float(v0[i]) + __shfl_down_sync(0xffffffffu, __uint_as_float(v1[i]), 1) +
                     __shfl_down_sync(0xffffffffu, __uint_as_float(v2[i]), 2);
          float x1 = __uint_as_float(v0[i + 1]) + __shfl_down_sync(0xffffffffu, __uint_as_float(v1[i + 1]), 1) +
                     __shfl_down_sync(0xffffffffu, __uint_as_float(v2[i + 1]), 2);
          x0 = fmaxf(x0 + bias2_s[c16 + i], 0.f);
          x1 = fmaxf(x1 + bias2_s[c16 + i + 1], 0.f);
          __nv_bfloat162 hh = __floats2bfloat162_rn(x0, x1);
          packed[i >> 1] = *reinterpret_cast<uint32_t*>(&hh);
        }
        const int chunk0 = c16 >> 3;
        if (a.out && col_ok) {
#pragma unroll
          for (int q = 0; q < 2; ++q)
            *reinterpret_cast<uint4*>(stage_row + (((chunk0 + q) ^ (rr & 7)) << 4)) =
                make_uint4(packed[q * 4], packed[q * 4 + 1], packed[q * 4 + 2], packed[q * 4 + 3]);
        }
        if (a.pooled) {
          pool2x2<8>(packed, 1, 16);  // columns j, j + 1 (next lane) of rows ph, ph + 1 (16 lanes on)
          if (pool_lane) {
            uint4* pp = reinterpret_cast<uint4*>(pool_row + c16);
            pp[0] = make_uint4(packed[0], packed[1], packed[2], packed[3]);
            pp[1] = make_uint4(packed[4], packed[5], packed[6], packed[7]);
          }
        }
      }
      tc_fence_before();
      mbar_arrive(acc_empty(group));
      if (a.out) {
        fence_async_smem();
        named_bar_sync(bar_id, kGroupThreads);
        if (issuer) {
          tma_store_4d(&map_y, out_smem + group * OUT_BYTES, 0, w0, h0, img);
          tma_store_commit();
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
    tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace

bool tc_conv12_fused_supported(ConvShape s) {
  return s.Cin == 3 && s.Cout == 64 && s.W % TW == 0 && s.H % TH == 0 && s.W >= 56 && s.H % 2 == 0 &&
         (long)s.N * s.H * s.W < (1L << 31) - 256;
}

cudaError_t tc_conv12_fused(const bf16* x8, const bf16* w8, const float* bias1, const bf16* wt2_tap_major, const float* bias2,
                            bf16* out, bf16* pooled, ConvShape s, int* dev_error, cudaStream_t st) {
  if (!tc_conv12_fused_supported(s) || (!out && !pooled)) return cudaErrorInvalidValue;
  CUtensorMap mi, mw, m8;
  if (!make_patch_map_c8(&mi, x8, s.N, s.H, s.W, IMG_W, IMG_H)) return cudaErrorInvalidValue;
  if (!make_filter_row_map(&mw, wt2_tap_major, 64, 64, 64)) return cudaErrorInvalidValue;
  if (!make_tiled_map_2d_c8(&m8, w8, 64, 80, 64)) return cudaErrorInvalidValue;
  CUtensorMap my = mw;  // only read when there is a full-resolution output
  if (out && !make_patch_map(&my, out, s.N, s.H, s.W, 64, TW, TH)) return cudaErrorInvalidValue;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(conv12_fused_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  F12Args a;
  a.N = s.N; a.H = s.H; a.W = s.W;
  a.tiles_w = s.W / TW; a.tiles_h = s.H / TH;
  a.tiles = s.N * a.tiles_w * a.tiles_h;
  a.bias1 = bias1; a.bias2 = bias2; a.out = out; a.pooled = pooled; a.dev_error = dev_error;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  conv12_fused_tc_kernel<<<a.tiles < sms ? a.tiles : sms, kThreads, SMEM_BYTES, st>>>(mi, mw, m8, my, a);
  return cudaGetLastError();
}

}  // namespace vgg
