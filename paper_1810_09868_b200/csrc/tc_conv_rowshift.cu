// 3x3 convolution with 64 output channels on tcgen05: the three taps of a filter row share one MMA.
//
// With 64 output channels an MMA of one tap is 128 x 64 x 16: its A operand (4 KB) takes longer to
// read from shared memory than the tensor pipe needs for the arithmetic, and nine taps mean 36 such
// MMAs per 64 input channels.  Here the accumulator row of a pixel does not hold that pixel's output
// but three partial sums, one per filter column s, each belonging to the output pixel s places to
// its left:
//
//   D[(ph, j)][s * 64 + k] = sum over r, c of  X[h0 - 1 + ph + r][w0 - 1 + j][c] * Wt[k][r][s][c]
//   out[h0 + ph][w0 + j][k] = D[(ph, j)][k] + D[(ph, j + 1)][64 + k] + D[(ph, j + 2)][128 + k]
//
// so that for a filter row r all 128 accumulator rows read the SAME input pixels for every s: the A
// operand is 128 consecutive rows of the input patch (start r * 16 rows), the B operand the 192 rows
// [s][k] of that filter row, and one MMA is 128 x 192 x 16.  Twelve MMAs per 64 input channels
// instead of 36, each bound by the tensor pipe (96 cycles) rather than by operand reads.  The price:
// a tile is 8 rows x 16 columns of accumulator for 8 x 14 output pixels (the last two columns only
// feed their left neighbours), and the epilogue adds the three partial sums with two warp shuffles
// per value (lane = (ph & 1) * 16 + j: the neighbours are the next lanes).
//
// Input patch per tile and 64 channels: 10 rows x 16 columns (halo included; zero outside the image
// by TMA), 20 KB, 128-byte swizzled.  Filter from the tap-major copy [9][64][Cin]: resident in shared
// memory when Cin = 64, else a ring of filter rows.  Output: swizzled staging tile of 8 x 14 pixels and
// one TMA store; optional 2x2 max-pool stored directly; optional ReLU-mask tile (input gradient) by TMA.
// Warps: 0 patch producer, 1 MMA issuer + TMEM owner, 2 filter producer, 4-19 epilogue: two groups of
// eight warps that take alternate tiles (two warps per tensor-memory lane quarter, each 32 of the 64
// output channels).  A tile's MMAs last well under a microsecond; four epilogue warps (one per
// scheduler, nothing to hide their shuffle and tensor-memory latencies behind) needed two.
#include "tc_common.cuh"
#include "tc_kernels.cuh"

namespace vgg {
namespace {

using namespace tc;

constexpr int BM = 128, BK = 64, BN3 = 192;       // accumulator tile: 128 rows x (3 x 64) columns
constexpr int TH = 8, TW = 14;                    // output pixels of a tile
constexpr int AW = 16;                            // accumulator (and patch) columns
constexpr int IH = TH + 2;                        // patch rows
constexpr int A_BYTES = IH * AW * 128;            // 20480: a multiple of 1024
constexpr int B_BYTES = 3 * 64 * BK * 2;          // one filter row: three taps x 64 channels out x 64 in
constexpr int OUT_BYTES = TH * TW * 128;          // 14336: staging tile of the TMA store (and the mask tile)
constexpr int kThreads = 640;
constexpr int kGroupThreads = 256;  // one of the two epilogue groups
constexpr int kMaxPatchSlots = 6, kMaxFilterSlots = 4;
constexpr int kLimit = 227 * 1024 - 2560;
constexpr int ACC_STRIDE = 256;                   // tensor-memory columns between the two accumulators

struct RowArgs {
  int N, H, W;
  int cin_blocks;
  int tiles_w, tiles_h, tiles;
  int relu;
  const float* bias;
  int na, nb, resident, b_region_bytes;
  const bf16* mask;
  bf16* out;     // full-resolution output or null
  bf16* pooled;  // 2x2 max-pooled output or null
  uint8_t* code; // with pooled: arg-max code of every window (see simt_maxpool_fwd), or null
  // Pool scatter (input gradient of a layer whose input is a pooled tensor): instead of storing the tile,
  // store it four times, once per window position, into the full-resolution gradient of the layer below
  // the pool, keeping a value only at the position its window's stored code names.
  const uint8_t* scatter_code;  // [N][H][W][64] at this kernel's resolution, or null
  int* dev_error;
};

// MODE 0: plain (output, mask, pooled output); 1: pooled output with arg-max codes; 2: pool scatter.
// Compile-time so that the plain kernel carries none of the other two's registers and instructions.
template <int MODE>
__global__ void __launch_bounds__(kThreads, 1)
conv3x3_rowshift_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                           const __grid_constant__ CUtensorMap map_y, const __grid_constant__ CUtensorMap map_m,
                           const __grid_constant__ CUtensorMap map_s0, const __grid_constant__ CUtensorMap map_s1,
                           const __grid_constant__ CUtensorMap map_s2, const __grid_constant__ CUtensorMap map_s3,
                           RowArgs a) {
  constexpr int NA = kMaxPatchSlots, NB = kMaxFilterSlots;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t b_base = smem_base + a.na * A_BYTES;
  const uint32_t out_smem = b_base + a.b_region_bytes;  // 1024-byte aligned
  const uint32_t mask_smem = out_smem + 2 * OUT_BYTES;
  const uint32_t bars = mask_smem + (a.mask ? 2 * OUT_BYTES : 0);
  auto a_full = [&](int s) { return bars + 8u * s; };
  auto a_empty = [&](int s) { return bars + 8u * (NA + s); };
  auto b_full = [&](int s) { return bars + 8u * (2 * NA + s); };
  auto b_empty = [&](int s) { return bars + 8u * (2 * NA + NB + s); };
  auto acc_full = [&](int b) { return bars + 8u * (2 * NA + 2 * NB + b); };
  auto acc_empty = [&](int b) { return bars + 8u * (2 * NA + 2 * NB + 2 + b); };
  const uint32_t drain_bar = bars + 8u * (2 * NA + 2 * NB + 4);
  auto mask_bar = [&](int g) { return bars + 8u * (2 * NA + 2 * NB + 5 + g); };
  const uint32_t w_bar = bars + 8u * (2 * NA + 2 * NB + 7);  // resident filter loaded
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  __shared__ __align__(16) float bias_s[64];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x < 64) bias_s[threadIdx.x] = a.bias ? a.bias[threadIdx.x] : 0.f;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < NA; ++s) { mbar_init(a_full(s), 1); mbar_init(a_empty(s), 1); }
    for (int s = 0; s < NB; ++s) { mbar_init(b_full(s), 1); mbar_init(b_empty(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), kGroupThreads); }
    mbar_init(drain_bar, 1);
    mbar_init(mask_bar(0), 1);
    mbar_init(mask_bar(1), 1);
    mbar_init(w_bar, 1);
    mbar_fence_init();
    tma_prefetch_desc(&map_x);
    tma_prefetch_desc(&map_w);
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
    // ---------------- input-patch producer ----------------
    if (lane == 0) {
      uint32_t fills[NA];
#pragma unroll
      for (int s = 0; s < NA; ++s) fills[s] = 0;
      int slot = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < a.tiles && ok; tile += gridDim.x) {
        const int tw = tile % a.tiles_w, t = tile / a.tiles_w;
        const int w0 = tw * TW, h0 = (t % a.tiles_h) * TH, img = t / a.tiles_h;
        for (int cb = 0; cb < a.cin_blocks; ++cb) {
          if (!mbar_wait(a_empty(slot), phase ^ 1, &abort_flag, a.dev_error, kDevTimeoutStageFree)) { ok = false; break; }
          mbar_expect_tx(a_full(slot), A_BYTES);
          tma_load_4d(smem_base + slot * A_BYTES, &map_x, a_full(slot), cb * BK, w0 - 1, h0 - 1, img);
          ++fills[slot];
          if (++slot == a.na) { slot = 0; phase ^= 1; }
        }
      }
      if (!ok)
        for (int s = 0; s < NA; ++s)
          if (fills[s]) {
            const unsigned long long t0 = global_timer_ns();
            while (!mbar_try_wait(a_full(s), (fills[s] - 1) & 1) && global_timer_ns() - t0 < 100000000ull) {}
          }
    }
  } else if (warp == 2) {
    // ---------------- filter producer ----------------
    if (lane == 0) {
      uint32_t fills[NB];
#pragma unroll
      for (int s = 0; s < NB; ++s) fills[s] = 0;
      int slot = 0;
      uint32_t phase = 0;
      bool ok = true;
      if (a.resident) {
        mbar_expect_tx(w_bar, (uint32_t)(a.cin_blocks * 3 * B_BYTES));
        for (int cb = 0; cb < a.cin_blocks; ++cb)
          for (int r = 0; r < 3; ++r)
            tma_load_3d(b_base + (cb * 3 + r) * B_BYTES, &map_w, w_bar, cb * BK, 0, 3 * r);
        const unsigned long long t0 = global_timer_ns();  // never leave with the copy in flight
        while (!mbar_try_wait(w_bar, 0) && global_timer_ns() - t0 < 100000000ull) {}
      }
      for (int tile = blockIdx.x; tile < a.tiles && ok && !a.resident; tile += gridDim.x) {
        for (int cb = 0; cb < a.cin_blocks && ok; ++cb)
          for (int r = 0; r < 3; ++r) {
            if (!mbar_wait(b_empty(slot), phase ^ 1, &abort_flag, a.dev_error, kDevTimeoutStageFree)) { ok = false; break; }
            mbar_expect_tx(b_full(slot), B_BYTES);
            tma_load_3d(b_base + slot * B_BYTES, &map_w, b_full(slot), cb * BK, 0, 3 * r);
            ++fills[slot];
            if (++slot == a.nb) { slot = 0; phase ^= 1; }
          }
      }
      if (!ok)
        for (int s = 0; s < NB; ++s)
          if (fills[s]) {
            const unsigned long long t0 = global_timer_ns();
            while (!mbar_try_wait(b_full(s), (fills[s] - 1) & 1) && global_timer_ns() - t0 < 100000000ull) {}
          }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(BM, BN3, 0, 0);
      int aslot = 0, bslot = 0;
      uint32_t aphase = 0, bphase = 0;
      int local = 0;
      bool ok = true;
      if (a.resident) ok = mbar_wait(w_bar, 0, &abort_flag, a.dev_error, kDevTimeoutTmaFull);
      for (int tile = blockIdx.x; tile < a.tiles && ok; tile += gridDim.x, ++local) {
        const int buf = local & 1;
        const uint32_t use = (uint32_t)(local >> 1);
        if (!mbar_wait(acc_empty(buf), (use & 1) ^ 1, &abort_flag, a.dev_error, kDevTimeoutTmemFree)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * ACC_STRIDE);
        for (int cb = 0; cb < a.cin_blocks && ok; ++cb) {
          if (!mbar_wait(a_full(aslot), aphase, &abort_flag, a.dev_error, kDevTimeoutTmaFull)) { ok = false; break; }
          const uint32_t sa = smem_base + aslot * A_BYTES;
          for (int r = 0; r < 3; ++r) {
            if (a.resident) bslot = cb * 3 + r;
            else if (!mbar_wait(b_full(bslot), bphase, &abort_flag, a.dev_error, kDevTimeoutTmaFull)) { ok = false; break; }
            tc_fence_after();
            // filter row r: accumulator row (ph, j) reads patch row (ph + r) * 16 + j, i.e. the 128 rows
            // that start r * 16 rows (2 KB) into the patch; B is the row's 192 x 64 slice [s][k][c]
            const uint64_t da = smem_desc_sw128(sa + (uint32_t)r * (AW * 128u), 16);
            const uint64_t db = smem_desc_sw128(b_base + bslot * B_BYTES, 16);
            umma_bf16(d_tmem, da, db, idesc, (cb | r) != 0 ? 1u : 0u);
#pragma unroll
            for (int k = 1; k < BK / 16; ++k)
              umma_bf16_acc(d_tmem, desc_advance(da, k * 32), desc_advance(db, k * 32), idesc);
            if (!a.resident) umma_commit(b_empty(bslot));
            if (!a.resident && ++bslot == a.nb) { bslot = 0; bphase ^= 1; }
          }
          if (!ok) break;
          umma_commit(a_empty(aslot));
          if (++aslot == a.na) { aslot = 0; aphase ^= 1; }
        }
        if (ok) umma_commit(acc_full(buf));
      }
      if (!ok) {
        umma_commit(drain_bar);
        const unsigned long long t0 = global_timer_ns();
        while (!mbar_try_wait(drain_bar, 0) && global_timer_ns() - t0 < 100000000ull) {}
      }
    }
  } else if (warp >= 4) {
    // ---------------- epilogue ----------------
    // Two groups of eight warps take alternate tiles, each with its own accumulator buffer, staging
    // tile, mask tile and named barrier, so that the latency chain of one tile's epilogue (wait,
    // tensor-memory loads, shuffles, staging, store) overlaps the other group's.
    const int group = (warp - 4) >> 3;            // accumulator buffer, staging tile and barrier of this group
    const int quarter = warp & 3;                 // the tensor-memory lane quarter this warp may read
    const int c_first = (((warp - 4) >> 2) & 1) * 32;  // this warp's 32 output channels, 16 at a time
    const int ph = quarter * 2 + (lane >> 4);     // accumulator row (ph, j)
    const int j = lane & 15;
    const bool col_ok = j < TW;                   // columns 14, 15 only feed their left neighbours
    const int rr = ph * TW + j;                   // row of the 8 x 14 staging / mask tile
    const bool issuer = threadIdx.x == 128 + group * kGroupThreads;  // owns the group's TMA stores and mask loads
    const int bar_id = 1 + group;
    uint8_t* stage_row = smem_raw + (out_smem - smem_u32(smem_raw)) + group * OUT_BYTES + rr * 128;
    const uint32_t my_mask = mask_smem + group * OUT_BYTES;
    const uint8_t* mask_row = smem_raw + (my_mask - smem_u32(smem_raw)) + rr * 128;
    const uint32_t my_mask_bar = mask_bar(group);
    const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(group * ACC_STRIDE);
    const bool pool_lane = lane < 16 && (j & 1) == 0 && col_ok;
    uint32_t use = 0;  // tiles this group has taken
    bool mask_pending = false;  // issuer only: a mask copy is in flight or unread
    // Input gradient: the group's mask tile (the layer below's output at the tile's pixels) by TMA.  The
    // issuer requests the NEXT tile's as soon as the whole group has read the current one, so the copy's
    // latency hides behind the store and the wait for the next accumulator.
    auto request_mask = [&](int tile) {
      if (tile >= a.tiles) return;
      const int tw = tile % a.tiles_w, t = tile / a.tiles_w;
      mbar_expect_tx(my_mask_bar, OUT_BYTES);
      tma_load_4d(my_mask, &map_m, my_mask_bar, 0, tw * TW, (t % a.tiles_h) * TH, t / a.tiles_h);
      mask_pending = true;
    };
    if (a.mask && issuer) request_mask(blockIdx.x + group * gridDim.x);
    for (int tile = blockIdx.x + group * gridDim.x; tile < a.tiles; tile += 2 * gridDim.x, ++use) {
      const bool got = mbar_wait(acc_full(group), use & 1, &abort_flag, a.dev_error, kDevTimeoutAccum);
      if (named_bar_or(bar_id, kGroupThreads, !got)) break;  // the group's warps leave together
      tc_fence_after();
      const int tw = tile % a.tiles_w, t = tile / a.tiles_w;
      const int w0 = tw * TW, h0 = (t % a.tiles_h) * TH, img = t / a.tiles_h;
      // Phase 1: the accumulator into registers (three partial sums per value, added across lanes), bias, ReLU,
      // bf16 - and the accumulator goes back to the MMA thread at once: everything that can make this group wait
      // (its previous store still reading the staging tile, the mask tile's copy) comes after.
      uint32_t packed[16];
#pragma unroll
      for (int pass = 0; pass < 2; ++pass) {
        const int c16 = c_first + 16 * pass;
        uint32_t v0[16], v1[16], v2[16];
        tmem_ld_32x16(t_row + (uint32_t)c16, v0);
        tmem_ld_32x16(t_row + (uint32_t)(64 + c16), v1);
        tmem_ld_32x16(t_row + (uint32_t)(128 + c16), v2);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 16; i += 2) {
          // out(ph, j) = D(ph, j)[s = 0] + D(ph, j + 1)[s = 1] + D(ph, j + 2)[s = 2]
          float x0 = __uint_as_float(v0[i]) + __shfl_down_sync(0xffffffffu, __uint_as_float(v1[i]), 1) +
                     __shfl_down_sync(0xffffffffu, __uint_as_float(v2[i]), 2);
          float x1 = __uint_as_float(v0[i + 1]) + __shfl_down_sync(0xffffffffu, __uint_as_float(v1[i + 1]), 1) +
                     __shfl_down_sync(0xffffffffu, __uint_as_float(v2[i + 1]), 2);
          x0 += bias_s[c16 + i]; x1 += bias_s[c16 + i + 1];
          if (a.relu) { x0 = fmaxf(x0, 0.f); x1 = fmaxf(x1, 0.f); }
          __nv_bfloat162 hh = __floats2bfloat162_rn(x0, x1);
          packed[pass * 8 + (i >> 1)] = *reinterpret_cast<uint32_t*>(&hh);
        }
      }
      tc_fence_before();
      mbar_arrive(acc_empty(group));
      // Phase 2: mask, staging tile, pooled output
      if (a.out) {
        // the group's previous store has read the staging tile, and (barrier above) every thread of
        // the group is done with the previous mask tile
        if (issuer) tma_store_wait_read<0>();
        named_bar_sync(bar_id, kGroupThreads);
      }
      // a failed wait leaves the tile unmasked; the error word says so
      if (a.mask) mbar_wait(my_mask_bar, use & 1, &abort_flag, a.dev_error, kDevTimeoutTmaFull);
      bf16* pool_row = a.pooled ? a.pooled + (((long)img * (a.H / 2) + (h0 + ph) / 2) * (a.W / 2) + (w0 + j) / 2) * 64
                                : nullptr;
      uint8_t* code_row = (MODE == 1 && a.code) ? a.code + (((long)img * (a.H / 2) + (h0 + ph) / 2) * (a.W / 2) + (w0 + j) / 2) * 64
                                 : nullptr;
      // pool scatter: this thread's 32 code bytes
      uint4 sc[2];
      if (MODE == 2 && col_ok) {
        const uint4* cp = reinterpret_cast<const uint4*>(a.scatter_code + (((long)img * a.H + h0 + ph) * a.W + w0 + j) * 64 + c_first);
        sc[0] = __ldg(cp); sc[1] = __ldg(cp + 1);
      }
#pragma unroll
      for (int pass = 0; pass < 2; ++pass) {
        const int c16 = c_first + 16 * pass;
        uint32_t (&pk)[8] = reinterpret_cast<uint32_t (&)[8]>(packed[pass * 8]);
        const int chunk0 = c16 >> 3;  // first of this pass's two 16-byte chunks of the 128-byte row
        if (a.mask && col_ok) {
#pragma unroll
          for (int q = 0; q < 2; ++q) {
            const uint4 m = *reinterpret_cast<const uint4*>(mask_row + (((chunk0 + q) ^ (rr & 7)) << 4));
            const uint32_t mw[4] = {m.x, m.y, m.z, m.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              // a bf16 is > 0 iff its sign bit is clear and it is not zero
              const uint32_t lo = mw[e] & 0xFFFFu, hi = mw[e] >> 16;
              uint32_t keep = 0;
              if (lo != 0 && !(lo & 0x8000u)) keep |= 0x0000FFFFu;
              if (hi != 0 && !(hi & 0x8000u)) keep |= 0xFFFF0000u;
              pk[q * 4 + e] &= keep;
            }
          }
        }
        if (a.out && col_ok) {
#pragma unroll
          for (int q = 0; q < 2; ++q)
            *reinterpret_cast<uint4*>(stage_row + (((chunk0 + q) ^ (rr & 7)) << 4)) =
                make_uint4(pk[q * 4], pk[q * 4 + 1], pk[q * 4 + 2], pk[q * 4 + 3]);
        }
        if (a.pooled) {
          // 2x2 window: columns j, j + 1 (next lane) of rows ph, ph + 1 (16 lanes on); in place (the tile is
          // already in the staging tile, and the pool scatter, which reads these values again, has no pooled output)
          uint32_t codes[4];
          if (MODE == 1) pool2x2_codes<8>(pk, 1, 16, codes);
          else pool2x2<8>(pk, 1, 16);
          if (pool_lane) {
            uint4* pp = reinterpret_cast<uint4*>(pool_row + c16);
            pp[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            pp[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
            if (code_row) *reinterpret_cast<uint4*>(code_row + c16) = make_uint4(codes[0], codes[1], codes[2], codes[3]);
          }
        }
      }
      if (a.out) {
        fence_async_smem();
        named_bar_sync(bar_id, kGroupThreads);  // the staging tile is complete, and the group has read its mask tile
        if (issuer) {
          tma_store_4d(&map_y, out_smem + group * OUT_BYTES, 0, w0, h0, img);
          tma_store_commit();
          if (a.mask) {
            mask_pending = false;
            request_mask(tile + 2 * gridDim.x);
          }
        }
      }
      if (MODE == 2) {
        // four rounds through the group's staging tile, one per window position q = 2a + b: the value where
        // the window's code names q, zero elsewhere; the store's tensor map addresses pixel (2h + a, 2w + b)
        // of the full-resolution gradient for tile coordinate (h, w)
        const uint32_t kw[8] = {sc[0].x, sc[0].y, sc[0].z, sc[0].w, sc[1].x, sc[1].y, sc[1].z, sc[1].w};
#pragma unroll 1
        for (uint32_t q = 0; q < 4; ++q) {
          if (issuer) tma_store_wait_read<0>();  // the previous round's store has read the staging tile
          named_bar_sync(bar_id, kGroupThreads);
          if (col_ok) {
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {  // 16-byte chunks: 8 channels, 8 code bytes (two words)
              uint32_t o[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const uint32_t k2 = kw[ch * 2 + (e >> 1)] >> (16 * (e & 1));  // the codes of channels 2e, 2e + 1 of this chunk
                uint32_t keep = 0;
                if ((k2 & 0xFFu) == q) keep |= 0x0000FFFFu;
                if (((k2 >> 8) & 0xFFu) == q) keep |= 0xFFFF0000u;
                o[e] = packed[ch * 4 + e] & keep;
              }
              *reinterpret_cast<uint4*>(stage_row + ((((c_first >> 3) + ch) ^ (rr & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
            }
          }
          fence_async_smem();
          named_bar_sync(bar_id, kGroupThreads);
          if (issuer) {
            const uint32_t src = out_smem + group * OUT_BYTES;
            if (q == 0) tma_store_4d(&map_s0, src, 0, w0, h0, img);
            else if (q == 1) tma_store_4d(&map_s1, src, 0, w0, h0, img);
            else if (q == 2) tma_store_4d(&map_s2, src, 0, w0, h0, img);
            else tma_store_4d(&map_s3, src, 0, w0, h0, img);
            tma_store_commit();
          }
        }
      }
    }
    if (issuer && mask_pending) {
      // left early (a wait ran out) with a mask copy in flight: let it land before shared memory goes away
      const unsigned long long t0 = global_timer_ns();
      while (!mbar_try_wait(my_mask_bar, use & 1) && global_timer_ns() - t0 < 100000000ull) {}
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

bool tc_conv3x3_rowshift_supported(ConvShape s) {
  return s.Cout == 64 && s.Cin % 64 == 0 && s.W % TW == 0 && s.H % TH == 0 && s.W >= 56 && s.H % 2 == 0 &&
         (long)s.N * s.H * s.W < (1L << 31) - 256;
}

cudaError_t tc_conv3x3_rowshift(const bf16* in, const bf16* wt_tap_major, const float* bias, const bf16* mask, bf16* out,
                                bf16* pooled, ConvShape s, bool relu, int* dev_error, cudaStream_t st, uint8_t* code,
                                const uint8_t* scatter_code, bf16* scatter_out) {
  if (!out && !pooled && !scatter_out) return cudaErrorInvalidValue;
  if (mask && !out) return cudaErrorInvalidValue;
  if ((scatter_code == nullptr) != (scatter_out == nullptr) || (scatter_out && (out || pooled || mask))) return cudaErrorInvalidValue;
  if (code && !pooled) return cudaErrorInvalidValue;
  if (!tc_conv3x3_rowshift_supported(s)) return cudaErrorInvalidValue;
  CUtensorMap mx, mw;
  if (!make_patch_map(&mx, in, s.N, s.H, s.W, s.Cin, AW, IH)) return cudaErrorInvalidValue;
  if (!make_filter_row_map(&mw, wt_tap_major, s.Cout, s.Cin, 64)) return cudaErrorInvalidValue;
  CUtensorMap my = mw;  // only read when there is a full-resolution output
  if (out && !make_patch_map(&my, out, s.N, s.H, s.W, s.Cout, TW, TH)) return cudaErrorInvalidValue;
  CUtensorMap mm = mw;  // only read when there is a mask
  if (mask && !make_patch_map(&mm, mask, s.N, s.H, s.W, s.Cout, TW, TH)) return cudaErrorInvalidValue;
  // pool scatter: four views of the full-resolution gradient [N][2H][2W][64], one per window position
  // (a, b): pixel (h, w) of the view is pixel (2h + a, 2w + b) of the tensor
  CUtensorMap ms[4] = {mw, mw, mw, mw};
  if (scatter_out)
    for (int q = 0; q < 4; ++q)
      if (!make_window_map(&ms[q], scatter_out, s.N, 2 * s.H, 2 * s.W, s.Cout, q >> 1, q & 1, TW, TH)) return cudaErrorInvalidValue;
  RowArgs a;
  a.code = code; a.scatter_code = scatter_code;
  a.N = s.N; a.H = s.H; a.W = s.W;
  a.cin_blocks = s.Cin / 64;
  a.tiles_w = s.W / TW; a.tiles_h = s.H / TH;
  a.tiles = s.N * a.tiles_w * a.tiles_h;
  a.relu = relu ? 1 : 0; a.bias = bias; a.mask = mask; a.out = out; a.pooled = pooled; a.dev_error = dev_error;
  // shared-memory plan: the whole filter resident beside at least two patch slots if it fits, else a
  // ring of filter rows; the rest goes to patch slots
  const int fixed = (mask ? 4 : 2) * OUT_BYTES + 1024 + 512;  // a staging (and a mask) tile per epilogue group
  const int res_bytes = a.cin_blocks * 3 * B_BYTES;
  if (res_bytes + 2 * A_BYTES + fixed <= kLimit) {
    a.resident = 1; a.nb = 0; a.b_region_bytes = res_bytes;
  } else {
    a.resident = 0;
    int nb = kMaxFilterSlots;
    while (nb > 2 && nb * B_BYTES + 2 * A_BYTES + fixed > kLimit) --nb;
    a.nb = nb; a.b_region_bytes = nb * B_BYTES;
  }
  int na = (kLimit - fixed - a.b_region_bytes) / A_BYTES;
  a.na = na > kMaxPatchSlots ? kMaxPatchSlots : na;
  if (a.na < 2) return cudaErrorInvalidValue;
  const int smem = a.na * A_BYTES + a.b_region_bytes + fixed;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(conv3x3_rowshift_tc_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, kLimit);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(conv3x3_rowshift_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kLimit);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(conv3x3_rowshift_tc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kLimit);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int grid = a.tiles < sms ? a.tiles : sms;
  if (scatter_out) conv3x3_rowshift_tc_kernel<2><<<grid, kThreads, smem, st>>>(mx, mw, my, mm, ms[0], ms[1], ms[2], ms[3], a);
  else if (code) conv3x3_rowshift_tc_kernel<1><<<grid, kThreads, smem, st>>>(mx, mw, my, mm, ms[0], ms[1], ms[2], ms[3], a);
  else conv3x3_rowshift_tc_kernel<0><<<grid, kThreads, smem, st>>>(mx, mw, my, mm, ms[0], ms[1], ms[2], ms[3], a);
  return cudaGetLastError();
}

}  // namespace vgg
