// 3x3 convolution on tcgen05 with the input patch held in shared memory once
// for all nine filter taps.
//
// The general kernel (tc_kernels.cu) fetches the input tile again for every
// tap, so it moves nine times the input through the L2-to-SM path; on the
// large-image layers with few channels (224x224 and 112x112, 64-128 channels)
// that path, not the tensor pipe, sets the speed.  Here a tile is a patch of
// 8 (wide) x 16 (high) output pixels.  For each block of 64 input channels the
// producer loads the 10 x 18 input patch (one pixel of halo, zero-filled
// outside the image by TMA) once: 180 rows of 128 bytes, 128-byte swizzled.
// Output pixel (ph, pw) and tap (r, s) read patch row (ph + r) * 10 + pw + s, so
// for a fixed tap the 128 rows of the MMA's A operand are 16 groups of 8
// consecutive rows, 10 rows apart: a K-major operand with a stride of
// 1280 bytes between 8-row groups, starting (r * 10 + s) rows into the patch.
// The nine taps are nine MMAs on the same buffer with different start rows.
// The filter is read from a tap-major copy [9][Cout][Cin], so that one TMA box
// brings a whole filter row (three taps x BN x 64) into one slot of its own ring:
// one barrier hand-off per twelve MMAs instead of per four (with four the
// producer thread, not the tensor pipe, set the pace).
//
// Warps: 0 patch producer, 1 MMA issuer + TMEM owner, 2-5 epilogue, 6 filter
// producer.  Accumulator double-buffered; persistent CTAs; time-limited waits.
//
// PAIR: two CTAs (a cluster, tcgen05 cta_group::2) work as one: each loads the patch of its own
// tile and HALF of the filter's output channels, the even CTA issues MMAs of 256 rows (both
// patches) whose B operand the hardware gathers from both CTAs, and each CTA finds its 128
// accumulator rows in its own tensor memory.  With 128 output channels one CTA's MMA reads 8 KB of
// shared memory per 64 cycles, all the bandwidth there is; as a pair it reads 6 KB.
#include "tc_common.cuh"
#include "tc_kernels.cuh"

namespace vgg {
namespace {

using namespace tc;

constexpr int BM = 128, BK = 64;
constexpr int PW = 8, PH = 16;                  // output patch
constexpr int IW = PW + 2, IH = PH + 2;         // input patch with halo
constexpr int A_BYTES = IW * IH * 128;          // 23040
constexpr int A_SLOT = 23 * 1024;               // 1024-byte aligned slot
constexpr int kThreads = 224;
constexpr int kMaxPatchSlots = 6;

template <int BN, bool PAIR>
struct HaloTile {
  static constexpr int BNH = PAIR ? BN / 2 : BN;  // filter rows (output channels) this CTA stages per tap
  static constexpr int TAP_BYTES = BNH * BK * 2;  // one tap's slice of the filter
  static constexpr int B_BYTES = 3 * TAP_BYTES;   // a filter row: three taps
  static constexpr int OUT_BYTES = BM * 64 * 2;   // staging tile of the TMA store; a second one holds the mask tile
  // Shared memory: `na` input-patch slots, the filter region, two staging tiles, barriers.  The filter
  // region either holds the layer's whole filter slice for this kernel's BN output channels
  // (cin_blocks x 9 taps, loaded once per CTA: "resident") or is a ring of `nb` filter rows.
  // two output staging tiles (alternating, so a store can drain while the next chunk is converted),
  // plus a mask tile for the input gradient
  static constexpr int fixed_bytes(bool with_mask) { return (with_mask ? 3 : 2) * OUT_BYTES + 1024 + 512; }
  static constexpr int kLimit = 227 * 1024 - 2560;  // static shared memory (bias, flags) comes on top
};

struct HaloArgs {
  int N, H, W;
  int cin_blocks, Cin, Cout;
  int tiles_w, tiles_h, m_tiles, n_tiles;
  int relu;
  const float* bias;
  int na, nb, resident, b_region_bytes;  // shared-memory plan (see HaloTile)
  const bf16* mask;
  bf16* out;     // full-resolution output, or null when only the pooled output is wanted
  bf16* pooled;  // 2x2 max-pooled output [N][H/2][W/2][Cout], or null
  uint8_t* code; // with pooled: arg-max code of every window (see simt_maxpool_fwd), or null
  // Pool scatter (input gradient of a layer whose input is a pooled tensor): each 64-channel chunk of the
  // tile is stored four times, once per window position, into the full-resolution gradient of the layer
  // below the pool, keeping a value only at the position its window's stored code names.
  const uint8_t* scatter_code;  // [N][H][W][Cout] at this kernel's resolution, or null
  int* dev_error;
};

// MODE 0: plain (output, mask, pooled output); 1: pooled output with arg-max codes; 2: pool scatter.
// Compile-time so that the plain kernel carries none of the other two's registers and instructions.
template <int BN, bool PAIR, int MODE>
__global__ void __launch_bounds__(kThreads, 1)
conv3x3_halo_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                       const __grid_constant__ CUtensorMap map_y, const __grid_constant__ CUtensorMap map_m,
                       const __grid_constant__ CUtensorMap map_s0, const __grid_constant__ CUtensorMap map_s1,
                       const __grid_constant__ CUtensorMap map_s2, const __grid_constant__ CUtensorMap map_s3,
                       HaloArgs a) {
  using T = HaloTile<BN, PAIR>;
  constexpr int NA = kMaxPatchSlots, NB = 4;  // most slots a plan may use (barrier numbering)
  // Accumulator buffers in tensor memory.  A tile here lasts a microsecond or two, about as long as
  // the hand-off to the epilogue and back takes, so two buffers leave the tensor pipe waiting.
  constexpr int NACC = 4;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t b_base = smem_base + a.na * A_SLOT;
  const uint32_t out_smem = b_base + a.b_region_bytes;  // 1024-byte aligned
  const uint32_t mask_smem = out_smem + 2 * T::OUT_BYTES;
  const uint32_t bars = mask_smem + (a.mask ? T::OUT_BYTES : 0);
  auto a_full = [&](int s) { return bars + 8u * s; };
  auto a_empty = [&](int s) { return bars + 8u * (NA + s); };
  auto b_full = [&](int s) { return bars + 8u * (2 * NA + s); };
  auto b_empty = [&](int s) { return bars + 8u * (2 * NA + NB + s); };
  auto acc_full = [&](int b) { return bars + 8u * (2 * NA + 2 * NB + b); };
  auto acc_empty = [&](int b) { return bars + 8u * (2 * NA + 2 * NB + NACC + b); };
  const uint32_t drain_bar = bars + 8u * (2 * NA + 2 * NB + 2 * NACC);
  const uint32_t mask_bar = bars + 8u * (2 * NA + 2 * NB + 2 * NACC + 1);
  const uint32_t w_bar = bars + 8u * (2 * NA + 2 * NB + 2 * NACC + 2);  // resident filter loaded
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  __shared__ __align__(16) float bias_s[512];  // the layer's bias (zeros when it has none)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Work units: tiles, or with PAIR two tiles side by side in the tile order (m_tiles is even).
  // Barriers the MMA issuer waits on (patch, filter, accumulator drained) are the even CTA's.
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;
  const int first_unit = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int unit_stride = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  const int total_units = (PAIR ? a.m_tiles / 2 : a.m_tiles) * a.n_tiles;
  auto unit_m_tile = [&](int u) { return PAIR ? 2 * (u / a.n_tiles) + (int)rank : u / a.n_tiles; };

  for (int i = threadIdx.x; i < a.Cout; i += kThreads) bias_s[i] = a.bias ? a.bias[i] : 0.f;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < NA; ++s) { mbar_init(a_full(s), 1); mbar_init(a_empty(s), 1); }
    for (int s = 0; s < NB; ++s) { mbar_init(b_full(s), 1); mbar_init(b_empty(s), 1); }
    for (int b = 0; b < NACC; ++b) { mbar_init(acc_full(b), 1); mbar_init(acc_empty(b), PAIR ? 2 : 128); }
    mbar_init(drain_bar, 1);
    mbar_init(mask_bar, 1);
    mbar_init(w_bar, 1);
    mbar_fence_init();
    tma_prefetch_desc(&map_x);
    tma_prefetch_desc(&map_w);
  }
  if (warp == 1) {
    if (PAIR) {
      tmem_alloc_pair(smem_u32(&tmem_base_slot), NACC * BN);
      tmem_relinquish_pair();
    } else {
      tmem_alloc(smem_u32(&tmem_base_slot), NACC * BN);
      tmem_relinquish();
    }
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync_all();  // the peer's barriers are initialised before anything signals them
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
      for (int unit = first_unit; unit < total_units && ok; unit += unit_stride) {
        const int m_tile = unit_m_tile(unit);
        const int tw = m_tile % a.tiles_w, t = m_tile / a.tiles_w;
        const int w0 = tw * PW, h0 = (t % a.tiles_h) * PH, img = t / a.tiles_h;
        for (int cb = 0; cb < a.cin_blocks; ++cb) {
          if (!mbar_wait(a_empty(slot), phase ^ 1, &abort_flag, a.dev_error, kDevTimeoutStageFree)) { ok = false; break; }
          if (PAIR) {
            // both CTAs' patches are counted on the even CTA's barrier, which announces all their bytes
            if (rank == 0) mbar_expect_tx(a_full(slot), 2 * A_BYTES);
            tma_load_4d_pair(smem_base + slot * A_SLOT, &map_x, map_to_cta(a_full(slot), 0), cb * BK, w0 - 1, h0 - 1, img);
          } else {
            mbar_expect_tx(a_full(slot), A_BYTES);
            tma_load_4d(smem_base + slot * A_SLOT, &map_x, a_full(slot), cb * BK, w0 - 1, h0 - 1, img);
          }
          ++fills[slot];
          if (++slot == a.na) { slot = 0; phase ^= 1; }
        }
      }
      if (!ok && rank != 0) {
        // the peer's copies report to the even CTA's barriers: allow them a millisecond to land
        const unsigned long long t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 1000000ull) {}
      } else if (!ok)
        for (int s = 0; s < NA; ++s)
          if (fills[s]) {
            const unsigned long long t0 = global_timer_ns();
            while (!mbar_try_wait(a_full(s), (fills[s] - 1) & 1) && global_timer_ns() - t0 < 100000000ull) {}
          }
    }
  } else if (warp == 6) {
    // ---------------- filter producer ----------------
    if (lane == 0) {
      uint32_t fills[NB];
#pragma unroll
      for (int s = 0; s < NB; ++s) fills[s] = 0;
      int slot = 0;
      uint32_t phase = 0;
      bool ok = true;
      const int row_in_tile = (int)rank * T::BNH;  // this CTA's output channels within the BN of a tile
      if (a.resident) {
        // n_tiles == 1: the whole filter for these output channels, once
        if (PAIR) {
          const uint32_t wb = map_to_cta(w_bar, 0);
          if (rank == 0) mbar_expect_tx(w_bar, (uint32_t)(2 * a.cin_blocks * 3 * T::B_BYTES));
          for (int cb = 0; cb < a.cin_blocks; ++cb)
            for (int r = 0; r < 3; ++r)
              tma_load_3d_pair(b_base + (cb * 3 + r) * T::B_BYTES, &map_w, wb, cb * BK, row_in_tile, 3 * r);
        } else {
          mbar_expect_tx(w_bar, (uint32_t)(a.cin_blocks * 3 * T::B_BYTES));
          for (int cb = 0; cb < a.cin_blocks; ++cb)
            for (int r = 0; r < 3; ++r)
              tma_load_3d(b_base + (cb * 3 + r) * T::B_BYTES, &map_w, w_bar, cb * BK, 0, 3 * r);
        }
        // never leave with the copy in flight.  (The peer of a pair cannot see the even CTA's barrier;
        // its epilogue does not finish before MMAs that needed this filter have.)
        if (rank == 0) {
          const unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(w_bar, 0) && global_timer_ns() - t0 < 100000000ull) {}
        }
      }
      for (int unit = first_unit; unit < total_units && ok && !a.resident; unit += unit_stride) {
        const int n_tile = unit % a.n_tiles;
        for (int cb = 0; cb < a.cin_blocks && ok; ++cb)
          for (int r = 0; r < 3; ++r) {
            if (!mbar_wait(b_empty(slot), phase ^ 1, &abort_flag, a.dev_error, kDevTimeoutStageFree)) { ok = false; break; }
            if (PAIR) {
              if (rank == 0) mbar_expect_tx(b_full(slot), 2 * T::B_BYTES);
              tma_load_3d_pair(b_base + slot * T::B_BYTES, &map_w, map_to_cta(b_full(slot), 0), cb * BK,
                               n_tile * BN + row_in_tile, 3 * r);
            } else {
              mbar_expect_tx(b_full(slot), T::B_BYTES);
              tma_load_3d(b_base + slot * T::B_BYTES, &map_w, b_full(slot), cb * BK, n_tile * BN, 3 * r);
            }
            ++fills[slot];
            if (++slot == a.nb) { slot = 0; phase ^= 1; }
          }
      }
      if (!ok && rank != 0) {
        const unsigned long long t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 1000000ull) {}
      } else if (!ok)
        for (int s = 0; s < NB; ++s)
          if (fills[s]) {
            const unsigned long long t0 = global_timer_ns();
            while (!mbar_try_wait(b_full(s), (fills[s] - 1) & 1) && global_timer_ns() - t0 < 100000000ull) {}
          }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(PAIR ? 2 * BM : BM, BN, 0, 0);
      int aslot = 0, bslot = 0;
      uint32_t aphase = 0, bphase = 0;
      int local = 0;
      bool ok = true;
      if (a.resident) ok = mbar_wait(w_bar, 0, &abort_flag, a.dev_error, kDevTimeoutTmaFull);
      for (int unit = first_unit; unit < total_units && ok; unit += unit_stride, ++local) {
        const int buf = local % NACC;
        const uint32_t use = (uint32_t)(local / NACC);
        if (!mbar_wait(acc_empty(buf), (use & 1) ^ 1, &abort_flag, a.dev_error, kDevTimeoutTmemFree)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
        for (int cb = 0; cb < a.cin_blocks && ok; ++cb) {
          if (!mbar_wait(a_full(aslot), aphase, &abort_flag, a.dev_error, kDevTimeoutTmaFull)) { ok = false; break; }
          const uint32_t sa = smem_base + aslot * A_SLOT;
          for (int r = 0; r < 3; ++r) {
            if (a.resident) bslot = cb * 3 + r;
            else if (!mbar_wait(b_full(bslot), bphase, &abort_flag, a.dev_error, kDevTimeoutTmaFull)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int s = 0; s < 3; ++s) {
              const uint32_t sb = b_base + bslot * T::B_BYTES + s * T::TAP_BYTES;
              const uint32_t a_tap = sa + (uint32_t)(r * IW + s) * 128u;
              const uint64_t da = smem_desc_sw128_sbo(a_tap, IW * 128), db = smem_desc_sw128(sb, 16);
              if (PAIR) {
                umma_bf16_pair(d_tmem, da, db, idesc, (cb | r | s) != 0 ? 1u : 0u);
#pragma unroll
                for (int k = 1; k < BK / 16; ++k)
                  umma_bf16_pair_acc(d_tmem, desc_advance(da, k * 32), desc_advance(db, k * 32), idesc);
              } else {
                umma_bf16(d_tmem, da, db, idesc, (cb | r | s) != 0 ? 1u : 0u);
#pragma unroll
                for (int k = 1; k < BK / 16; ++k)
                  umma_bf16_acc(d_tmem, desc_advance(da, k * 32), desc_advance(db, k * 32), idesc);
              }
            }
            if (!a.resident) { if (PAIR) umma_commit_pair(b_empty(bslot), 3); else umma_commit(b_empty(bslot)); }
            if (!a.resident && ++bslot == a.nb) { bslot = 0; bphase ^= 1; }
          }
          if (!ok) break;
          if (PAIR) umma_commit_pair(a_empty(aslot), 3); else umma_commit(a_empty(aslot));
          if (++aslot == a.na) { aslot = 0; aphase ^= 1; }
        }
        if (ok) { if (PAIR) umma_commit_pair(acc_full(buf), 3); else umma_commit(acc_full(buf)); }
      }
      if (!ok) {
        if (PAIR) umma_commit_pair(drain_bar, 1); else umma_commit(drain_bar);
        const unsigned long long t0 = global_timer_ns();
        while (!mbar_try_wait(drain_bar, 0) && global_timer_ns() - t0 < 100000000ull) {}
      }
    }
  } else {
    // ---------------- epilogue ----------------
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    int local = 0;
    // The full-resolution tile leaves 64 channels at a time through a 128-byte-swizzled staging tile
    // and one TMA store; the pooled output (a quarter of it) is stored directly.  Thread 64 owns the
    // store groups.
    const bool issuer = threadIdx.x == 64;
    uint8_t* stage_row0 = smem_raw + (out_smem - smem_u32(smem_raw)) + row * 128;
    uint32_t stage_sel = 0;  // which of the two staging tiles the next chunk uses
    const uint8_t* mask_srow = smem_raw + (mask_smem - smem_u32(smem_raw)) + row * 128;
    uint32_t mask_phase = 0;
    bool mask_pending = false;  // issuer only: a mask copy is in flight or unread
    // Input gradient: the ReLU mask (the layer below's output at the same pixels) of a 64-channel chunk
    // arrives as one tiled box in the staging layout.  The issuer requests the NEXT chunk's box as soon
    // as every thread has read the current one, so that the copy's latency hides behind the rest of
    // the epilogue and the wait for the next accumulator.
    auto request_mask = [&](int unit, int c64) {
      if (unit >= total_units) return;
      const int mt = unit_m_tile(unit), nt = unit % a.n_tiles;
      const int tw = mt % a.tiles_w, t = mt / a.tiles_w;
      mbar_expect_tx(mask_bar, T::OUT_BYTES);
      tma_load_4d(mask_smem, &map_m, mask_bar, nt * BN + c64, tw * PW, (t % a.tiles_h) * PH, t / a.tiles_h);
      mask_pending = true;
    };
    if (a.mask && issuer) request_mask(first_unit, 0);
    for (int unit = first_unit; unit < total_units; unit += unit_stride, ++local) {
      const int buf = local % NACC;
      const uint32_t use = (uint32_t)(local / NACC);
      const int m_tile = unit_m_tile(unit), n_tile = unit % a.n_tiles;
      const bool got = mbar_wait(acc_full(buf), use & 1, &abort_flag, a.dev_error, kDevTimeoutAccum);
      if (named_bar_or(1, 128, !got)) break;  // all four warps leave together
      tc_fence_after();
      const int tw = m_tile % a.tiles_w, t = m_tile / a.tiles_w;
      const int th = t % a.tiles_h, img = t / a.tiles_h;
      const int h = th * PH + row / PW;
      const int w = tw * PW + row % PW;
      const int c_base = n_tile * BN;
      // 2x2 pooling: a warp holds four patch rows of eight pixels (lane = 8 * row + column), so every
      // window lies inside one warp; the lane of the window's top-left pixel stores the maximum
      const bool pool_lane = (lane & 1) == 0 && (lane & 8) == 0;
      bf16* pool_row = a.pooled ? a.pooled + (((long)img * (a.H / 2) + h / 2) * (a.W / 2) + w / 2) * a.Cout + c_base
                                : nullptr;
      uint8_t* code_row = (MODE == 1 && a.code) ? a.code + (((long)img * (a.H / 2) + h / 2) * (a.W / 2) + w / 2) * a.Cout + c_base : nullptr;
      const uint8_t* scode_row = (MODE == 2 && h < a.H) ? a.scatter_code + (((long)img * a.H + h) * a.W + w) * a.Cout + c_base
                                                             : nullptr;
#pragma unroll 1
      for (int c64 = 0; c64 < BN; c64 += 64) {
        if (a.out) {
          if (issuer) tma_store_wait_read<1>();  // the store before last, which used this staging tile, has read it
          named_bar_sync(1, 128);
        }
        // pool scatter: this pixel's 64 code bytes, requested before the tensor-memory loads
        uint4 sc[4];
        if (MODE != 2) {
        } else if (scode_row) {
#pragma unroll
          for (int q = 0; q < 4; ++q) sc[q] = __ldg(reinterpret_cast<const uint4*>(scode_row + c64) + q);
        } else {
#pragma unroll
          for (int q = 0; q < 4; ++q) sc[q] = make_uint4(0x04040404u, 0x04040404u, 0x04040404u, 0x04040404u);
        }
        uint32_t kept[32];  // pool scatter: the chunk's values (bf16 pairs) of this pixel
        bool mask_ready = false;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const int cc = c64 + half * 32;
          uint32_t v[32];
          tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN + cc), v);
          tmem_ld_wait();
          uint32_t packed[16];
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            float x0 = __uint_as_float(v[j]), x1 = __uint_as_float(v[j + 1]);
            x0 += bias_s[c_base + cc + j]; x1 += bias_s[c_base + cc + j + 1];
            if (a.relu) { x0 = fmaxf(x0, 0.f); x1 = fmaxf(x1, 0.f); }
            __nv_bfloat162 hh = __floats2bfloat162_rn(x0, x1);
            packed[j >> 1] = *reinterpret_cast<uint32_t*>(&hh);
          }
          if (a.mask) {
            if (!mask_ready) {  // a failed wait leaves the tile unmasked; the error word says so
              mbar_wait(mask_bar, mask_phase, &abort_flag, a.dev_error, kDevTimeoutTmaFull);
              mask_phase ^= 1;
              mask_ready = true;
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const uint4 m = *reinterpret_cast<const uint4*>(mask_srow + (((half * 4 + q) ^ (row & 7)) << 4));
              const uint32_t mw[4] = {m.x, m.y, m.z, m.w};
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const uint32_t lo = mw[e] & 0xFFFFu, hi = mw[e] >> 16;
                uint32_t keep = 0;
                if (lo != 0 && !(lo & 0x8000u)) keep |= 0x0000FFFFu;
                if (hi != 0 && !(hi & 0x8000u)) keep |= 0xFFFF0000u;
                packed[q * 4 + e] &= keep;
              }
            }
          }
          if (MODE == 2) {
#pragma unroll
            for (int i = 0; i < 16; ++i) kept[half * 16 + i] = packed[i];
          }
          if (a.out) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const int chunk = half * 4 + q;  // 16-byte chunk of the 128-byte staging row
              *reinterpret_cast<uint4*>(stage_row0 + stage_sel * T::OUT_BYTES + ((chunk ^ (row & 7)) << 4)) =
                  make_uint4(packed[q * 4], packed[q * 4 + 1], packed[q * 4 + 2], packed[q * 4 + 3]);
            }
          }
          if (a.pooled) {
            // 2x2 window: columns w, w + 1 (next lane) of rows h, h + 1 (8 lanes on)
            uint32_t codes[8];
            if (MODE == 1) pool2x2_codes<16>(packed, 1, 8, codes);
            else pool2x2<16>(packed, 1, 8);
            if (pool_lane) {
              uint4* pp = reinterpret_cast<uint4*>(pool_row + cc);
#pragma unroll
              for (int q = 0; q < 4; ++q)
                pp[q] = make_uint4(packed[q * 4], packed[q * 4 + 1], packed[q * 4 + 2], packed[q * 4 + 3]);
              if (code_row) {
                uint4* kp = reinterpret_cast<uint4*>(code_row + cc);
                kp[0] = make_uint4(codes[0], codes[1], codes[2], codes[3]);
                kp[1] = make_uint4(codes[4], codes[5], codes[6], codes[7]);
              }
            }
          }
        }
        if (a.out) {
          fence_async_smem();
          named_bar_sync(1, 128);  // the staging tile is complete, and everyone has read the mask tile
          if (issuer) {
            tma_store_4d(&map_y, out_smem + stage_sel * T::OUT_BYTES, c_base + c64, tw * PW, th * PH, img);
            tma_store_commit();
            if (a.mask) {
              mask_pending = false;
              if (c64 + 64 < BN) request_mask(unit, c64 + 64); else request_mask(unit + unit_stride, 0);
            }
          }
          stage_sel ^= 1;
        }
        if (MODE == 2) {
          // four rounds through the two staging tiles in turn, one per window position q = 2a + b: the value
          // where the window's code names q, zero elsewhere; the store's tensor map addresses pixel
          // (2h + a, 2w + b) of the full-resolution gradient for patch coordinate (h, w)
          const uint32_t kw[16] = {sc[0].x, sc[0].y, sc[0].z, sc[0].w, sc[1].x, sc[1].y, sc[1].z, sc[1].w,
                                   sc[2].x, sc[2].y, sc[2].z, sc[2].w, sc[3].x, sc[3].y, sc[3].z, sc[3].w};
#pragma unroll 1
          for (uint32_t q = 0; q < 4; ++q) {
            if (issuer) tma_store_wait_read<1>();  // the store before last, which used this staging tile, has read it
            named_bar_sync(1, 128);
#pragma unroll
            for (int ch = 0; ch < 8; ++ch) {  // 16-byte chunks: 8 channels, 8 code bytes (two words)
              uint32_t o[4];
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const uint32_t k2 = kw[ch * 2 + (e >> 1)] >> (16 * (e & 1));  // codes of channels 2e, 2e + 1 of the chunk
                uint32_t keep = 0;
                if ((k2 & 0xFFu) == q) keep |= 0x0000FFFFu;
                if (((k2 >> 8) & 0xFFu) == q) keep |= 0xFFFF0000u;
                o[e] = kept[ch * 4 + e] & keep;
              }
              *reinterpret_cast<uint4*>(stage_row0 + stage_sel * T::OUT_BYTES + ((ch ^ (row & 7)) << 4)) =
                  make_uint4(o[0], o[1], o[2], o[3]);
            }
            fence_async_smem();
            named_bar_sync(1, 128);
            if (issuer) {
              const uint32_t src = out_smem + stage_sel * T::OUT_BYTES;
              if (q == 0) tma_store_4d(&map_s0, src, c_base + c64, tw * PW, th * PH, img);
              else if (q == 1) tma_store_4d(&map_s1, src, c_base + c64, tw * PW, th * PH, img);
              else if (q == 2) tma_store_4d(&map_s2, src, c_base + c64, tw * PW, th * PH, img);
              else tma_store_4d(&map_s3, src, c_base + c64, tw * PW, th * PH, img);
              tma_store_commit();
            }
            stage_sel ^= 1;
          }
        }
      }
      tc_fence_before();
      if (PAIR) {
        // one arrival per CTA, on the even CTA's barrier: an arrival that crosses the cluster costs far
        // more than a local one, and a tile here lasts a microsecond or two
        named_bar_sync(1, 128);
        if (issuer) mbar_arrive_cluster(map_to_cta(acc_empty(buf), 0));
      } else {
        mbar_arrive(acc_empty(buf));
      }
    }
    if (issuer && mask_pending) {
      // left early (a wait ran out) with a mask copy in flight: let it land before shared memory goes away
      const unsigned long long t0 = global_timer_ns();
      while (!mbar_try_wait(mask_bar, mask_phase) && global_timer_ns() - t0 < 100000000ull) {}
    }
    if (issuer) tma_store_wait_all();  // shared memory must outlive the stores that read it
  }

  tc_fence_before();
  __syncthreads();
  // a pair meets before either CTA releases tensor memory or exits: until then the peer may still
  // signal this CTA's barriers, and the even CTA's MMAs read the peer's shared memory
  if (PAIR) cluster_sync_all();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    if (PAIR) tmem_dealloc_pair(tmem_base, NACC * BN); else tmem_dealloc(tmem_base, NACC * BN);
  }
}

template <int BN, bool PAIR, int MODE>
cudaError_t launch_halo(const CUtensorMap& mx, const CUtensorMap& mw, const CUtensorMap& my, const CUtensorMap& mm,
                        const CUtensorMap* ms, HaloArgs a, cudaStream_t st) {
  using T = HaloTile<BN, PAIR>;
  // plan the shared memory: keep the whole filter resident when it fits beside two or three patch slots
  // (then only the input patches cross the L2-to-SM path, which is what bounds these layers), else
  // stream filter rows through a ring
  const int res_bytes = a.cin_blocks * 3 * T::B_BYTES;
  const int fixed = T::fixed_bytes(a.mask != nullptr);
  a.resident = 0;
  for (int na = kMaxPatchSlots; na >= 2 && !a.resident; --na)
    if (a.n_tiles == 1 && na * A_SLOT + res_bytes + fixed <= T::kLimit) {
      a.resident = 1; a.na = na; a.nb = 0; a.b_region_bytes = res_bytes;
    }
  if (!a.resident) {
    // filter ring of up to four rows (never fewer than two), the rest for patch slots
    int nb = 4;
    while (nb > 2 && 2 * A_SLOT + nb * T::B_BYTES + fixed > T::kLimit) --nb;
    a.nb = nb;
    int na = (T::kLimit - fixed - nb * T::B_BYTES) / A_SLOT;
    a.na = na > kMaxPatchSlots ? kMaxPatchSlots : na;
    if (a.na < 2) return cudaErrorInvalidValue;
    a.b_region_bytes = a.nb * T::B_BYTES;
  }
  const int smem = a.na * A_SLOT + a.b_region_bytes + fixed;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(conv3x3_halo_tc_kernel<BN, PAIR, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, T::kLimit);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (PAIR) {
    const int units = (a.m_tiles / 2) * a.n_tiles;
    const int pairs = units < sms / 2 ? units : sms / 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, conv3x3_halo_tc_kernel<BN, PAIR, MODE>, mx, mw, my, mm, ms[0], ms[1], ms[2], ms[3], a);
  }
  const int tiles = a.m_tiles * a.n_tiles;
  conv3x3_halo_tc_kernel<BN, PAIR, MODE><<<tiles < sms ? tiles : sms, kThreads, smem, st>>>(mx, mw, my, mm, ms[0], ms[1], ms[2], ms[3], a);
  return cudaGetLastError();
}

}  // namespace

namespace {
// forward : out[tap][k][c] = w[k][tap][c]                       (rows k = Cout, columns c = Cin)
// dgrad   : out[tap][c][k] = w[k][8 - tap][c]  (filter rotated by 180 degrees, channel roles exchanged:
//           rows c = Cin, columns k = Cout)
__global__ void tap_major_kernel(const float* __restrict__ w, bf16* __restrict__ out, int Cin, int Cout, int dgrad) {
  const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  const long total = 9L * Cin * Cout;
  if (i >= total) return;
  if (!dgrad) {
    const int c = i % Cin; const long t = i / Cin;
    const int k = t % Cout, tap = t / Cout;
    out[i] = __float2bfloat16_rn(w[((long)k * 9 + tap) * Cin + c]);
  } else {
    const int k = i % Cout; const long t = i / Cout;
    const int c = t % Cin, tap = t / Cin;
    out[i] = __float2bfloat16_rn(w[((long)k * 9 + (8 - tap)) * Cin + c]);
  }
}
}  // namespace

cudaError_t tc_make_tap_major(const float* w, bf16* out, int Cin, int Cout, bool for_dgrad, cudaStream_t st) {
  const long total = 9L * Cin * Cout;
  tap_major_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(w, out, Cin, Cout, for_dgrad ? 1 : 0);
  return cudaGetLastError();
}

bool tc_conv3x3_halo_supported(ConvShape s) {
  return tc_conv3x3_halo_supported_unpooled(s) && s.H % PH == 0 && s.W >= 64;
}

// Without a pooled output the image height need not be a whole number of patches: the copy engine
// zero-fills the rows a last patch reads past the image and clips the rows it would store there.
bool tc_conv3x3_halo_supported_unpooled(ConvShape s) {
  return s.Cin % 64 == 0 && s.Cout % 64 == 0 && s.Cout <= 128 && s.W % PW == 0 && s.H >= PH && s.W >= 56 &&
         (long)s.N * (s.H + PH) * s.W < (1L << 31) - 256;
}

cudaError_t tc_conv3x3_halo(const bf16* in, const bf16* wt_tap_major, const float* bias, const bf16* mask, bf16* out,
                            bf16* pooled, ConvShape s, bool relu, int* dev_error, cudaStream_t st, bool pairs, uint8_t* code,
                            const uint8_t* scatter_code, bf16* scatter_out) {
  if (!out && !pooled && !scatter_out) return cudaErrorInvalidValue;
  if ((scatter_code == nullptr) != (scatter_out == nullptr) || (scatter_out && (out || pooled || mask))) return cudaErrorInvalidValue;
  if (code && !pooled) return cudaErrorInvalidValue;
  if (!(pooled ? tc_conv3x3_halo_supported(s) : tc_conv3x3_halo_supported_unpooled(s))) return cudaErrorInvalidValue;
  const int BN = s.Cout % 128 == 0 ? 128 : 64;
  // CTA pairs take two tiles at a time.  They pay with 128 output channels, where one CTA's MMAs are
  // bound by shared-memory reads; with 64 they measure the same as single CTAs, which are kept there.
  const bool pair = pairs && BN == 128 && (s.N * (s.W / PW) * ((s.H + PH - 1) / PH)) % 2 == 0;
  CUtensorMap mx, mw;
  if (!make_patch_map(&mx, in, s.N, s.H, s.W, s.Cin, IW, IH)) return cudaErrorInvalidValue;
  if (!make_filter_row_map(&mw, wt_tap_major, s.Cout, s.Cin, (uint32_t)(pair ? BN / 2 : BN))) return cudaErrorInvalidValue;
  CUtensorMap my = mw;  // only read when there is a full-resolution output
  if (out && !make_patch_map(&my, out, s.N, s.H, s.W, s.Cout, PW, PH)) return cudaErrorInvalidValue;
  CUtensorMap mm = mw;  // only read when there is a mask
  if (mask && !make_patch_map(&mm, mask, s.N, s.H, s.W, s.Cout, PW, PH)) return cudaErrorInvalidValue;
  if (mask && !out) return cudaErrorInvalidValue;
  // pool scatter: four views of the full-resolution gradient [N][2H][2W][Cout], one per window position
  CUtensorMap ms[4] = {mw, mw, mw, mw};
  if (scatter_out)
    for (int q = 0; q < 4; ++q)
      if (!make_window_map(&ms[q], scatter_out, s.N, 2 * s.H, 2 * s.W, s.Cout, q >> 1, q & 1, PW, PH)) return cudaErrorInvalidValue;
  HaloArgs a;
  a.code = code; a.scatter_code = scatter_code;
  a.N = s.N; a.H = s.H; a.W = s.W;
  a.cin_blocks = s.Cin / 64; a.Cin = s.Cin; a.Cout = s.Cout;
  a.tiles_w = s.W / PW; a.tiles_h = (s.H + PH - 1) / PH;
  a.m_tiles = s.N * a.tiles_w * a.tiles_h;
  a.n_tiles = s.Cout / BN;
  a.relu = relu ? 1 : 0; a.bias = bias; a.mask = mask; a.out = out; a.pooled = pooled; a.dev_error = dev_error;
  const int mode = scatter_out ? 2 : (code ? 1 : 0);
#define HALO_LAUNCH(MODE)                                                                      \
  (pair ? launch_halo<128, true, MODE>(mx, mw, my, mm, ms, a, st)                              \
        : (BN == 128 ? launch_halo<128, false, MODE>(mx, mw, my, mm, ms, a, st)                \
                     : launch_halo<64, false, MODE>(mx, mw, my, mm, ms, a, st)))
  return mode == 2 ? HALO_LAUNCH(2) : (mode == 1 ? HALO_LAUNCH(1) : HALO_LAUNCH(0));
#undef HALO_LAUNCH
}

}  // namespace vgg
