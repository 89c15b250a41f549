// 3x3 convolution as an implicit GEMM on CTA pairs (tcgen05 cta_group::2) for the layers with many
// output channels (56x56 images and below).
//
//   D[pixel][cout] = sum over (r, s, c) of  X[pixel shifted by (r-1, s-1)][c] * Wt[cout][r][s][c]
//
// A cluster of two CTAs computes a 256 (pixels) x BN (output channels) tile with one MMA stream:
// each CTA stages its own 128 pixels (TMA im2col, zero padding from the out-of-bounds fill) and only
// HALF of the BN x 64 filter slice per K block, and keeps its 128 accumulator rows in its own tensor
// memory.  Against one CTA per 128 x BN tile that halves the filter bytes written to and read from
// shared memory per MMA, which is what bounds the single-CTA kernel (per 128 x 256 x 16 MMA it
// reads 12 KB and the copy engine writes another 12 KB, against 128 B per cycle of shared memory).
//
// Roles per CTA: warp 0 TMA producer (one thread), warp 1 tensor-memory owner and, in the even CTA
// only, the single MMA-issuing thread; warps 2-5 epilogue (bias, ReLU / ReLU mask, bf16, swizzled
// staging tile, TMA store).  Barriers the issuer waits on (stage full, accumulator drained) live in
// the even CTA and receive the peer's signals through the cluster; barriers the issuer signals
// (stage free, accumulator full) exist in both CTAs and are reached by one multicast commit.
// Every wait has a time limit; a CTA that gives up drains its copies and MMAs, and both CTAs meet
// at a cluster barrier before either releases tensor memory or exits.
#include "tc_common.cuh"
#include "tc_kernels.cuh"

namespace vgg {
namespace {

using namespace tc;

constexpr int BM = 128;   // pixels per CTA (tensor-memory lanes); the pair's tile has 2 * BM
constexpr int BK = 64;    // channels per K block (one 128-byte swizzle row)
constexpr int A_BYTES = BM * BK * 2;
constexpr int kThreads = 192;
constexpr int kSmemLimit = 227 * 1024;

// MASK: the kernel applies a ReLU mask and keeps a mask tile in shared memory (one stage fewer).
template <int BN, bool MASK>
struct PairTile {
  static constexpr int B_BYTES = (BN / 2) * BK * 2;  // this CTA's half of the filter slice
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int OUT_BYTES = BM * 64 * 2;      // staging tile of the TMA store
  static constexpr int TILES = MASK ? 2 : 1;         // staging tile, mask tile
  // beside the dynamic shared memory: alignment slack and barriers (1280 B) and the static part, which is the
  // 2 KB bias table unless MASK (an input gradient has no bias)
  static constexpr int kOther = MASK ? 1792 : 4608;
  static constexpr int STAGES = (kSmemLimit - kOther - TILES * OUT_BYTES) / STAGE_BYTES > 8 ? 8 : (kSmemLimit - kOther - TILES * OUT_BYTES) / STAGE_BYTES;
  static constexpr int TMEM_COLS = 2 * BN;           // double-buffered accumulator
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + TILES * OUT_BYTES + 1024 + 256;
};

struct PairArgs {
  int pixels;      // N*H*W
  int H, W;
  int cin_blocks;  // Cin / 64
  int Cout;
  int m_pairs;     // ceil(pixels / 256)
  int n_tiles;     // Cout / BN
  int relu;
  const float* bias;
  const bf16* mask;
  // Forward-only passes of a block-ending layer: the full-resolution output is not kept; every value
  // goes straight into the 2x2 max-pooled tensor [N][H/2][W/2][Cout] (zeroed beforehand) with a
  // vector max-reduction on global memory.  A window's four pixels may sit in different tiles and
  // CTAs: the reduction needs no meeting point, and a maximum does not depend on the order.
  bf16* pooled;
  int* dev_error;
  // Tail split.  The first main_tiles tiles are whole rounds of the resident pairs; the rest (fewer
  // than half a round) are each cut into tail_splits ranges of tail_kb K blocks so that the last
  // round keeps every pair busy for a fraction of a tile's time.  Those work items leave raw fp32
  // sums in `partial` ([split][tail_rows][Cout], rows counted from pixel tail_row0) for
  // pair_tail_finish_kernel.  main_tiles = all tiles when there is no tail.
  int main_tiles, tail_splits, tail_kb;
  int tail_row0, tail_rows;
  float* partial;
};

// One unit of a pair's work: a whole tile (split < 0) or a range of a tail tile's K blocks.
struct Work {
  int tile, kb0, kb1, split;
};
__device__ __forceinline__ Work get_work(int w, const PairArgs& a, int k_blocks) {
  if (w < a.main_tiles) return Work{w, 0, k_blocks, -1};
  const int j = w - a.main_tiles;
  const int t = j / a.tail_splits, z = j - t * a.tail_splits;
  const int kb0 = z * a.tail_kb;
  return Work{a.main_tiles + t, kb0, min(k_blocks, kb0 + a.tail_kb), z};
}

// pooled[row][0..7] = max(pooled[row][0..7], v): eight bf16 in one reduction (ReLU outputs: the tensor starts at zero)
__device__ __forceinline__ void red_max_bf16x8(bf16* dst, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("red.global.max.noftz.v4.bf16x2 [%0], {%1, %2, %3, %4};" ::"l"(dst), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

template <int BN, bool POOL, bool MASK>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
conv3x3_pair_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                       const __grid_constant__ CUtensorMap map_y, const __grid_constant__ CUtensorMap map_m, PairArgs a) {
  using T = PairTile<BN, MASK>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t out_smem = smem_base + T::STAGES * T::STAGE_BYTES;
  const uint32_t mask_smem = out_smem + T::OUT_BYTES;  // ReLU-mask tile of the chunk being finished (input gradient)
  const uint32_t bars = mask_smem + (MASK ? T::OUT_BYTES : 0);
  auto full_bar = [&](int s) { return bars + 8u * s; };                       // used in the even CTA
  auto empty_bar = [&](int s) { return bars + 8u * (T::STAGES + s); };        // both CTAs
  auto acc_full_bar = [&](int b) { return bars + 8u * (2 * T::STAGES + b); };       // both CTAs
  auto acc_empty_bar = [&](int b) { return bars + 8u * (2 * T::STAGES + 2 + b); };  // used in the even CTA
  const uint32_t drain_bar = bars + 8u * (2 * T::STAGES + 4);
  const uint32_t mask_bar = bars + 8u * (2 * T::STAGES + 5);  // this CTA's own
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  __shared__ __align__(16) float bias_s[MASK ? 4 : 512];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int k_blocks = 9 * a.cin_blocks;
  const int total_work = a.main_tiles + (a.m_pairs * a.n_tiles - a.main_tiles) * a.tail_splits;

  if (!MASK)
    for (int i = threadIdx.x; i < a.Cout; i += kThreads) bias_s[i] = a.bias ? a.bias[i] : 0.f;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < T::STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(acc_full_bar(b), 1); mbar_init(acc_empty_bar(b), 2); }
    mbar_init(drain_bar, 1);
    mbar_init(mask_bar, 1);
    mbar_fence_init();
    tma_prefetch_desc(&map_x);
    tma_prefetch_desc(&map_w);
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(&tmem_base_slot), T::TMEM_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers are initialised before anything signals them
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
      for (int w = pair; w < total_work && ok; w += n_pairs) {
        const Work wk = get_work(w, a, k_blocks);
        const int m_pair = wk.tile / a.n_tiles, n_tile = wk.tile - m_pair * a.n_tiles;
        // a CTA whose 128 pixels all lie past the end of the tensor (odd tile count) stages the
        // tensor's first pixels instead: its accumulator rows are never stored
        int p0 = (2 * m_pair + (int)rank) * BM;
        if (p0 >= a.pixels) p0 = 0;
        const int w0 = p0 % a.W, t = p0 / a.W;
        const int h0 = t % a.H, n0 = t / a.H;
        const int filter_row = n_tile * BN + (int)rank * (BN / 2);
        // K block kb = (tap (r, s), channel block cb), channel blocks fastest
        const int tap0 = wk.kb0 / a.cin_blocks;
        int cb = wk.kb0 - tap0 * a.cin_blocks, r = tap0 / 3, s = tap0 - 3 * (tap0 / 3);
        for (int kb = wk.kb0; kb < wk.kb1; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1, &abort_flag, a.dev_error, kDevTimeoutStageFree)) { ok = false; break; }
          const uint32_t sa = smem_base + stage * T::STAGE_BYTES, sb = sa + A_BYTES;
          const uint32_t full = map_to_cta(full_bar(stage), 0);
          // the even CTA announces the bytes of both CTAs' copies for this stage
          if (leader) mbar_expect_tx(full_bar(stage), 2 * T::STAGE_BYTES);
          tma_load_im2col_4d_pair(sa, &map_x, full, cb * BK, w0 - 1, h0 - 1, n0, (uint16_t)s, (uint16_t)r);
          tma_load_2d_pair(sb, &map_w, full, kb * BK, filter_row);
          ++fills[stage];
          if (++stage == T::STAGES) { stage = 0; phase ^= 1; }
          if (++cb == a.cin_blocks) { cb = 0; if (++s == 3) { s = 0; ++r; } }
        }
      }
      if (!ok) {
        // let every copy already in flight land before the CTA may go on to exit: the even CTA sees
        // them on its stage barriers, the peer (whose copies report there too) allows them a millisecond
        if (leader) {
          for (int s = 0; s < T::STAGES; ++s)
            if (fills[s]) {
              const unsigned long long t0 = global_timer_ns();
              while (!mbar_try_wait(full_bar(s), (fills[s] - 1) & 1) && global_timer_ns() - t0 < 100000000ull) {}
            }
        } else {
          const unsigned long long t0 = global_timer_ns();
          while (global_timer_ns() - t0 < 1000000ull) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------- MMA issuer (even CTA only) -------------------------
    if (lane == 0 && leader) {
      constexpr uint32_t idesc = umma_idesc_bf16(2 * BM, BN, 0, 0);
      int stage = 0;
      uint32_t phase = 0;
      int local = 0;
      bool ok = true;
      for (int w = pair; w < total_work && ok; w += n_pairs, ++local) {
        const Work wk = get_work(w, a, k_blocks);
        const int buf = local & 1;
        const uint32_t use = (uint32_t)(local >> 1);
        if (!mbar_wait(acc_empty_bar(buf), (use & 1) ^ 1, &abort_flag, a.dev_error, kDevTimeoutTmemFree)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * BN);
        for (int kb = wk.kb0; kb < wk.kb1; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, &abort_flag, a.dev_error, kDevTimeoutTmaFull)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_base + stage * T::STAGE_BYTES, sb = sa + A_BYTES;
          const uint64_t da = smem_desc_sw128(sa, 16), db = smem_desc_sw128(sb, 16);
          umma_bf16_pair(d_tmem, da, db, idesc, kb != wk.kb0 ? 1u : 0u);
#pragma unroll
          for (int k = 1; k < BK / 16; ++k)
            umma_bf16_pair_acc(d_tmem, desc_advance(da, k * 32), desc_advance(db, k * 32), idesc);
          umma_commit_pair(empty_bar(stage), 3);  // frees the stage in both CTAs
          if (++stage == T::STAGES) { stage = 0; phase ^= 1; }
        }
        if (ok) umma_commit_pair(acc_full_bar(buf), 3);
      }
      if (!ok) {
        umma_commit_pair(drain_bar, 1);  // arrives in this CTA only, once the pair's MMAs are done
        const unsigned long long t0 = global_timer_ns();
        while (!mbar_try_wait(drain_bar, 0) && global_timer_ns() - t0 < 100000000ull) {}
      }
    }
  } else {
    // -------------------------------- epilogue --------------------------------
    const int quarter = warp & 3;  // the tensor-memory lane quarter this warp may read
    const int row = quarter * 32 + lane;
    int local = 0;
    const bool issuer = threadIdx.x == 64;  // owns the TMA store groups
    uint8_t* stage_row = smem_raw + (out_smem - smem_u32(smem_raw)) + row * 128;
    const uint8_t* mask_srow = smem_raw + (mask_smem - smem_u32(smem_raw)) + row * 128;
    // Input gradient: the ReLU mask (the stored output of the layer below at the same pixels and
    // channels) of a 128 x 64 chunk arrives by TMA in the staging tile's layout.  The issuer requests
    // the NEXT chunk's tile as soon as every thread has read the current one, so the copy's latency
    // hides behind the rest of the epilogue and the wait for the next accumulator.
    uint32_t mask_phase = 0;
    bool mask_pending = false;  // issuer only: a mask copy is in flight or unread
    // first chunk (work item, 64-column block) at or after (w, c64) whose epilogue applies a mask here
    auto request_mask = [&](int w, int c64) {
      for (; w < total_work; w += n_pairs, c64 = 0) {
        const Work wk = get_work(w, a, k_blocks);
        if (wk.split >= 0) return;  // tail items (all that follow, too) are masked by the finishing kernel
        const int mp = wk.tile / a.n_tiles, nt = wk.tile - mp * a.n_tiles;
        const int mt = 2 * mp + (int)rank;
        if ((long)mt * BM >= a.pixels) continue;
        mbar_expect_tx(mask_bar, T::OUT_BYTES);
        tma_load_2d(mask_smem, &map_m, mask_bar, nt * BN + c64, mt * BM);  // rows past the end read as zero
        mask_pending = true;
        return;
      }
    };
    if (MASK && issuer) request_mask(pair, 0);
    for (int w = pair; w < total_work; w += n_pairs, ++local) {
      const Work wk = get_work(w, a, k_blocks);
      const int buf = local & 1;
      const uint32_t use = (uint32_t)(local >> 1);
      const int m_pair = wk.tile / a.n_tiles, n_tile = wk.tile - m_pair * a.n_tiles;
      const int m_tile = 2 * m_pair + (int)rank;
      const bool got = mbar_wait(acc_full_bar(buf), use & 1, &abort_flag, a.dev_error, kDevTimeoutAccum);
      if (named_bar_or(1, 128, !got)) break;  // all four warps leave together
      tc_fence_after();
      const long pixel = (long)m_tile * BM + row;
      const bool valid = pixel < a.pixels;
      const bool tile_valid = (long)m_tile * BM < a.pixels;
      const int c_base = n_tile * BN;
      bf16* pool_row = nullptr;
      if (POOL && valid) {
        const int pw = (int)(pixel % a.W), t = (int)(pixel / a.W);
        const int ph = t % a.H, pn = t / a.H;
        pool_row = a.pooled + (((long)pn * (a.H / 2) + ph / 2) * (a.W / 2) + pw / 2) * a.Cout + c_base;
      }
      if (wk.split >= 0) {
        // part of a tail tile's K range: raw sums, one row per thread, for the finishing kernel
        float* dst = a.partial + ((size_t)wk.split * a.tail_rows + (size_t)(pixel - a.tail_row0)) * a.Cout + c_base;
#pragma unroll 1
        for (int cc = 0; cc < BN && tile_valid; cc += 32) {
          uint32_t v[32];
          tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN + cc), v);
          tmem_ld_wait();
          if (valid) {
#pragma unroll
            for (int j = 0; j < 32; j += 4)
              *reinterpret_cast<float4*>(dst + cc + j) = make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]),
                                                                     __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
          }
        }
        tc_fence_before();
        named_bar_sync(1, 128);
        if (issuer) mbar_arrive_cluster(map_to_cta(acc_empty_bar(buf), 0));
        continue;
      }
#pragma unroll 1
      for (int c64 = 0; c64 < BN && tile_valid; c64 += 64) {
        if (!POOL) {
          if (issuer) tma_store_wait_read<0>();  // the previous store has read the staging tile
          named_bar_sync(1, 128);
        }
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
            if (!MASK) { x0 += bias_s[c_base + cc + j]; x1 += bias_s[c_base + cc + j + 1]; }
            if (a.relu) { x0 = fmaxf(x0, 0.f); x1 = fmaxf(x1, 0.f); }
            __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
            packed[j >> 1] = *reinterpret_cast<uint32_t*>(&h);
          }
          if (POOL) {
            if (pool_row) {
#pragma unroll
              for (int q = 0; q < 4; ++q)
                red_max_bf16x8(pool_row + cc + 8 * q, packed[q * 4], packed[q * 4 + 1], packed[q * 4 + 2], packed[q * 4 + 3]);
            }
            continue;
          }
          if (MASK) {
            if (!mask_ready) {  // a failed wait leaves the chunk unmasked; the error word says so
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
        if (POOL) continue;
        fence_async_smem();
        named_bar_sync(1, 128);  // the staging tile is complete, and everyone has read the mask tile
        if (issuer) {
          // rows past the end of the tensor (last tile) are clipped by the copy engine
          tma_store_2d(&map_y, out_smem, c_base + c64, m_tile * BM);
          tma_store_commit();
          if (MASK) {
            mask_pending = false;
            if (c64 + 64 < BN) request_mask(w, c64 + 64); else request_mask(w + n_pairs, 0);
          }
        }
      }
      tc_fence_before();
      named_bar_sync(1, 128);
      if (issuer) mbar_arrive_cluster(map_to_cta(acc_empty_bar(buf), 0));  // one arrival per CTA of the pair
    }
    if (issuer && mask_pending) {
      // left early (a wait ran out) with a mask copy in flight: let it land before shared memory goes away
      const unsigned long long t0 = global_timer_ns();
      while (!mbar_try_wait(mask_bar, mask_phase) && global_timer_ns() - t0 < 100000000ull) {}
    }
    if (issuer) tma_store_wait_all();  // shared memory must outlive the stores that read it
  }

  // Neither CTA may release tensor memory or exit while the other can still signal its barriers,
  // read its shared memory or write its accumulator.
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, T::TMEM_COLS);
  }
}

// out[row][c] = epilogue(sum over splits of partial[split][row][c]) for the rows of the tail tiles
// (out, mask already point at the first tail row); eight channels per thread, splits added in order.
__global__ void pair_tail_finish_kernel(const float* __restrict__ partial, int splits, long elems, int Cout,
                                        const float* __restrict__ bias, int relu, const bf16* __restrict__ mask,
                                        bf16* __restrict__ out, bf16* __restrict__ pooled, long row0, int H, int W) {
  const long i = ((long)blockIdx.x * blockDim.x + threadIdx.x) * 8;
  if (i >= elems) return;
  float x[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  for (int z = 0; z < splits; ++z) {
    const float4 p0 = *reinterpret_cast<const float4*>(partial + (long)z * elems + i);
    const float4 p1 = *reinterpret_cast<const float4*>(partial + (long)z * elems + i + 4);
    x[0] += p0.x; x[1] += p0.y; x[2] += p0.z; x[3] += p0.w;
    x[4] += p1.x; x[5] += p1.y; x[6] += p1.z; x[7] += p1.w;
  }
  const int c = (int)(i % Cout);
  uint32_t packed[4];
#pragma unroll
  for (int e = 0; e < 8; e += 2) {
    float x0 = x[e], x1 = x[e + 1];
    if (bias) { x0 += bias[c + e]; x1 += bias[c + e + 1]; }
    if (relu) { x0 = fmaxf(x0, 0.f); x1 = fmaxf(x1, 0.f); }
    __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
    packed[e >> 1] = *reinterpret_cast<uint32_t*>(&h);
  }
  if (mask) {
    const uint4 m = *reinterpret_cast<const uint4*>(mask + i);
    const uint32_t mw[4] = {m.x, m.y, m.z, m.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const uint32_t lo = mw[e] & 0xFFFFu, hi = mw[e] >> 16;
      uint32_t keep = 0;
      if (lo != 0 && !(lo & 0x8000u)) keep |= 0x0000FFFFu;
      if (hi != 0 && !(hi & 0x8000u)) keep |= 0xFFFF0000u;
      packed[e] &= keep;
    }
  }
  if (pooled) {
    // forward-only pass of a block-ending layer: straight into the pooled tensor (see PairArgs::pooled)
    const long pixel = row0 + i / Cout;
    const int pw = (int)(pixel % W), t = (int)(pixel / W);
    const int ph = t % H, pn = t / H;
    red_max_bf16x8(pooled + (((long)pn * (H / 2) + ph / 2) * (W / 2) + pw / 2) * Cout + c, packed[0], packed[1], packed[2],
                   packed[3]);
    return;
  }
  *reinterpret_cast<uint4*>(out + i) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
}

// CTA pairs of this kernel that can be resident at once (one pair per two SMs at most)
template <int BN, bool POOL, bool MASK>
cudaError_t resident_pairs(int* out) {
  using T = PairTile<BN, MASK>;
  static int max_pairs = 0;
  if (!max_pairs) {
    cudaError_t e = cudaFuncSetAttribute(conv3x3_pair_tc_kernel<BN, POOL, MASK>, cudaFuncAttributeMaxDynamicSharedMemorySize, T::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(sms & ~1));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = T::SMEM_BYTES;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
    cfg.attrs = &attr; cfg.numAttrs = 1;
    int n = 0;
    e = cudaOccupancyMaxActiveClusters(&n, conv3x3_pair_tc_kernel<BN, POOL, MASK>, &cfg);
    if (e != cudaSuccess || n < 1) { cudaGetLastError(); n = sms / 2; }
    max_pairs = n < sms / 2 ? n : sms / 2;
    if (max_pairs < 1) max_pairs = 1;
  }
  *out = max_pairs;
  return cudaSuccess;
}

constexpr int kTailMaxPairs = 128;  // bound used to size the tail scratch (SMs / 2 on any device this runs on)

}  // namespace

bool tc_conv3x3_pair_supported(ConvShape s) {
  return s.Cin % 64 == 0 && s.Cout % 256 == 0 && s.Cout <= 512 && s.H >= 2 && s.W >= 2 && s.N >= 1 &&
         (long)s.N * s.H * s.W < (1L << 31) - 512;
}

size_t tc_conv3x3_pair_scratch_elems(ConvShape s) {
  // at most one work item per resident pair, each 256 rows x 256 columns of fp32
  return tc_conv3x3_pair_supported(s) ? (size_t)kTailMaxPairs * 2 * BM * 256 : 0;
}

cudaError_t tc_conv3x3_pair(const bf16* in, const bf16* wt, const float* bias, const bf16* mask, bf16* out, ConvShape s,
                            bool relu, int* dev_error, cudaStream_t st, float* partial, int* launches, bf16* pooled) {
  if (launches) *launches = 0;
  if (!tc_conv3x3_pair_supported(s)) return cudaErrorInvalidValue;
  if (pooled && (mask || !relu || (s.H & 1) || (s.W & 1))) return cudaErrorInvalidValue;  // maxima of ReLU outputs only
  if (mask && bias) return cudaErrorInvalidValue;  // a masked result is an input gradient: no bias
  if (!pooled && !out) return cudaErrorInvalidValue;
  constexpr int BN = 256;
  CUtensorMap mx, mw, my, mm;
  if (!make_im2col_map(&mx, in, s.N, s.H, s.W, s.Cin, BM)) return cudaErrorInvalidValue;
  if (!make_tiled_map_2d(&mw, wt, (uint64_t)s.Cout, (uint64_t)9 * s.Cin, BN / 2)) return cudaErrorInvalidValue;
  my = mw;  // only read when there is a full-resolution output
  if (!pooled && !make_tiled_map_2d(&my, out, (uint64_t)s.N * s.H * s.W, (uint64_t)s.Cout, BM)) return cudaErrorInvalidValue;
  mm = my;  // only read when there is a mask
  if (mask && !make_tiled_map_2d(&mm, mask, (uint64_t)s.N * s.H * s.W, (uint64_t)s.Cout, BM)) return cudaErrorInvalidValue;
  PairArgs a;
  a.pixels = s.N * s.H * s.W;
  a.H = s.H; a.W = s.W;
  a.cin_blocks = s.Cin / 64;
  a.Cout = s.Cout;
  a.m_pairs = (a.pixels + 2 * BM - 1) / (2 * BM);
  a.n_tiles = s.Cout / BN;
  a.relu = relu ? 1 : 0;
  a.bias = bias; a.mask = mask; a.dev_error = dev_error; a.pooled = pooled;
  int cap = 0;
  cudaError_t e = pooled ? resident_pairs<BN, true, false>(&cap)
                         : (mask ? resident_pairs<BN, false, true>(&cap) : resident_pairs<BN, false, false>(&cap));
  if (e != cudaSuccess) return e;
  if (pooled) {
    e = cudaMemsetAsync(pooled, 0, (size_t)s.N * (s.H / 2) * (s.W / 2) * s.Cout * sizeof(bf16), st);
    if (e != cudaSuccess) return e;
  }
  const int tiles = a.m_pairs * a.n_tiles, k_blocks = 9 * a.cin_blocks;
  a.main_tiles = tiles; a.tail_splits = 1; a.tail_kb = k_blocks; a.tail_row0 = 0; a.tail_rows = 0; a.partial = nullptr;
  // Whole rounds of `cap` tiles, then a tail of fewer than half a round: cut each tail tile's K range
  // so that the last round occupies (nearly) every pair for 1/splits of a tile's time.
  const int rounds = tiles / cap, left = tiles - rounds * cap;
  if (partial && rounds >= 1 && left > 0 && 2 * left <= cap && cap <= kTailMaxPairs && (rounds * cap) % a.n_tiles == 0) {
    int splits = cap / left;
    if (splits > k_blocks) splits = k_blocks;
    const int per = (k_blocks + splits - 1) / splits;
    splits = (k_blocks + per - 1) / per;
    // The pieces cost a second kernel and a round trip of fp32 partial sums (about the time of 50 K
    // blocks at batch 100): only worth it when the shortened round saves more than that.
    if (splits >= 2 && k_blocks - per >= 56) {
      a.main_tiles = rounds * cap;
      a.tail_splits = splits; a.tail_kb = per;
      a.tail_row0 = (a.main_tiles / a.n_tiles) * 2 * BM;
      a.tail_rows = a.pixels - a.tail_row0;
      a.partial = partial;
    }
  }
  const int work = a.main_tiles + (tiles - a.main_tiles) * a.tail_splits;
  const int pairs = work < cap ? work : cap;
  if (pooled) conv3x3_pair_tc_kernel<BN, true, false><<<2 * pairs, kThreads, PairTile<BN, false>::SMEM_BYTES, st>>>(mx, mw, my, mm, a);
  else if (mask) conv3x3_pair_tc_kernel<BN, false, true><<<2 * pairs, kThreads, PairTile<BN, true>::SMEM_BYTES, st>>>(mx, mw, my, mm, a);
  else conv3x3_pair_tc_kernel<BN, false, false><<<2 * pairs, kThreads, PairTile<BN, false>::SMEM_BYTES, st>>>(mx, mw, my, mm, a);
  e = cudaGetLastError();
  if (launches) *launches = 1;
  if (e != cudaSuccess || !a.partial) return e;
  const long elems = (long)a.tail_rows * a.Cout;
  const size_t row_off = (size_t)a.tail_row0 * a.Cout;
  pair_tail_finish_kernel<<<(unsigned)((elems / 8 + 255) / 256), 256, 0, st>>>(
      partial, a.tail_splits, elems, a.Cout, bias, a.relu, mask ? mask + row_off : nullptr, pooled ? nullptr : out + row_off,
      pooled, (long)a.tail_row0, s.H, s.W);
  if (launches) *launches = 2;
  return cudaGetLastError();
}

}  // namespace vgg
