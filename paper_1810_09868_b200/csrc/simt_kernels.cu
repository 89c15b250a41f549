// CUDA-core (SIMT) kernels of the VGG19 pass.  They carry the fp32
// configuration end to end (fp32 FMA, no tensor cores) and serve every layer
// shape the tensor-core kernels do not take (3 input channels, tiny images).
//
// One tiled GEMM main loop (64x64 tile, 16-deep K slices, 4x4 outputs per
// thread, fp32 accumulation) is shared by convolution (implicit GEMM over
// M = N*H*W pixels, K = 9*Cin), its filter gradient (M = Cout, N = 9*Cin,
// K = pixels, split over K with a second reduction pass), and the dense
// layers.  What differs is how an operand element is fetched ("loader") and
// what happens to the finished tile ("epilogue").
#include "common.cuh"

#include <type_traits>

namespace vgg {

namespace {

constexpr int TM = 64, TN = 64, TK = 16, THREADS = 256;

// ---- operand loaders: element (row i of the operand, reduction index k) ----

template <typename T>
struct RowMajorLoad {  // op[i][k], k contiguous
  const T* p; long ld;
  static constexpr bool kContigK = true;
  __device__ float operator()(int i, int k) const { return to_f32(p[(long)i * ld + k]); }
};

template <typename T>
struct ColMajorLoad {  // op[k][i], i contiguous
  const T* p; long ld;
  static constexpr bool kContigK = false;
  __device__ float operator()(int i, int k) const { return to_f32(p[(long)k * ld + i]); }
};

template <typename T>
struct ConvPatchLoad {  // i = pixel (n,h,w), k = (r*3+s)*C + c  ->  x[n][h+r-1][w+s-1][c] or 0
  const T* p; int H, W, C;
  static constexpr bool kContigK = true;
  __device__ float operator()(int i, int k) const {
    int rs = k / C, c = k - rs * C;
    int r = rs / 3, s = rs - r * 3;
    int w = i % W, t = i / W;
    int h = t % H, n = t / H;
    int hh = h + r - 1, ww = w + s - 1;
    if ((unsigned)hh >= (unsigned)H || (unsigned)ww >= (unsigned)W) return 0.f;
    return to_f32(p[(((long)n * H + hh) * W + ww) * C + c]);
  }
};

template <typename T>
struct ShiftedPixelLoad {  // i = (r*3+s)*C + c, k = pixel  ->  x[pixel shifted by (r-1,s-1)][c] or 0
  const T* p; int H, W, C;
  static constexpr bool kContigK = false;
  __device__ float operator()(int i, int k) const {
    int rs = i / C, c = i - rs * C;
    int r = rs / 3, s = rs - r * 3;
    int w = k % W, t = k / W;
    int h = t % H, n = t / H;
    int hh = h + r - 1, ww = w + s - 1;
    if ((unsigned)hh >= (unsigned)H || (unsigned)ww >= (unsigned)W) return 0.f;
    return to_f32(p[(((long)n * H + hh) * W + ww) * C + c]);
  }
};

// ---- epilogues -------------------------------------------------------------

template <typename T>
struct StoreEpilogue {  // + bias[n], ReLU, * (mask > 0); store T and/or fp32, row-major ldc
  const float* bias; const T* mask; T* out_t; float* out_f; long ldc; int relu;
  __device__ void operator()(int m, int n, float v, int /*split*/) const {
    if (bias) v += bias[n];
    if (relu) v = fmaxf(v, 0.f);
    long o = (long)m * ldc + n;
    if (mask && !(to_f32(mask[o]) > 0.f)) v = 0.f;
    if (out_t) out_t[o] = from_f32<T>(v);
    if (out_f) out_f[o] = v;
  }
};

struct PartialEpilogue {  // raw fp32 partial sums, one [M][N] slab per K split
  float* partial; long slab; long ldc;
  __device__ void operator()(int m, int n, float v, int split) const {
    partial[(long)split * slab + (long)m * ldc + n] = v;
  }
};

template <class ALoad, class BLoad, class Epi>
__global__ void __launch_bounds__(THREADS)
gemm_simt_kernel(ALoad a, BLoad b, Epi epi, int M, int N, int K, int k_per_split) {
  __shared__ float As[TK][TM + 4];
  __shared__ float Bs[TK][TN + 4];
  const int t = threadIdx.x;
  const int m0 = blockIdx.x * TM, n0 = blockIdx.y * TN;  // M tiles on x: up to 2^31-1 of them
  const int k_begin = blockIdx.z * k_per_split;
  const int k_end = min(K, k_begin + k_per_split);
  const int ty = t / 16, tx = t % 16;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int k0 = k_begin; k0 < k_end; k0 += TK) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int kk, mm;
      if (ALoad::kContigK) { kk = t % TK; mm = t / TK + i * (THREADS / TK); }
      else { mm = t % TM; kk = t / TM + i * (THREADS / TM); }
      int gm = m0 + mm, gk = k0 + kk;
      As[kk][mm] = (gm < M && gk < k_end) ? a(gm, gk) : 0.f;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int kk, nn;
      if (BLoad::kContigK) { kk = t % TK; nn = t / TK + i * (THREADS / TK); }
      else { nn = t % TN; kk = t / TN + i * (THREADS / TN); }
      int gn = n0 + nn, gk = k0 + kk;
      Bs[kk][nn] = (gn < N && gk < k_end) ? b(gn, gk) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      float av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) av[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) bv[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int gm = m0 + ty * 4 + i, gn = n0 + tx * 4 + j;
      if (gm < M && gn < N) epi(gm, gn, acc[i][j], blockIdx.z);
    }
}

template <class ALoad, class BLoad, class Epi>
cudaError_t launch_gemm(ALoad a, BLoad b, Epi e, int M, int N, int K, int splits, cudaStream_t st) {
  int k_per_split = ((K + splits - 1) / splits + TK - 1) / TK * TK;
  dim3 grid((M + TM - 1) / TM, (N + TN - 1) / TN, splits);
  gemm_simt_kernel<<<grid, THREADS, 0, st>>>(a, b, e, M, N, K, k_per_split);
  return cudaGetLastError();
}

// out[i] = sum over splits of partial[split][i], in split order (deterministic)
__global__ void reduce_splits_kernel(const float* partial, float* out, long n, int splits) {
  long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float s = 0.f;
  for (int z = 0; z < splits; ++z) s += partial[(long)z * n + i];
  out[i] = s;
}

// out[c] = sum over chunks of partial[chunk][c]: eight threads per column add interleaved
// chunks, then the eight sums are added in a fixed order
__global__ void reduce_columns_kernel(const float* __restrict__ partial, float* __restrict__ out, int C, int chunks) {
  __shared__ float sm[8][33];
  const int c = blockIdx.x * 32 + threadIdx.x;
  float s = 0.f;
  if (c < C)
    for (int z = threadIdx.y; z < chunks; z += 8) s += partial[(long)z * C + c];
  sm[threadIdx.y][threadIdx.x] = s;
  __syncthreads();
  if (threadIdx.y == 0 && c < C) {
    float tot = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) tot += sm[i][threadIdx.x];
    out[c] = tot;
  }
}

// partial[chunk][c] = sum of dz[p][c] over the chunk's pixels
template <typename T>
__global__ void colsum_partial_kernel(const T* dz, float* partial, long P, int C, long p_per_chunk) {
  int c = blockIdx.x * 32 + threadIdx.x;
  long p0 = (long)blockIdx.y * p_per_chunk, p1 = min(P, p0 + p_per_chunk);
  __shared__ float sm[8][33];
  float s = 0.f;
  if (c < C)
    for (long p = p0 + threadIdx.y; p < p1; p += 8) s += to_f32(dz[p * C + c]);
  sm[threadIdx.y][threadIdx.x] = s;
  __syncthreads();
  if (threadIdx.y == 0 && c < C) {
    float tot = 0.f;
    for (int i = 0; i < 8; ++i) tot += sm[i][threadIdx.x];
    partial[(long)blockIdx.y * C + c] = tot;
  }
}

int wgrad_splits(ConvShape s) {
  long P = (long)s.N * s.H * s.W;
  int tiles = ((s.Cout + TM - 1) / TM) * ((9 * s.Cin + TN - 1) / TN);
  long splits = (148 * 4 + tiles - 1) / tiles;
  long max_by_k = (P + 255) / 256;
  if (splits > max_by_k) splits = max_by_k;
  if (splits < 1) splits = 1;
  return (int)splits;
}

int colsum_chunks(long P) {
  long c = (P + 1023) / 1024;
  return (int)(c > 256 ? 256 : (c < 1 ? 1 : c));
}

}  // namespace

template <typename T>
cudaError_t simt_conv3x3(const T* in, const T* wt, const float* bias, const T* mask, T* out,
                         ConvShape s, bool relu, cudaStream_t st) {
  ConvPatchLoad<T> a{in, s.H, s.W, s.Cin};
  RowMajorLoad<T> b{wt, 9L * s.Cin};
  StoreEpilogue<T> e{bias, mask, out, nullptr, (long)s.Cout, relu ? 1 : 0};
  return launch_gemm(a, b, e, s.N * s.H * s.W, s.Cout, 9 * s.Cin, 1, st);
}

size_t simt_wgrad_scratch_elems(ConvShape s) {
  size_t a = (size_t)wgrad_splits(s) * s.Cout * 9 * s.Cin;
  size_t b = (size_t)colsum_chunks((long)s.N * s.H * s.W) * s.Cout;
  return a > b ? a : b;
}

template <typename T>
cudaError_t simt_conv3x3_wgrad(const T* x, const T* dz, float* dW, float* db, float* partial,
                               ConvShape s, cudaStream_t st) {
  const long P = (long)s.N * s.H * s.W;
  const int J = 9 * s.Cin;
  if (db) {
    int chunks = colsum_chunks(P);
    long per = (P + chunks - 1) / chunks;
    dim3 grid((s.Cout + 31) / 32, chunks), block(32, 8);
    colsum_partial_kernel<T><<<grid, block, 0, st>>>(dz, partial, P, s.Cout, per);
    reduce_splits_kernel<<<(s.Cout + 255) / 256, 256, 0, st>>>(partial, db, s.Cout, chunks);
  }
  int splits = wgrad_splits(s);
  ColMajorLoad<T> a{dz, (long)s.Cout};
  ShiftedPixelLoad<T> b{x, s.H, s.W, s.Cin};
  long n_out = (long)s.Cout * J;
  if (splits == 1) {
    StoreEpilogue<float> e{nullptr, nullptr, nullptr, dW, (long)J, 0};
    return launch_gemm(a, b, e, s.Cout, J, (int)P, 1, st);
  }
  PartialEpilogue e{partial, n_out, (long)J};
  cudaError_t err = launch_gemm(a, b, e, s.Cout, J, (int)P, splits, st);
  if (err != cudaSuccess) return err;
  reduce_splits_kernel<<<(unsigned)((n_out + 255) / 256), 256, 0, st>>>(partial, dW, n_out, splits);
  return cudaGetLastError();
}


// ---- bf16 fast paths: eight channels (16 bytes) per thread -------------------

union Pack8 {
  uint4 u;
  __nv_bfloat162 h2[4];
  bf16 h[8];
};

__global__ void maxpool_fwd_bf16x8_kernel(const bf16* __restrict__ x, bf16* __restrict__ y, uint8_t* __restrict__ code,
                                          long total8, int H, int W, int C8) {
  long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total8) return;
  int Wo = W / 2, Ho = H / 2;
  int c8 = i % C8; long t = i / C8;
  int j = t % Wo; t /= Wo;
  int ii = t % Ho; long n = t / Ho;
  const uint4* p = reinterpret_cast<const uint4*>(x) + ((n * H + 2 * ii) * W + 2 * j) * C8 + c8;
  Pack8 a, b, c, d, r;
  a.u = __ldg(p); b.u = __ldg(p + C8); c.u = __ldg(p + (long)W * C8); d.u = __ldg(p + (long)W * C8 + C8);
#pragma unroll
  for (int e = 0; e < 4; ++e) r.h2[e] = __hmax2(__hmax2(a.h2[e], b.h2[e]), __hmax2(c.h2[e], d.h2[e]));
  reinterpret_cast<uint4*>(y)[i] = r.u;
  if (code) {
    // where the window's maximum sits (first one in the order (0,0), (0,1), (1,0), (1,1)), or 4 when
    // it is not positive: all the backward pass needs to know about this window
    uint32_t w[2] = {0u, 0u};
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const float v[4] = {__bfloat162float(a.h[e]), __bfloat162float(b.h[e]), __bfloat162float(c.h[e]),
                          __bfloat162float(d.h[e])};
      float m = v[0];
      uint32_t best = 0;
#pragma unroll
      for (int q = 1; q < 4; ++q)
        if (v[q] > m) { m = v[q]; best = q; }
      if (!(m > 0.f)) best = 4;
      w[e >> 2] |= best << (8 * (e & 3));
    }
    reinterpret_cast<uint2*>(code)[i] = make_uint2(w[0], w[1]);
  }
}

// dy[window position q] = dp[window] where q is the stored arg-max code, else 0 (code 4: nowhere)
__global__ void pool_scatter_bf16x8_kernel(const uint8_t* __restrict__ code, const bf16* __restrict__ dp,
                                           bf16* __restrict__ dy, long total8, int H, int W, int C8) {
  long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total8) return;
  int Wo = W / 2, Ho = H / 2;
  int c8 = i % C8; long t = i / C8;
  int j = t % Wo; t /= Wo;
  int ii = t % Ho; long n = t / Ho;
  const long base = ((n * H + 2 * ii) * W + 2 * j) * C8 + c8;
  const long off[4] = {0, (long)C8, (long)W * C8, (long)W * C8 + C8};
  Pack8 g, o[4];
  g.u = __ldg(reinterpret_cast<const uint4*>(dp) + i);
  const uint2 k = __ldg(reinterpret_cast<const uint2*>(code) + i);
  const uint32_t kw[2] = {k.x, k.y};
  const bf16 zero = __float2bfloat16_rn(0.f);
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const uint32_t best = (kw[e >> 2] >> (8 * (e & 3))) & 0xFFu;
#pragma unroll
    for (int q = 0; q < 4; ++q) o[q].h[e] = (uint32_t)q == best ? g.h[e] : zero;
  }
#pragma unroll
  for (int q = 0; q < 4; ++q) reinterpret_cast<uint4*>(dy)[base + off[q]] = o[q].u;
}

__global__ void maxpool_bwd_relu_bf16x8_kernel(const bf16* __restrict__ y, const bf16* __restrict__ dp,
                                               bf16* __restrict__ dy, long total8, int H, int W, int C8) {
  long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total8) return;
  int Wo = W / 2, Ho = H / 2;
  int c8 = i % C8; long t = i / C8;
  int j = t % Wo; t /= Wo;
  int ii = t % Ho; long n = t / Ho;
  const long base = ((n * H + 2 * ii) * W + 2 * j) * C8 + c8;
  const long off[4] = {0, (long)C8, (long)W * C8, (long)W * C8 + C8};
  Pack8 v[4], g, o[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) v[q].u = __ldg(reinterpret_cast<const uint4*>(y) + base + off[q]);
  g.u = __ldg(reinterpret_cast<const uint4*>(dp) + i);
  const bf16 zero = __float2bfloat16_rn(0.f);
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    float m = __bfloat162float(v[0].h[e]);
    int best = 0;
#pragma unroll
    for (int q = 1; q < 4; ++q) {
      float w = __bfloat162float(v[q].h[e]);
      if (w > m) { m = w; best = q; }
    }
    const bf16 gv = m > 0.f ? g.h[e] : zero;
#pragma unroll
    for (int q = 0; q < 4; ++q) o[q].h[e] = q == best ? gv : zero;
  }
#pragma unroll
  for (int q = 0; q < 4; ++q) reinterpret_cast<uint4*>(dy)[base + off[q]] = o[q].u;
}

// partial[chunk][c] = sum over the chunk's pixels; a block covers 256 / C8 pixels per step
__global__ void colsum_bf16x8_kernel(const bf16* __restrict__ dz, float* __restrict__ partial, long P, int C8,
                                     long p_per_chunk) {
  __shared__ float sm[256][9];
  const int rows = 256 / C8;             // pixels in flight per step (C8 divides 256)
  const int c8 = threadIdx.x % C8, r = threadIdx.x / C8;
  const long p0 = (long)blockIdx.x * p_per_chunk, p1 = min(P, p0 + p_per_chunk);
  float acc[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) acc[e] = 0.f;
  if (r < rows)
    for (long p = p0 + r; p < p1; p += rows) {
      Pack8 v;
      v.u = __ldg(reinterpret_cast<const uint4*>(dz) + p * C8 + c8);
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] += __bfloat162float(v.h[e]);
    }
#pragma unroll
  for (int e = 0; e < 8; ++e) sm[threadIdx.x][e] = acc[e];
  __syncthreads();
  for (int idx = threadIdx.x; idx < C8 * 8; idx += blockDim.x) {
    const int cc = idx / 8, e = idx % 8;
    float tot = 0.f;
    for (int q = 0; q < rows; ++q) tot += sm[q * C8 + cc][e];
    partial[(long)blockIdx.x * (C8 * 8) + idx] = tot;
  }
}

bool colsum_fast_ok(int C) { return C % 8 == 0 && 256 % (C / 8) == 0 && C <= 256 * 8; }
int colsum_fast_chunks(long P, int C) {
  long rows = 256 / (C / 8);
  long c = (P + rows * 16 - 1) / (rows * 16);
  return (int)(c > 592 ? 592 : (c < 1 ? 1 : c));
}

template <typename T>
cudaError_t simt_bias_grad(const T* dz, float* db, float* partial, long P, int C, cudaStream_t st) {
  if (std::is_same<T, bf16>::value && colsum_fast_ok(C)) {
    int chunks = colsum_fast_chunks(P, C);
    long per = (P + chunks - 1) / chunks;
    colsum_bf16x8_kernel<<<chunks, 256, 0, st>>>((const bf16*)dz, partial, P, C / 8, per);
    reduce_columns_kernel<<<(C + 31) / 32, dim3(32, 8), 0, st>>>(partial, db, C, chunks);
    return cudaGetLastError();
  }
  int chunks = colsum_chunks(P);
  long per = (P + chunks - 1) / chunks;
  dim3 grid((C + 31) / 32, chunks), block(32, 8);
  colsum_partial_kernel<T><<<grid, block, 0, st>>>(dz, partial, P, C, per);
  reduce_splits_kernel<<<(C + 255) / 256, 256, 0, st>>>(partial, db, C, chunks);
  return cudaGetLastError();
}

// ---- pooling ---------------------------------------------------------------

template <typename T>
__global__ void maxpool_fwd_kernel(const T* x, T* y, uint8_t* code, long total, int H, int W, int C) {
  long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  int Wo = W / 2, Ho = H / 2;
  int c = i % C; long t = i / C;
  int j = t % Wo; t /= Wo;
  int ii = t % Ho; long n = t / Ho;
  const T* p = x + ((n * H + 2 * ii) * W + 2 * j) * C + c;
  const float v[4] = {to_f32(p[0]), to_f32(p[C]), to_f32(p[(long)W * C]), to_f32(p[(long)W * C + C])};
  float m = v[0];
  int best = 0;
#pragma unroll
  for (int q = 1; q < 4; ++q)
    if (v[q] > m) { m = v[q]; best = q; }
  y[i] = from_f32<T>(m);
  if (code) code[i] = (uint8_t)(m > 0.f ? best : 4);
}

template <typename T>
__global__ void pool_scatter_kernel(const uint8_t* code, const T* dp, T* dy, long total, int H, int W, int C) {
  long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  int Wo = W / 2, Ho = H / 2;
  int c = i % C; long t = i / C;
  int j = t % Wo; t /= Wo;
  int ii = t % Ho; long n = t / Ho;
  long base = ((n * H + 2 * ii) * W + 2 * j) * C + c;
  long off[4] = {0, (long)C, (long)W * C, (long)W * C + C};
  const int best = code[i];
  const T g = dp[i];
#pragma unroll
  for (int q = 0; q < 4; ++q) dy[base + off[q]] = (q == best) ? g : from_f32<T>(0.f);
}

template <typename T>
__global__ void maxpool_bwd_relu_kernel(const T* y, const T* dp, T* dy, long total, int H, int W, int C) {
  long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  int Wo = W / 2, Ho = H / 2;
  int c = i % C; long t = i / C;
  int j = t % Wo; t /= Wo;
  int ii = t % Ho; long n = t / Ho;
  long base = ((n * H + 2 * ii) * W + 2 * j) * C + c;
  long off[4] = {0, (long)C, (long)W * C, (long)W * C + C};
  float m = to_f32(y[base]);
  int best = 0;
#pragma unroll
  for (int q = 1; q < 4; ++q) {
    float v = to_f32(y[base + off[q]]);
    if (v > m) { m = v; best = q; }
  }
  T g = (m > 0.f) ? dp[i] : from_f32<T>(0.f);
#pragma unroll
  for (int q = 0; q < 4; ++q) dy[base + off[q]] = (q == best) ? g : from_f32<T>(0.f);
}

template <typename T>
cudaError_t simt_maxpool_fwd(const T* x, T* y, int N, int H, int W, int C, cudaStream_t st, uint8_t* code) {
  long total = (long)N * (H / 2) * (W / 2) * C;
  if (std::is_same<T, bf16>::value && C % 8 == 0) {
    maxpool_fwd_bf16x8_kernel<<<(unsigned)((total / 8 + 255) / 256), 256, 0, st>>>((const bf16*)x, (bf16*)y, code,
                                                                                 total / 8, H, W, C / 8);
    return cudaGetLastError();
  }
  maxpool_fwd_kernel<T><<<(unsigned)((total + 255) / 256), 256, 0, st>>>(x, y, code, total, H, W, C);
  return cudaGetLastError();
}

template <typename T>
cudaError_t simt_pool_scatter(const uint8_t* code, const T* dp, T* dy, int N, int H, int W, int C, cudaStream_t st) {
  long total = (long)N * (H / 2) * (W / 2) * C;
  if (std::is_same<T, bf16>::value && C % 8 == 0) {
    pool_scatter_bf16x8_kernel<<<(unsigned)((total / 8 + 255) / 256), 256, 0, st>>>(code, (const bf16*)dp, (bf16*)dy,
                                                                                  total / 8, H, W, C / 8);
    return cudaGetLastError();
  }
  pool_scatter_kernel<T><<<(unsigned)((total + 255) / 256), 256, 0, st>>>(code, dp, dy, total, H, W, C);
  return cudaGetLastError();
}

template <typename T>
cudaError_t simt_maxpool_bwd_relu(const T* y, const T* dp, T* dy, int N, int H, int W, int C,
                                  cudaStream_t st) {
  long total = (long)N * (H / 2) * (W / 2) * C;
  if (std::is_same<T, bf16>::value && C % 8 == 0) {
    maxpool_bwd_relu_bf16x8_kernel<<<(unsigned)((total / 8 + 255) / 256), 256, 0, st>>>(
        (const bf16*)y, (const bf16*)dp, (bf16*)dy, total / 8, H, W, C / 8);
    return cudaGetLastError();
  }
  maxpool_bwd_relu_kernel<T><<<(unsigned)((total + 255) / 256), 256, 0, st>>>(y, dp, dy, total, H, W, C);
  return cudaGetLastError();
}

// ---- dense layers ----------------------------------------------------------

template <typename T>
cudaError_t simt_dense_nt(const T* A, const T* B, const float* bias, const T* mask, T* out_t,
                          float* out_f, int M, int N, int K, bool relu, cudaStream_t st) {
  RowMajorLoad<T> a{A, (long)K}, b{B, (long)K};
  StoreEpilogue<T> e{bias, mask, out_t, out_f, (long)N, relu ? 1 : 0};
  return launch_gemm(a, b, e, M, N, K, 1, st);
}

template <typename T>
cudaError_t simt_dense_dx(const T* dY, const T* W, const T* mask, T* dX, int M, int In, int Out,
                          cudaStream_t st) {
  RowMajorLoad<T> a{dY, (long)Out};
  ColMajorLoad<T> b{W, (long)In};
  StoreEpilogue<T> e{nullptr, mask, dX, nullptr, (long)In, 0};
  return launch_gemm(a, b, e, M, In, Out, 1, st);
}

template <typename T>
__global__ void dense_db_kernel(const T* dY, float* db, int M, int Out) {
  int o = blockIdx.x * blockDim.x + threadIdx.x;
  if (o >= Out) return;
  float s = 0.f;
  for (int m = 0; m < M; ++m) s += to_f32(dY[(long)m * Out + o]);
  db[o] = s;
}

template <typename T>
cudaError_t simt_dense_db(const T* dY, float* db, int M, int Out, cudaStream_t st) {
  dense_db_kernel<T><<<(Out + 127) / 128, 128, 0, st>>>(dY, db, M, Out);
  return cudaGetLastError();
}

template <typename T>
cudaError_t simt_dense_dw(const T* dY, const T* X, float* dW, float* db, int M, int In, int Out,
                          cudaStream_t st) {
  if (db) dense_db_kernel<T><<<(Out + 127) / 128, 128, 0, st>>>(dY, db, M, Out);
  ColMajorLoad<T> a{dY, (long)Out}, b{X, (long)In};
  StoreEpilogue<float> e{nullptr, nullptr, nullptr, dW, (long)In, 0};
  return launch_gemm(a, b, e, Out, In, M, 1, st);
}

// ---- softmax and cross-entropy ---------------------------------------------
// One warp per row; maximum and sum by shuffle reductions (butterfly, so every
// lane ends with the same value).

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

template <typename T>
__global__ void softmax_xent_kernel(const float* logits, const int32_t* labels, float* probs,
                                    T* dlogits, float* row_loss, int rows, int classes, int* dev_error) {
  int row = blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
  int lane = threadIdx.x % 32;
  if (row >= rows) return;
  const float* l = logits + (long)row * classes;
  float m = -INFINITY;
  for (int j = lane; j < classes; j += 32) m = fmaxf(m, l[j]);
  m = warp_max(m);
  float s = 0.f;
  for (int j = lane; j < classes; j += 32) s += expf(l[j] - m);
  s = warp_sum(s);
  float inv = 1.f / s;
  int label = labels ? labels[row] : -1;
  const bool bad_label = labels && (unsigned)label >= (unsigned)classes;
  if (bad_label) {  // never index with it: no one-hot term, a NaN loss, and a code for the host
    label = -1;
    if (lane == 0 && dev_error) atomicCAS(dev_error, 0, (int)kDevBadLabel);
  }
  float scale = 1.f / (float)rows;
  for (int j = lane; j < classes; j += 32) {
    float p = expf(l[j] - m) * inv;
    if (probs) probs[(long)row * classes + j] = p;
    if (dlogits) dlogits[(long)row * classes + j] = from_f32<T>((p - (j == label ? 1.f : 0.f)) * scale);
  }
  if (row_loss && lane == 0 && (label >= 0 || bad_label))
    row_loss[row] = bad_label ? __int_as_float(0x7fc00000) : (m + logf(s)) - l[label];
}

__global__ void mean_loss_kernel(const float* row_loss, float* loss, int rows) {
  float s = 0.f;
  for (int i = threadIdx.x; i < rows; i += 32) s += row_loss[i];
  s = warp_sum(s);
  if (threadIdx.x == 0) *loss = s / (float)rows;
}

template <typename T>
cudaError_t softmax_xent(const float* logits, const int32_t* labels, float* probs, T* dlogits,
                         float* row_loss, float* loss, int rows, int classes, cudaStream_t st, int* dev_error) {
  const int warps = 4;
  softmax_xent_kernel<T><<<(rows + warps - 1) / warps, warps * 32, 0, st>>>(
      logits, labels, probs, dlogits, row_loss, rows, classes, dev_error);
  if (loss && row_loss) mean_loss_kernel<<<1, 32, 0, st>>>(row_loss, loss, rows);
  return cudaGetLastError();
}

// ---- parameter preparation --------------------------------------------------

template <typename T>
__global__ void convert_kernel(const float* src, T* dst, size_t n) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = from_f32<T>(src[i]);
}

template <typename T>
cudaError_t convert_f32(const float* src, T* dst, size_t n, cudaStream_t st) {
  convert_kernel<T><<<(unsigned)((n + 255) / 256), 256, 0, st>>>(src, dst, n);
  return cudaGetLastError();
}

// p -= lr * g on the fp32 master copy, and the storage-type copy follows in the same pass
// (four elements per thread where the count allows; the tail one at a time).
template <typename T>
__global__ void sgd_update_kernel(float* __restrict__ p, const float* __restrict__ g, T* __restrict__ pt, float lr,
                                  const float* __restrict__ lr_dev, size_t n) {
  if (lr_dev) lr = *lr_dev;  // the rate of a recorded training step lives in device memory
  const size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i + 3 < n) {
    float4 w = *reinterpret_cast<float4*>(p + i);
    const float4 d = *reinterpret_cast<const float4*>(g + i);
    w.x = fmaf(-lr, d.x, w.x); w.y = fmaf(-lr, d.y, w.y); w.z = fmaf(-lr, d.z, w.z); w.w = fmaf(-lr, d.w, w.w);
    *reinterpret_cast<float4*>(p + i) = w;
    if (pt) {
      if (sizeof(T) == 2) {  // four bf16 as one 8-byte store (i is a multiple of 4, the buffer 256-byte aligned)
        __nv_bfloat162 lo = __floats2bfloat162_rn(w.x, w.y), hi = __floats2bfloat162_rn(w.z, w.w);
        *reinterpret_cast<uint2*>(pt + i) = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
      } else {
        pt[i] = from_f32<T>(w.x); pt[i + 1] = from_f32<T>(w.y); pt[i + 2] = from_f32<T>(w.z); pt[i + 3] = from_f32<T>(w.w);
      }
    }
  } else {
    for (size_t k = i; k < n; ++k) {
      const float w = fmaf(-lr, g[k], p[k]);
      p[k] = w;
      if (pt) pt[k] = from_f32<T>(w);
    }
  }
}

template <typename T>
cudaError_t sgd_update(float* params, const float* grads, T* params_t, float lr, size_t n, cudaStream_t st,
                       const float* lr_dev) {
  sgd_update_kernel<T><<<(unsigned)((n / 4 + 256) / 256), 256, 0, st>>>(params, grads, params_t, lr, lr_dev, n);
  return cudaGetLastError();
}

__global__ void set_scalar_kernel(float* dst, float v) { *dst = v; }
cudaError_t set_scalar(float* dst, float v, cudaStream_t st) {
  set_scalar_kernel<<<1, 1, 0, st>>>(dst, v);
  return cudaGetLastError();
}

// wt_t[c][r][s][k] = w[k][2-r][2-s][c]: the filter rotated by 180 degrees with
// the channel roles exchanged, so that the input gradient is itself a 3x3
// correlation of dz (appendix row "reverse").
template <typename T>
__global__ void dgrad_filter_kernel(const float* w, T* wt_t, int Cin, int Cout) {
  long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  long total = (long)Cin * 9 * Cout;
  if (i >= total) return;
  int k = i % Cout; long t = i / Cout;
  int rs = t % 9; int c = t / 9;
  wt_t[i] = from_f32<T>(w[((long)k * 9 + (8 - rs)) * Cin + c]);
}

template <typename T>
cudaError_t make_dgrad_filter(const float* w, T* wt_t, int Cin, int Cout, cudaStream_t st) {
  long total = (long)Cin * 9 * Cout;
  dgrad_filter_kernel<T><<<(unsigned)((total + 255) / 256), 256, 0, st>>>(w, wt_t, Cin, Cout);
  return cudaGetLastError();
}

// All three bf16 copies of the filters of up to 15 layers in one pass over the fp32 master: for
// w[k][tap][c] of a layer, the rotated filter of the input gradient [c][8 - tap][k], the tap-major
// filter [tap][k][c] and the rotated tap-major filter [8 - tap][c][k].  Two of the three are
// transposes of the [Cout][Cin] matrix of a tap: a block takes a 32 x 32 tile of it through shared
// memory so that reads and all three writes are contiguous.  first[] counts tiles here.
__global__ void refresh_filter_copies_kernel(const float* __restrict__ params, bf16* __restrict__ dgrad_w,
                                             bf16* __restrict__ tap_fwd, bf16* __restrict__ tap_bwd,
                                             FilterCopyTable tab) {
  __shared__ float tile[32][33];
  const long b = blockIdx.x;
  int l = 0;
  while (l + 1 < tab.layers && b >= tab.first[l + 1]) ++l;  // first[] is ascending
  const int Cin = tab.Cin[l], Cout = tab.Cout[l];
  long t = b - tab.first[l];
  const int c_tiles = Cin / 32;
  const int c0 = (int)(t % c_tiles) * 32; t /= c_tiles;
  const int k_tiles = Cout / 32;
  const int k0 = (int)(t % k_tiles) * 32;
  const int tap = (int)(t / k_tiles);
  const float* w = params + tab.w_off[l];
  const size_t base = tab.copy_off[l];
  const int tx = threadIdx.x, ty = threadIdx.y;  // 32 x 8
#pragma unroll
  for (int j = 0; j < 32; j += 8) {
    const int k = k0 + ty + j, c = c0 + tx;
    const float v = w[((size_t)k * 9 + tap) * Cin + c];
    tile[ty + j][tx] = v;
    tap_fwd[base + ((size_t)tap * Cout + k) * Cin + c] = __float2bfloat16_rn(v);
  }
  __syncthreads();
#pragma unroll
  for (int j = 0; j < 32; j += 8) {
    const int c = c0 + ty + j, k = k0 + tx;
    const bf16 v = __float2bfloat16_rn(tile[tx][ty + j]);
    dgrad_w[base + ((size_t)c * 9 + (8 - tap)) * Cout + k] = v;
    tap_bwd[base + ((size_t)(8 - tap) * Cin + c) * Cout + k] = v;
  }
}

cudaError_t refresh_filter_copies(const float* params, bf16* dgrad_w, bf16* tap_fwd, bf16* tap_bwd,
                                  const FilterCopyTable& tab, cudaStream_t st) {
  refresh_filter_copies_kernel<<<(unsigned)tab.total, dim3(32, 8), 0, st>>>(params, dgrad_w, tap_fwd, tap_bwd, tab);
  return cudaGetLastError();
}

#define INSTANTIATE(T)                                                                               \
  template cudaError_t simt_conv3x3<T>(const T*, const T*, const float*, const T*, T*, ConvShape,    \
                                       bool, cudaStream_t);                                          \
  template cudaError_t simt_conv3x3_wgrad<T>(const T*, const T*, float*, float*, float*, ConvShape,  \
                                             cudaStream_t);                                          \
  template cudaError_t simt_maxpool_fwd<T>(const T*, T*, int, int, int, int, cudaStream_t, uint8_t*); \
  template cudaError_t simt_pool_scatter<T>(const uint8_t*, const T*, T*, int, int, int, int,        \
                                            cudaStream_t);                                           \
  template cudaError_t simt_maxpool_bwd_relu<T>(const T*, const T*, T*, int, int, int, int,          \
                                                cudaStream_t);                                       \
  template cudaError_t simt_dense_nt<T>(const T*, const T*, const float*, const T*, T*, float*, int, \
                                        int, int, bool, cudaStream_t);                               \
  template cudaError_t simt_dense_dx<T>(const T*, const T*, const T*, T*, int, int, int,             \
                                        cudaStream_t);                                               \
  template cudaError_t simt_dense_dw<T>(const T*, const T*, float*, float*, int, int, int,           \
                                        cudaStream_t);                                               \
  template cudaError_t simt_bias_grad<T>(const T*, float*, float*, long, int, cudaStream_t);           \
  template cudaError_t simt_dense_db<T>(const T*, float*, int, int, cudaStream_t);                    \
  template cudaError_t softmax_xent<T>(const float*, const int32_t*, float*, T*, float*, float*,     \
                                       int, int, cudaStream_t, int*);                                \
  template cudaError_t convert_f32<T>(const float*, T*, size_t, cudaStream_t);                       \
  template cudaError_t sgd_update<T>(float*, const float*, T*, float, size_t, cudaStream_t,          \
                                     const float*);                                                  \
  template cudaError_t make_dgrad_filter<T>(const float*, T*, int, int, cudaStream_t);

INSTANTIATE(float)
INSTANTIATE(bf16)

}  // namespace vgg
