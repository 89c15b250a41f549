/*
 * TEST INFRASTRUCTURE - not part of the product path.
 *
 * Plain fp64 CPU definitions of the operations the VGG19 forward and
 * backward pass is made of (paper section 7.2 "VGG19 forward pass", 7.3
 * "VGG19 backward pass", and the appendix table of HLO instruction kinds:
 * convolution, dot, reduce-window, maximum, select-and-scatter, reverse,
 * reduce, exponential, divide).  Each function is the textbook definition
 * written as a loop nest: no tiling, no fusion, no algebraic shortcuts.  The
 * only liberty taken is the order in which a sum's terms are added (OpenMP
 * simd reductions), which changes the fp64 result by rounding only.
 *
 * Layouts: activations x[n][h][w][c] (c fastest); 3x3 filters
 * W[k][r][s][c] (k = output channel, c fastest); dense weights W[o][i].
 * Every pointer is a host pointer owned by the caller.  Nothing here is
 * shared with, or derived from, the CUDA implementation.
 *
 * Pins (see tests/test_oracle_pins.py): delta kernel = identity, constant
 * input closed form, a hand-worked 3x3 example that tells correlation from
 * flipped convolution, adjoint identities <conv(x),dz> = <x,dgrad(dz)> =
 * <W,wgrad(x,dz)>, agreement with torch.nn.functional.conv2d / autograd in
 * fp64, pooling on a ramp, softmax/cross-entropy closed forms, the dense()
 * example of section 7.1, and central finite differences on a tiny net.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>

typedef ptrdiff_t idx;

/* Section 7.2 / appendix row "convolution": 3x3, stride 1, zero padding 1,
 * cross-correlation (the filter is not flipped):
 *   z[n,h,w,k] = b[k] + sum_{r,s,c} x[n,h+r-1,w+s-1,c] * W[k,r,s,c]        */
void oracle_conv3x3_fwd(const double *x, const double *W, const double *b, double *z,
                        int N, int H, int Wd, int Cin, int Cout) {
#pragma omp parallel for collapse(2) schedule(static)
  for (int n = 0; n < N; ++n)
    for (int h = 0; h < H; ++h)
      for (int w = 0; w < Wd; ++w)
        for (int k = 0; k < Cout; ++k) {
          double acc = b ? b[k] : 0.0;
          for (int r = 0; r < 3; ++r) {
            int hh = h + r - 1;
            if (hh < 0 || hh >= H) continue;
            for (int s = 0; s < 3; ++s) {
              int ww = w + s - 1;
              if (ww < 0 || ww >= Wd) continue;
              const double *xp = x + (((idx)n * H + hh) * Wd + ww) * Cin;
              const double *wp = W + (((idx)k * 3 + r) * 3 + s) * Cin;
              double part = 0.0;
#pragma omp simd reduction(+ : part)
              for (int c = 0; c < Cin; ++c) part += xp[c] * wp[c];
              acc += part;
            }
          }
          z[(((idx)n * H + h) * Wd + w) * Cout + k] = acc;
        }
}

/* Section 7.3 / appendix rows "convolution" (backward) and "reverse":
 * gradient with respect to the input.  Gathering form of the adjoint:
 *   dx[n,h,w,c] = sum_{k,r,s} dz[n,h-r+1,w-s+1,k] * W[k,r,s,c]
 * i.e. a correlation of dz with the filter rotated by 180 degrees.          */
void oracle_conv3x3_dgrad(const double *dz, const double *W, double *dx,
                          int N, int H, int Wd, int Cin, int Cout) {
#pragma omp parallel for collapse(2) schedule(static)
  for (int n = 0; n < N; ++n)
    for (int h = 0; h < H; ++h)
      for (int w = 0; w < Wd; ++w) {
        double *dxp = dx + (((idx)n * H + h) * Wd + w) * Cin;
        for (int c = 0; c < Cin; ++c) dxp[c] = 0.0;
        for (int r = 0; r < 3; ++r) {
          int hh = h - r + 1;
          if (hh < 0 || hh >= H) continue;
          for (int s = 0; s < 3; ++s) {
            int ww = w - s + 1;
            if (ww < 0 || ww >= Wd) continue;
            const double *dzp = dz + (((idx)n * H + hh) * Wd + ww) * Cout;
            for (int k = 0; k < Cout; ++k) {
              const double d = dzp[k];
              const double *wp = W + (((idx)k * 3 + r) * 3 + s) * Cin;
#pragma omp simd
              for (int c = 0; c < Cin; ++c) dxp[c] += d * wp[c];
            }
          }
        }
      }
}

/* Section 7.3 / appendix row "convolution" (backward): gradient with respect
 * to the filter, accumulated INTO dW (the caller zeroes it, or keeps a
 * running sum over chunks of the batch):
 *   dW[k,r,s,c] += sum_{n,h,w} dz[n,h,w,k] * x[n,h+r-1,w+s-1,c]
 * and (appendix row "reduce") the bias gradient db[k] += sum_{n,h,w} dz.   */
void oracle_conv3x3_wgrad(const double *x, const double *dz, double *dW, double *db,
                          int N, int H, int Wd, int Cin, int Cout) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int k = 0; k < Cout; ++k) {
    double bsum = 0.0;
    for (int n = 0; n < N; ++n)
      for (int h = 0; h < H; ++h)
        for (int w = 0; w < Wd; ++w) {
          const double d = dz[(((idx)n * H + h) * Wd + w) * Cout + k];
          bsum += d;
          if (d == 0.0) continue; /* adds exact zeros only */
          for (int r = 0; r < 3; ++r) {
            int hh = h + r - 1;
            if (hh < 0 || hh >= H) continue;
            for (int s = 0; s < 3; ++s) {
              int ww = w + s - 1;
              if (ww < 0 || ww >= Wd) continue;
              const double *xp = x + (((idx)n * H + hh) * Wd + ww) * Cin;
              double *gp = dW + (((idx)k * 3 + r) * 3 + s) * Cin;
#pragma omp simd
              for (int c = 0; c < Cin; ++c) gp[c] += d * xp[c];
            }
          }
        }
    if (db) db[k] += bsum;
  }
}

/* Appendix row "maximum": ReLU y = max(z, 0). */
void oracle_relu_fwd(const double *z, double *y, idx n) {
  for (idx i = 0; i < n; ++i) y[i] = z[i] > 0.0 ? z[i] : 0.0;
}

/* Appendix rows "less-than"/"select": dz = dy where z > 0, else 0
 * (the derivative at exactly 0 is taken as 0).                              */
void oracle_relu_bwd(const double *z, const double *dy, double *dz, idx n) {
  for (idx i = 0; i < n; ++i) dz[i] = 0.0 < z[i] ? dy[i] : 0.0;
}

/* Appendix row "reduce-window": 2x2 max-pool, stride 2.
 *   p[n,i,j,c] = max_{a,b in {0,1}} y[n,2i+a,2j+b,c]                        */
void oracle_maxpool2x2_fwd(const double *y, double *p, int N, int H, int Wd, int C) {
  const int Ho = H / 2, Wo = Wd / 2;
  for (int n = 0; n < N; ++n)
    for (int i = 0; i < Ho; ++i)
      for (int j = 0; j < Wo; ++j)
        for (int c = 0; c < C; ++c) {
          double m = y[(((idx)n * H + 2 * i) * Wd + 2 * j) * C + c];
          for (int a = 0; a < 2; ++a)
            for (int b = 0; b < 2; ++b) {
              double v = y[(((idx)n * H + 2 * i + a) * Wd + 2 * j + b) * C + c];
              if (v > m) m = v;
            }
          p[(((idx)n * Ho + i) * Wo + j) * C + c] = m;
        }
}

/* Appendix row "select-and-scatter": each dp goes to the position of its
 * window's maximum; on ties the first position in the scan order
 * (0,0),(0,1),(1,0),(1,1) takes it.  dy is fully overwritten.               */
void oracle_maxpool2x2_bwd(const double *y, const double *dp, double *dy,
                           int N, int H, int Wd, int C) {
  const int Ho = H / 2, Wo = Wd / 2;
  for (idx i = 0; i < (idx)N * H * Wd * C; ++i) dy[i] = 0.0;
  for (int n = 0; n < N; ++n)
    for (int i = 0; i < Ho; ++i)
      for (int j = 0; j < Wo; ++j)
        for (int c = 0; c < C; ++c) {
          int ba = 0, bb = 0;
          double m = y[(((idx)n * H + 2 * i) * Wd + 2 * j) * C + c];
          for (int a = 0; a < 2; ++a)
            for (int b = 0; b < 2; ++b) {
              double v = y[(((idx)n * H + 2 * i + a) * Wd + 2 * j + b) * C + c];
              if (v > m) { m = v; ba = a; bb = b; }
            }
          dy[(((idx)n * H + 2 * i + ba) * Wd + 2 * j + bb) * C + c] =
              dp[(((idx)n * Ho + i) * Wo + j) * C + c];
        }
}

/* Section 7.1: dense(W, x, b) = (W * x) .+ b, for a batch of N columns kept
 * as rows:  y[n,o] = b[o] + sum_i W[o,i] * x[n,i]   (appendix row "dot").   */
void oracle_dense_fwd(const double *x, const double *W, const double *b, double *y,
                      int N, int In, int Out) {
#pragma omp parallel for schedule(static)
  for (int o = 0; o < Out; ++o)
    for (int n = 0; n < N; ++n) {
      double acc = 0.0;
      const double *wp = W + (idx)o * In, *xp = x + (idx)n * In;
#pragma omp simd reduction(+ : acc)
      for (int i = 0; i < In; ++i) acc += wp[i] * xp[i];
      y[(idx)n * Out + o] = acc + (b ? b[o] : 0.0);
    }
}

/* Adjoint of dense: dx = W^T dy (overwritten); dW += dy x^T; db += sum_n dy. */
void oracle_dense_bwd(const double *x, const double *W, const double *dy,
                      double *dx, double *dW, double *db, int N, int In, int Out) {
  if (dx) {
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
      double *dxp = dx + (idx)n * In;
      for (int i = 0; i < In; ++i) dxp[i] = 0.0;
      for (int o = 0; o < Out; ++o) {
        const double d = dy[(idx)n * Out + o];
        const double *wp = W + (idx)o * In;
#pragma omp simd
        for (int i = 0; i < In; ++i) dxp[i] += d * wp[i];
      }
    }
  }
#pragma omp parallel for schedule(static)
  for (int o = 0; o < Out; ++o) {
    double *gp = dW + (idx)o * In;
    double bsum = 0.0;
    for (int n = 0; n < N; ++n) {
      const double d = dy[(idx)n * Out + o];
      const double *xp = x + (idx)n * In;
      bsum += d;
#pragma omp simd
      for (int i = 0; i < In; ++i) gp[i] += d * xp[i];
    }
    if (db) db[o] += bsum;
  }
}

/* Section 7.1: softmax(xs) = exp.(xs) ./ sum(exp.(xs)), per row.  The row
 * maximum is subtracted first, which leaves the quotient unchanged.         */
void oracle_softmax(const double *l, double *p, int N, int C) {
  for (int n = 0; n < N; ++n) {
    const double *lp = l + (idx)n * C;
    double m = lp[0], sum = 0.0;
    for (int j = 1; j < C; ++j) if (lp[j] > m) m = lp[j];
    for (int j = 0; j < C; ++j) { p[(idx)n * C + j] = exp(lp[j] - m); sum += p[(idx)n * C + j]; }
    for (int j = 0; j < C; ++j) p[(idx)n * C + j] /= sum;
  }
}

/* Mean cross-entropy of the softmax of l against integer labels, computed as
 * log-sum-exp minus the label's logit:  L = (1/Ntot) sum_n -ln p[n,label_n].
 * Ntot is the size of the whole batch (>= N when N is a chunk of it).       */
double oracle_cross_entropy(const double *l, const int32_t *labels, int N, int C, int Ntot) {
  double total = 0.0;
  for (int n = 0; n < N; ++n) {
    const double *lp = l + (idx)n * C;
    double m = lp[0], sum = 0.0;
    for (int j = 1; j < C; ++j) if (lp[j] > m) m = lp[j];
    for (int j = 0; j < C; ++j) sum += exp(lp[j] - m);
    total += (m + log(sum)) - lp[labels[n]];
  }
  return total / (double)Ntot;
}

/* dL/dlogits of the mean cross-entropy: (p - onehot(label)) / Ntot. */
void oracle_softmax_ce_bwd(const double *p, const int32_t *labels, double *dl,
                           int N, int C, int Ntot) {
  for (int n = 0; n < N; ++n)
    for (int j = 0; j < C; ++j)
      dl[(idx)n * C + j] = (p[(idx)n * C + j] - (j == labels[n] ? 1.0 : 0.0)) / (double)Ntot;
}

/* Jacobian-transpose of softmax applied to an upstream gradient g (used for
 * the paper's stand-in loss sum(m(x)), section 7.3, whose g is all ones):
 *   dl[n,j] = p[n,j] * (g[n,j] - sum_i g[n,i] p[n,i])                       */
void oracle_softmax_bwd(const double *p, const double *g, double *dl, int N, int C) {
  for (int n = 0; n < N; ++n) {
    double dot = 0.0;
    for (int j = 0; j < C; ++j) dot += g[(idx)n * C + j] * p[(idx)n * C + j];
    for (int j = 0; j < C; ++j)
      dl[(idx)n * C + j] = p[(idx)n * C + j] * (g[(idx)n * C + j] - dot);
  }
}

/* Storage format of the bf16 configurations ("bf16 activations/weights with
 * fp32 accumulate"): round every element to the nearest bfloat16 (8 significant
 * bits, ties to even), keeping it as a double.  A value v = m * 2^e with
 * 0.5 <= |m| < 1 lies in a binade whose bf16 spacing is 2^(e-8); below the
 * smallest normal the spacing stays at 2^-133.  rint() rounds ties to even in
 * the default rounding mode and the scaling by a power of two is exact.      */
void oracle_round_bf16(double *x, idx n) {
  for (idx i = 0; i < n; ++i) {
    double v = x[i];
    if (v == 0.0 || !isfinite(v)) continue;
    int e;
    frexp(v, &e);
    int q = e - 8;
    if (q < -133) q = -133;
    x[i] = ldexp(rint(ldexp(v, -q)), q);
  }
}
