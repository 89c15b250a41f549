/*
 * Seeded synthetic inputs for the VGG19 pass: weights, images, labels.
 *
 * This file holds no arithmetic of the network itself.  It only turns
 * (seed, stream, index) into numbers, so that the CUDA library and the CPU
 * checker can be handed bit-identical inputs.  It is compiled twice: into a
 * small shared library of its own that Python loads, and into the CUDA
 * library for vgg19_create(seed).
 *
 * Generator (counter based, every element independent of the others):
 *   splitmix64 (Steele, Lea, Flood 2014; Vigna's public-domain constants)
 *   evaluated at state  s0 + (i + 1) * 0x9E3779B97F4A7C15,
 *   s0 = splitmix64 output of (seed * 1000003 + stream).
 *   uniform:  u = (x >> 11) * 2^-53                           in [0, 1)
 *   normal :  Box-Muller on outputs 2i and 2i+1,
 *             u1 = ((x0 >> 11) + 1) * 2^-53 in (0, 1],  u2 = (x1 >> 11) * 2^-53,
 *             z = sqrt(-2 ln u1) * cos(2 pi u2), computed in fp64, then
 *             scaled and rounded to fp32.
 *   label  :  x mod n_classes.
 * With bf16_exact != 0 the fp32 result is rounded to the nearest bfloat16
 * (ties to even) and widened back, so that a bf16 run and an fp64 check see
 * exactly the same numbers.
 */
#include "seeded_inputs.h"

#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

static inline uint64_t sm64_mix(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}

static inline uint64_t sm64_at(uint64_t s0, uint64_t i) {
  return sm64_mix(s0 + (i + 1) * 0x9E3779B97F4A7C15ULL);
}

static inline uint64_t stream_base(uint64_t seed, uint64_t stream) {
  return sm64_mix(seed * 1000003ULL + stream + 0x9E3779B97F4A7C15ULL);
}

static inline float to_bf16_exact(float v) {
  uint32_t b;
  memcpy(&b, &v, 4);
  if ((b & 0x7F800000u) != 0x7F800000u) {           /* finite */
    b += 0x7FFFu + ((b >> 16) & 1u);                /* nearest, ties to even */
    b &= 0xFFFF0000u;
  }
  memcpy(&v, &b, 4);
  return v;
}

void seeded_uniform_f32(float *out, size_t n, uint64_t seed, uint64_t stream,
                        double shift, double scale, int bf16_exact) {
  const uint64_t s0 = stream_base(seed, stream);
#pragma omp parallel for schedule(static)
  for (ptrdiff_t i = 0; i < (ptrdiff_t)n; ++i) {
    double u = (double)(sm64_at(s0, (uint64_t)i) >> 11) * 0x1.0p-53;
    float v = (float)((u - shift) * scale);
    out[i] = bf16_exact ? to_bf16_exact(v) : v;
  }
}

void seeded_normal_f32(float *out, size_t n, uint64_t seed, uint64_t stream,
                       double stddev, int take_abs, int bf16_exact) {
  const uint64_t s0 = stream_base(seed, stream);
  const double two_pi = 6.283185307179586476925286766559;
#pragma omp parallel for schedule(static)
  for (ptrdiff_t i = 0; i < (ptrdiff_t)n; ++i) {
    double u1 = (double)((sm64_at(s0, 2 * (uint64_t)i) >> 11) + 1) * 0x1.0p-53;
    double u2 = (double)(sm64_at(s0, 2 * (uint64_t)i + 1) >> 11) * 0x1.0p-53;
    double z = sqrt(-2.0 * log(u1)) * cos(two_pi * u2);
    if (take_abs) z = fabs(z);
    float v = (float)(z * stddev);
    out[i] = bf16_exact ? to_bf16_exact(v) : v;
  }
}

void seeded_labels_i32(int32_t *out, size_t n, uint64_t seed, uint64_t stream,
                       int32_t n_classes) {
  const uint64_t s0 = stream_base(seed, stream);
  for (size_t i = 0; i < n; ++i)
    out[i] = (int32_t)(sm64_at(s0, (uint64_t)i) % (uint64_t)n_classes);
}

/* ---- the VGG19 parameter set -------------------------------------------- */

static const int kConvOut[16] = {64, 64, 128, 128, 256, 256, 256, 256,
                                 512, 512, 512, 512, 512, 512, 512, 512};

size_t seeded_vgg19_param_count(int height, int width) {
  size_t total = 0;
  int cin = 3;
  for (int l = 0; l < 16; ++l) {
    total += (size_t)kConvOut[l] * 9 * cin + kConvOut[l];
    cin = kConvOut[l];
  }
  size_t fc_in = (size_t)512 * (height / 32) * (width / 32);
  total += fc_in * 4096 + 4096;
  total += (size_t)4096 * 4096 + 4096;
  total += (size_t)4096 * 1000 + 1000;
  return total;
}

void seeded_vgg19_params(float *out, int height, int width, uint64_t seed,
                         double bias_std, int bf16_exact) {
  /* Flat order: for layer 1..19, weight then bias.  Conv weight is
   * [Cout][3][3][Cin], dense weight [out][in].  Tensor t (0..37) draws from
   * stream t.  He-normal: stddev = sqrt(2 / fan_in). */
  size_t off = 0;
  int cin = 3;
  uint64_t t = 0;
  for (int l = 0; l < 19; ++l) {
    size_t fan_in, n_out;
    if (l < 16) {
      fan_in = (size_t)9 * cin;
      n_out = kConvOut[l];
      cin = kConvOut[l];
    } else if (l == 16) {
      fan_in = (size_t)512 * (height / 32) * (width / 32);
      n_out = 4096;
    } else if (l == 17) {
      fan_in = 4096;
      n_out = 4096;
    } else {
      fan_in = 4096;
      n_out = 1000;
    }
    seeded_normal_f32(out + off, n_out * fan_in, seed, t++,
                      sqrt(2.0 / (double)fan_in), 0, bf16_exact);
    off += n_out * fan_in;
    if (bias_std > 0.0) {
      seeded_normal_f32(out + off, n_out, seed, t++, bias_std, 0, bf16_exact);
    } else {
      for (size_t i = 0; i < n_out; ++i) out[off + i] = 0.0f;
      ++t;
    }
    off += n_out;
  }
}
