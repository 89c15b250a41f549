/* Seeded synthetic inputs (weights, images, labels) for the VGG19 pass.
 * All pointers are host pointers owned by the caller.  See seeded_inputs.c
 * for the generator's definition. */
#ifndef SEEDED_INPUTS_H_
#define SEEDED_INPUTS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* out[i] = (u_i - shift) * scale, u_i uniform in [0,1). */
void seeded_uniform_f32(float *out, size_t n, uint64_t seed, uint64_t stream,
                        double shift, double scale, int bf16_exact);

/* out[i] = stddev * z_i (|z_i| when take_abs), z_i standard normal. */
void seeded_normal_f32(float *out, size_t n, uint64_t seed, uint64_t stream,
                       double stddev, int take_abs, int bf16_exact);

/* out[i] uniform integer in [0, n_classes). */
void seeded_labels_i32(int32_t *out, size_t n, uint64_t seed, uint64_t stream,
                       int32_t n_classes);

/* Number of fp32 elements of the flat VGG19 parameter buffer for an
 * height x width x 3 input (multiples of 32). */
size_t seeded_vgg19_param_count(int height, int width);

/* He-normal weights; biases zero when bias_std == 0, else N(0, bias_std). */
void seeded_vgg19_params(float *out, int height, int width, uint64_t seed,
                         double bias_std, int bf16_exact);

#ifdef __cplusplus
}
#endif
#endif /* SEEDED_INPUTS_H_ */
