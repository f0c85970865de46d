/*
 * CPU oracle for the PCONV forward pass.  TEST INFRASTRUCTURE ONLY: nothing on the product path
 * may call, link or import this file; it shares no code with the CUDA library.
 *
 * What it computes is the plain definition the sparse method must reproduce exactly (up to
 * rounding order): a direct 3x3 cross-correlation (the paper's Eq. 1, g(x,y) = sum_{k,l}
 * f(x+k, y+l) h(k,l), no kernel flip) over the DENSE weight tensor, in which pattern pruning
 * (element-wise product of a kernel with a binary 3x3 Sparse Convolution Pattern, "Sparse
 * Convolution Pattern" section) and connectivity pruning (removal of whole kernels, same
 * section) appear only as zeros left in place.  There is no sparse walk, blocking, fusion or
 * reordering here: seven nested loops n, o, i, j, c, u, v with an fp64 accumulator.
 *
 *   H_out = floor((H + 2 - 3) / s) + 1,   W_out likewise            (zero padding 1, s in {1,2})
 *   y[n,o,i,j] = act( b[o] + sum_c sum_u sum_v xpad[n,c,i*s+u-1,j*s+v-1] * W[o,c,u,v] )
 *
 * The sum and the bias add are fp64; the activation is applied in fp64; the result is rounded
 * once to fp32.  Zero padding, stride, bias and the fused ReLU are this build's reading where the
 * paper is silent.
 *
 * Pins (tests/test_oracle_pins.py): scatter-form brute force, single-tap shifts, closed forms on
 * constant and ramp inputs, linearity / permutation / stride-subsampling invariants, torch's
 * fp64 conv2d.  Every function below is pinned; none is "parity unpinned".
 */
#include <stddef.h>
#include <stdint.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Eq. 1 with zero padding 1 and stride s; see the header comment. Returns 0, or -1 on bad args. */
int oracle_conv3x3(const float* x, const float* w, const float* bias, float* y, int n_img,
                   int c_in, int h, int w_in, int c_out, int stride, int relu) {
  if (!x || !w || !y || n_img < 0 || c_in <= 0 || c_out <= 0 || h <= 0 || w_in <= 0 ||
      (stride != 1 && stride != 2))
    return -1;
  const int h_out = (h + 2 - 3) / stride + 1;
  const int w_out = (w_in + 2 - 3) / stride + 1;
  const long long jobs = (long long)n_img * c_out;
#pragma omp parallel for schedule(static)
  for (long long job = 0; job < jobs; ++job) {
    const int n = (int)(job / c_out);
    const int o = (int)(job % c_out);
    for (int i = 0; i < h_out; ++i) {
      for (int j = 0; j < w_out; ++j) {
        double acc = 0.0;
        for (int c = 0; c < c_in; ++c) {
          for (int u = 0; u < 3; ++u) {
            const int r = i * stride + u - 1;
            if (r < 0 || r >= h) continue; /* zero padding row */
            for (int v = 0; v < 3; ++v) {
              const int q = j * stride + v - 1;
              if (q < 0 || q >= w_in) continue; /* zero padding column */
              acc += (double)x[(((size_t)n * c_in + c) * h + r) * w_in + q] *
                     (double)w[(((size_t)o * c_in + c) * 3 + u) * 3 + v];
            }
          }
        }
        if (bias) acc += (double)bias[o];
        if (relu && acc < 0.0) acc = 0.0;
        y[(((size_t)n * c_out + o) * h_out + i) * w_out + j] = (float)acc;
      }
    }
  }
  return 0;
}

/* 2x2 max-pool with stride 2 (floor on odd sizes): y[n,c,i,j] = max over rows 2i,2i+1 and
 * columns 2j,2j+1.  This is the plain pooling that sits between the VGG blocks. */
int oracle_maxpool2x2(const float* x, float* y, int n_img, int c, int h, int w_in) {
  if (!x || !y || n_img < 0 || c <= 0 || h < 2 || w_in < 2) return -1;
  const int h_out = h / 2, w_out = w_in / 2;
  const long long planes = (long long)n_img * c;
#pragma omp parallel for schedule(static)
  for (long long p = 0; p < planes; ++p) {
    const float* xp = x + (size_t)p * h * w_in;
    float* yp = y + (size_t)p * h_out * w_out;
    for (int i = 0; i < h_out; ++i)
      for (int j = 0; j < w_out; ++j) {
        float m = xp[(size_t)(2 * i) * w_in + 2 * j];
        const float b = xp[(size_t)(2 * i) * w_in + 2 * j + 1];
        const float cc = xp[(size_t)(2 * i + 1) * w_in + 2 * j];
        const float d = xp[(size_t)(2 * i + 1) * w_in + 2 * j + 1];
        if (b > m) m = b;
        if (cc > m) m = cc;
        if (d > m) m = d;
        yp[(size_t)i * w_out + j] = m;
      }
  }
  return 0;
}
