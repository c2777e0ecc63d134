/*
 * TEST INFRASTRUCTURE ONLY -- CPU oracle for the seven-nested-loop CNN (Eq. 1, Section 2).
 *
 * This file is the slow, plain definition against which the CUDA path is checked.  It shares no
 * code with the CUDA path and must never be called from it.
 *
 *   Out(k,h,w,b) = sum_{c<C} sum_{r<R} sum_{s<S} Image(r + sw*w, s + sh*h, c, b) * Filter(k,r,s,c)
 *
 * Reading of the array shapes (Section 2 gives subscripts only, no memory layout; boundary
 * conditions are ignored there): dense row-major arrays, last subscript fastest,
 *   Image  [Wi][Hi][C][B]   Wi = sw*(W-1)+R, Hi = sh*(H-1)+S   (the valid-window extent)
 *   Filter [K][R][S][C]
 *   Out    [K][H][W][B]     (note: h before w, while Image is indexed w-direction first)
 * r pairs with the w-direction (first Image subscript), s with the h-direction (second).
 * It is a cross-correlation: the filter is not flipped.  Out starts from zero.
 *
 * All arithmetic is fp64.  Inputs are either doubles or bf16 bit patterns (upper 16 bits of an
 * IEEE binary32), decoded exactly.  Besides Out the routines return
 *   Abs(k,h,w,b) = sum |Image * Filter| over the same C*R*S terms,
 * which is what the per-element tolerance of the parity tests is scaled by.
 *
 * Pins (tests, "not gpu"): delta filter / delta image index checks, brute force in pure Python on
 * tiny shapes, R=S=1 against a library matrix product, constant inputs against C*R*S*a*f,
 * loop-order invariance (cnn7nl_f64_paper_order), linearity, and a library fp64 conv2d.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_bits_to_f64(uint16_t v) {
  uint32_t u = ((uint32_t)v) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

int cnn7nl_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Eq. 1, loops ordered k,h,w | r,s,c | b.  Threads split k*h.  absum may be NULL. */
int cnn7nl_f64(const double* image, const double* filter, double* out, double* absum, int B,
               int C, int K, int W, int H, int R, int S, int sw, int sh) {
  if (B <= 0 || C <= 0 || K <= 0 || W <= 0 || H <= 0 || R <= 0 || S <= 0 || sw <= 0 || sh <= 0)
    return -1;
  const int64_t Hi = (int64_t)sh * (H - 1) + S;
  const int64_t KH = (int64_t)K * H;
#pragma omp parallel for schedule(static)
  for (int64_t kh = 0; kh < KH; ++kh) {
    const int k = (int)(kh / H), h = (int)(kh % H);
    for (int w = 0; w < W; ++w) {
      double* o = out + (((int64_t)k * H + h) * W + w) * B;
      double* a = absum ? absum + (((int64_t)k * H + h) * W + w) * B : NULL;
      for (int b = 0; b < B; ++b) o[b] = 0.0;
      if (a)
        for (int b = 0; b < B; ++b) a[b] = 0.0;
      for (int r = 0; r < R; ++r)
        for (int s = 0; s < S; ++s)
          for (int c = 0; c < C; ++c) {
            const double f = filter[(((int64_t)k * R + r) * S + s) * C + c];
            const double* im =
                image + ((((int64_t)r + (int64_t)sw * w) * Hi + (s + (int64_t)sh * h)) * C + c) * B;
            for (int b = 0; b < B; ++b) o[b] += im[b] * f;
            if (a)
              for (int b = 0; b < B; ++b) a[b] += fabs(im[b] * f);
          }
    }
  }
  return 0;
}

/* The same sum with the loops in the order the paper writes them (b,c,k,w,h,r,s), single thread,
 * accumulating straight into Out.  Used only to pin loop-order invariance. */
int cnn7nl_f64_paper_order(const double* image, const double* filter, double* out, int B, int C,
                           int K, int W, int H, int R, int S, int sw, int sh) {
  if (B <= 0 || C <= 0 || K <= 0 || W <= 0 || H <= 0 || R <= 0 || S <= 0 || sw <= 0 || sh <= 0)
    return -1;
  const int64_t Hi = (int64_t)sh * (H - 1) + S;
  memset(out, 0, sizeof(double) * (size_t)K * H * W * B);
  for (int b = 0; b < B; ++b)
    for (int c = 0; c < C; ++c)
      for (int k = 0; k < K; ++k)
        for (int w = 0; w < W; ++w)
          for (int h = 0; h < H; ++h)
            for (int r = 0; r < R; ++r)
              for (int s = 0; s < S; ++s)
                out[(((int64_t)k * H + h) * W + w) * B + b] +=
                    image[((((int64_t)r + (int64_t)sw * w) * Hi + (s + (int64_t)sh * h)) * C + c) * B + b] *
                    filter[(((int64_t)k * R + r) * S + s) * C + c];
  return 0;
}

/* bf16-bit inputs, whole result. */
int cnn7nl_bf16(const uint16_t* image, const uint16_t* filter, double* out, double* absum, int B,
                int C, int K, int W, int H, int R, int S, int sw, int sh) {
  if (B <= 0 || C <= 0 || K <= 0 || W <= 0 || H <= 0 || R <= 0 || S <= 0 || sw <= 0 || sh <= 0)
    return -1;
  const int64_t Wi = (int64_t)sw * (W - 1) + R, Hi = (int64_t)sh * (H - 1) + S;
  const int64_t ni = Wi * Hi * C * B, nf = (int64_t)K * R * S * C;
  double* di = (double*)malloc(sizeof(double) * (size_t)ni);
  double* df = (double*)malloc(sizeof(double) * (size_t)nf);
  if (!di || !df) {
    free(di);
    free(df);
    return -2;
  }
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < ni; ++i) di[i] = bf16_bits_to_f64(image[i]);
  for (int64_t i = 0; i < nf; ++i) df[i] = bf16_bits_to_f64(filter[i]);
  int rc = cnn7nl_f64(di, df, out, absum, B, C, K, W, H, R, S, sw, sh);
  free(di);
  free(df);
  return rc;
}

/* bf16-bit inputs, n selected output elements; khwb holds n quadruples (k,h,w,b).
 * Each element is the C*R*S-term sum of Eq. 1 evaluated on its own. */
int cnn7nl_bf16_at(const uint16_t* image, const uint16_t* filter, const int32_t* khwb, int64_t n,
                   double* out, double* absum, int B, int C, int K, int W, int H, int R, int S,
                   int sw, int sh) {
  if (B <= 0 || C <= 0 || K <= 0 || W <= 0 || H <= 0 || R <= 0 || S <= 0 || sw <= 0 || sh <= 0)
    return -1;
  const int64_t Hi = (int64_t)sh * (H - 1) + S;
  int bad = 0;
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) {
    const int k = khwb[4 * i], h = khwb[4 * i + 1], w = khwb[4 * i + 2], b = khwb[4 * i + 3];
    if (k < 0 || k >= K || h < 0 || h >= H || w < 0 || w >= W || b < 0 || b >= B) {
      bad = 1;
      continue;
    }
    double acc = 0.0, ab = 0.0;
    for (int r = 0; r < R; ++r)
      for (int s = 0; s < S; ++s)
        for (int c = 0; c < C; ++c) {
          const double f = bf16_bits_to_f64(filter[(((int64_t)k * R + r) * S + s) * C + c]);
          const double x = bf16_bits_to_f64(
              image[((((int64_t)r + (int64_t)sw * w) * Hi + (s + (int64_t)sh * h)) * C + c) * B + b]);
          acc += x * f;
          ab += fabs(x * f);
        }
    out[i] = acc;
    if (absum) absum[i] = ab;
  }
  return bad ? -3 : 0;
}
