/*
 * TEST INFRASTRUCTURE ONLY -- CPU oracle for the pooling loop nest of Section 6.
 *
 * This file is the slow, plain definition against which the CUDA pooling kernel is checked.  It
 * shares no code with the CUDA path and must never be called from it.
 *
 * Section 6 keeps the seven loops of Eq. 1 and drops the Filter:
 *
 *   for b,c,k,w,h,r,s:   Out(k,h,w,b) (+)= Image(r + sw*w, s + sh*h, c, b)
 *
 * with a (+) b = a + b/(R*S) ("average", Out starting from 0) or max(a, b) ("max", Out starting
 * from -infinity, the identity of max).  Read literally -- and this oracle reads it literally --
 * the subscript k does not occur on the right-hand side, so every k-plane of Out receives the same
 * value, and the reduction runs over the channel c as well as over the window (r,s):
 *
 *   average:  Out(k,h,w,b) = (1/(R*S)) * sum_{c,r,s} Image(r + sw*w, s + sh*h, c, b)
 *   max:      Out(k,h,w,b) = max_{c,r,s}             Image(r + sw*w, s + sh*h, c, b)
 *
 * The paper prints the divisor as "rs"; it is read as R*S (with the loop variables the first term
 * would divide by zero).  The usual per-channel pooling layer is the case C = K = 1 with the
 * channels folded into b.  Array shapes and layouts are those of the convolution oracle:
 *   Image [Wi][Hi][C][B], Wi = sw*(W-1)+R, Hi = sh*(H-1)+S;   Out [K][H][W][B]; last subscript fastest.
 *
 * All arithmetic is fp64 on the exact values of the bf16 inputs.  For the average the routine also
 * returns Abs(k,h,w,b) = (1/(R*S)) * sum |Image| over the same terms, which scales the tolerance.
 *
 * Pins (tests, "not gpu"): a library fp64 avg_pool2d / max_pool2d on the transposed arrays for
 * C = 1 and, summed / maximised over channels, for C > 1; the convolution oracle with a constant
 * Filter 1/(R*S) (average only); constant and delta images in closed form; pure-Python brute
 * force on tiny shapes; all k-planes equal.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double pool_bf16_to_f64(uint16_t v) {
  uint32_t u = ((uint32_t)v) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

/* op: 0 = average, 1 = max.  Loops nested in the order the paper lists them; single thread.
 * absum may be NULL (and is left untouched for max). */
int pool7nl_bf16(const uint16_t* image, double* out, double* absum, int B, int C, int K, int W,
                 int H, int R, int S, int sw, int sh, int op) {
  if (B <= 0 || C <= 0 || K <= 0 || W <= 0 || H <= 0 || R <= 0 || S <= 0 || sw <= 0 || sh <= 0)
    return -1;
  if (op != 0 && op != 1) return -1;
  const int64_t Hi = (int64_t)sh * (H - 1) + S;
  const int64_t n = (int64_t)K * H * W * B;
  const double rs = (double)R * (double)S;
  for (int64_t i = 0; i < n; ++i) out[i] = op == 0 ? 0.0 : -INFINITY;
  if (absum && op == 0)
    for (int64_t i = 0; i < n; ++i) absum[i] = 0.0;
  for (int b = 0; b < B; ++b)
    for (int c = 0; c < C; ++c)
      for (int k = 0; k < K; ++k)
        for (int w = 0; w < W; ++w)
          for (int h = 0; h < H; ++h)
            for (int r = 0; r < R; ++r)
              for (int s = 0; s < S; ++s) {
                const double x = pool_bf16_to_f64(
                    image[((((int64_t)r + (int64_t)sw * w) * Hi + (s + (int64_t)sh * h)) * C + c) * B + b]);
                double* o = out + (((int64_t)k * H + h) * W + w) * B + b;
                if (op == 0) {
                  *o = *o + x / rs;
                  if (absum) absum[(((int64_t)k * H + h) * W + w) * B + b] += fabs(x) / rs;
                } else {
                  *o = x > *o ? x : *o;
                }
              }
  return 0;
}

/* n selected output elements; khwb holds n quadruples (k,h,w,b).  Each element is reduced on its
 * own over (c,r,s). */
int pool7nl_bf16_at(const uint16_t* image, const int32_t* khwb, int64_t n, double* out,
                    double* absum, int B, int C, int K, int W, int H, int R, int S, int sw, int sh,
                    int op) {
  if (B <= 0 || C <= 0 || K <= 0 || W <= 0 || H <= 0 || R <= 0 || S <= 0 || sw <= 0 || sh <= 0)
    return -1;
  if (op != 0 && op != 1) return -1;
  const int64_t Hi = (int64_t)sh * (H - 1) + S;
  const double rs = (double)R * (double)S;
  int bad = 0;
  for (int64_t i = 0; i < n; ++i) {
    const int k = khwb[4 * i], h = khwb[4 * i + 1], w = khwb[4 * i + 2], b = khwb[4 * i + 3];
    if (k < 0 || k >= K || h < 0 || h >= H || w < 0 || w >= W || b < 0 || b >= B) {
      bad = 1;
      continue;
    }
    double acc = op == 0 ? 0.0 : -INFINITY, ab = 0.0;
    for (int c = 0; c < C; ++c)
      for (int r = 0; r < R; ++r)
        for (int s = 0; s < S; ++s) {
          const double x = pool_bf16_to_f64(
              image[((((int64_t)r + (int64_t)sw * w) * Hi + (s + (int64_t)sh * h)) * C + c) * B + b]);
          if (op == 0) {
            acc += x / rs;
            ab += fabs(x) / rs;
          } else {
            acc = x > acc ? x : acc;
          }
        }
    out[i] = acc;
    if (absum) absum[i] = ab;
  }
  return bad ? -3 : 0;
}
