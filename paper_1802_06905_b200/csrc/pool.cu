// Pooling (Section 6): the loop nest of Eq. 1 without its Filter,
//
//     for b,c,k,w,h,r,s:   Out(k,h,w,b) (+)= Image(r + sw*w, s + sh*h, c, b)
//
// read literally: k does not occur on the right-hand side, so the reduction runs over (c, r, s) and
// every k-plane of Out holds the same values.  The kernel therefore reduces once per output pixel
// and writes the result K times: Image is read once from HBM (window overlaps are served by L1/L2),
// Out is written once, which is the first two terms of the section's bound; the third term
// (B*C*K*W*H*R*S/M) never binds here because the reduction is shared by all k.
//
// The work is HBM-bound (no contraction, no tensor cores): b is the fastest subscript of both
// arrays, so a thread owns 8 consecutive images (one 16-byte vector) of one output pixel, a warp
// reads/writes 512 contiguous bytes per pixel group.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <string>

#include "../../include/cconv.h"
#include "host_setup.h"

namespace cconv {
namespace {

struct PoolParams {
  int B, C, K, W, H, R, S, sw, sh;
  int Hi;
  int nb;             // vectors per pixel: B / VEC
  long long total_v;  // H * W * nb output vectors per k-plane
  int kper;           // k-planes written by one blockIdx.y
  int terms;          // C * R * S
  float inv_rs;       // 1 / (R*S)
  int overlap;        // 1: launched so that the stream's next kernel may start before this one ends
  int wait_prev;      // 1: wait for the stream's earlier work before touching memory
};

// Overlap with the stream's neighbours (as the convolution kernels do it): the next kernel may be
// launched as soon as every block of this one has started; a call whose arrays meet those of a call
// that may still be running waits for the earlier work first; and thread 0 of every block leaves
// only after the kernel in front is complete, so completion still follows stream order.
__device__ __forceinline__ void pool_enter(const PoolParams& p) {
  if (p.overlap) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (p.wait_prev) asm volatile("griddepcontrol.wait;" ::: "memory");
  }
}
__device__ __forceinline__ void pool_leave(const PoolParams& p) {
  if (p.overlap && !p.wait_prev && threadIdx.x == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
}

template <int VEC>
__device__ __forceinline__ void load_vec(const __nv_bfloat16* p, float (&x)[VEC]) {
  if constexpr (VEC == 8) {
    const uint4 q = __ldg(reinterpret_cast<const uint4*>(p));
    const uint32_t u[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[2 * i] = __uint_as_float(u[i] << 16);
      x[2 * i + 1] = __uint_as_float(u[i] & 0xffff0000u);
    }
  } else {
    x[0] = __bfloat162float(*p);
  }
}

template <typename OutT, int VEC>
__device__ __forceinline__ void store_vec(OutT* p, const float (&x)[VEC]) {
  if constexpr (VEC == 8 && sizeof(OutT) == 2) {
    uint32_t u[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h2 = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
      u[i] = *reinterpret_cast<const uint32_t*>(&h2);
    }
    __stcs(reinterpret_cast<uint4*>(p), make_uint4(u[0], u[1], u[2], u[3]));
  } else if constexpr (VEC == 8) {
    __stcs(reinterpret_cast<float4*>(p), make_float4(x[0], x[1], x[2], x[3]));
    __stcs(reinterpret_cast<float4*>(p) + 1, make_float4(x[4], x[5], x[6], x[7]));
  } else if constexpr (sizeof(OutT) == 2) {
    *reinterpret_cast<__nv_bfloat16*>(p) = __float2bfloat16_rn(x[0]);
  } else {
    *reinterpret_cast<float*>(p) = x[0];
  }
}

// A block of 256 threads owns VPB consecutive output vectors; its G = 256/VPB thread groups split the
// C*R*S terms of the reduction (thread t: vector t % VPB, group t / VPB), combine through shared
// memory in a fixed order (the result does not depend on timing), then split the K planes of the
// write.  VPB = 256 (G = 1): a thread does everything for its own vector (few terms, few planes).
// Eight loads are kept in flight per thread: the loop is bound by memory latency otherwise.
template <typename OutT, int VEC, bool MAX, int VPB>
__global__ void __launch_bounds__(256) cconv_pool_kernel(const __nv_bfloat16* __restrict__ image,
                                                         OutT* __restrict__ out, PoolParams p) {
  constexpr int G = 256 / VPB;
  pool_enter(p);
  const int vi = threadIdx.x % VPB, g = threadIdx.x / VPB;
  const long long v = (long long)blockIdx.x * VPB + vi;
  const bool valid = v < p.total_v;
  const long long vv = valid ? v : 0;
  int bv, w, h;
  if (p.total_v <= 0x7fffffffll) {  // the usual case: 32-bit divisions
    const unsigned u = unsigned(vv), pix = u / unsigned(p.nb);
    bv = int(u - pix * unsigned(p.nb));
    h = int(pix / unsigned(p.W));
    w = int(pix - unsigned(h) * unsigned(p.W));
  } else {
    bv = int(vv % p.nb);
    const long long pix = vv / p.nb;
    w = int(pix % p.W);
    h = int(pix / p.W);
  }
  // Image element offset of (x = sw*w, y = sh*h, c = 0, b = bv*VEC)
  const __nv_bfloat16* base =
      image + (((long long)p.sw * w * p.Hi + (long long)p.sh * h) * p.C) * p.B + (long long)bv * VEC;
  const long long xstride = (long long)p.Hi * p.C * p.B, ystride = (long long)p.C * p.B;
  // Term t = (c*R + r)*S + s, stepped by G = dc*R*S + dr*S + ds with no division or multiplication
  // in the loop: the pointer moves by a constant, plus a correction whenever s or r wraps.
  const int RS = p.R * p.S;
  const int dc = G / RS, dr = (G - dc * RS) / p.S, ds = G - dc * RS - dr * p.S;
  const int c0 = g / RS;
  int r = (g - c0 * RS) / p.S, s = g - c0 * RS - r * p.S;
  const __nv_bfloat16* ptr = base + r * xstride + s * ystride + (long long)c0 * p.B;
  const long long step = ds * ystride + dr * xstride + (long long)dc * p.B;
  const long long wrap_s = xstride - p.S * ystride, wrap_r = (long long)p.B - p.R * xstride;
  auto next_ptr = [&]() {
    const __nv_bfloat16* cur = ptr;
    ptr += step;
    s += ds;
    if (s >= p.S) { s -= p.S; ptr += wrap_s; ++r; }
    r += dr;
    if (r >= p.R) { r -= p.R; ptr += wrap_r; }
    return cur;
  };

  float acc[VEC];
#pragma unroll
  for (int i = 0; i < VEC; ++i) acc[i] = MAX ? -INFINITY : 0.f;
  constexpr int U = 8;  // loads in flight per thread
  int t = g;
  if constexpr (MAX && VEC == 8) {
    // the maximum of bf16 values is taken on the packed pairs themselves (exact), 4 ops per vector
    const __nv_bfloat162 ninf = __floats2bfloat162_rn(-INFINITY, -INFINITY);
    __nv_bfloat162 m[4] = {ninf, ninf, ninf, ninf};
    // (the last round is a full round with some loads switched off, not a loop of single loads:
    // every round costs a memory latency)
    const uint4 ninf4 = make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
    for (; t < p.terms; t += U * G) {
      uint4 q[U];
#pragma unroll
      for (int u = 0; u < U; ++u)
        q[u] = (t + u * G < p.terms) ? __ldg(reinterpret_cast<const uint4*>(next_ptr())) : ninf4;
#pragma unroll
      for (int u = 0; u < U; ++u) {
        m[0] = __hmax2(m[0], *reinterpret_cast<const __nv_bfloat162*>(&q[u].x));
        m[1] = __hmax2(m[1], *reinterpret_cast<const __nv_bfloat162*>(&q[u].y));
        m[2] = __hmax2(m[2], *reinterpret_cast<const __nv_bfloat162*>(&q[u].z));
        m[3] = __hmax2(m[3], *reinterpret_cast<const __nv_bfloat162*>(&q[u].w));
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      acc[2 * i] = __low2float(m[i]);
      acc[2 * i + 1] = __high2float(m[i]);
    }
  } else {
    // (sums: a predicated last round was measured slower here -- 14.9 -> 16.6 us on the seven-loop
    // benchmark shape -- so the remainder goes load by load)
    for (; t + (U - 1) * G < p.terms; t += U * G) {
      float x[U][VEC];
#pragma unroll
      for (int u = 0; u < U; ++u) load_vec<VEC>(next_ptr(), x[u]);
#pragma unroll
      for (int u = 0; u < U; ++u) {
#pragma unroll
        for (int i = 0; i < VEC; ++i) acc[i] = MAX ? fmaxf(acc[i], x[u][i]) : acc[i] + x[u][i];
      }
    }
    for (; t < p.terms; t += G) {
      float x[VEC];
      load_vec<VEC>(next_ptr(), x);
#pragma unroll
      for (int i = 0; i < VEC; ++i) acc[i] = MAX ? fmaxf(acc[i], x[i]) : acc[i] + x[i];
    }
  }

  if constexpr (G > 1) {
    // Combine the G partial results of each output element: thread o < VPB*VEC owns element o and
    // reads part[j][o] for j = 0..G-1 (consecutive threads, consecutive words: no bank conflicts).
    __shared__ float part[G][VPB * VEC];
    __shared__ float total[VPB * VEC];
#pragma unroll
    for (int i = 0; i < VEC; ++i) part[g][vi * VEC + i] = acc[i];
    __syncthreads();
    for (int o = threadIdx.x; o < VPB * VEC; o += 256) {
      float a = part[0][o];
      for (int j = 1; j < G; ++j) a = MAX ? fmaxf(a, part[j][o]) : a + part[j][o];
      total[o] = a;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < VEC; ++i) acc[i] = total[vi * VEC + i];
  }
  if (!MAX) {
#pragma unroll
    for (int i = 0; i < VEC; ++i) acc[i] *= p.inv_rs;
  }
  if (valid) {
    const int k0 = blockIdx.y * p.kper;
    const int k1 = min(p.K, k0 + p.kper);
    for (int k = k0 + g; k < k1; k += G)
      store_vec<OutT, VEC>(out + ((long long)k * p.total_v + v) * VEC, acc);
  }
  pool_leave(p);
}

// The usual pooling layer (C = 1 with the channels folded into b, 8 images per thread, a 2x2 or
// 3x3 window): a thread per output vector with the whole window loaded before the first use -- no
// term stepping, 32-bit index arithmetic -- then the K planes written in turn.  The general kernel
// above takes a 3x3 window in two rounds of loads (eight, then one) and ran 25 % slower on it.
template <typename OutT, int R, int S, bool MAX>
__global__ void __launch_bounds__(256) cconv_pool_window_kernel(const __nv_bfloat16* __restrict__ image,
                                                                OutT* __restrict__ out, PoolParams p) {
  pool_enter(p);
  const unsigned v = blockIdx.x * 256u + threadIdx.x;   // the host sends total_v < 2^31 here
  if (v >= unsigned(p.total_v)) {
    pool_leave(p);
    return;
  }
  const unsigned pix = v / unsigned(p.nb), bv = v - pix * unsigned(p.nb);
  const unsigned h = pix / unsigned(p.W), w = pix - h * unsigned(p.W);
  const long long ystride = (long long)p.B, xstride = (long long)p.Hi * p.B;
  const __nv_bfloat16* base =
      image + ((long long)p.sw * w * p.Hi + (long long)p.sh * h) * p.B + (long long)bv * 8;
  uint4 q[R * S];
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int s = 0; s < S; ++s)
      q[r * S + s] = __ldg(reinterpret_cast<const uint4*>(base + r * xstride + s * ystride));
  float acc[8];
  if constexpr (MAX) {
    __nv_bfloat162 m[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) m[i] = reinterpret_cast<const __nv_bfloat162*>(&q[0])[i];
#pragma unroll
    for (int t = 1; t < R * S; ++t)
#pragma unroll
      for (int i = 0; i < 4; ++i) m[i] = __hmax2(m[i], reinterpret_cast<const __nv_bfloat162*>(&q[t])[i]);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      acc[2 * i] = __low2float(m[i]);
      acc[2 * i + 1] = __high2float(m[i]);
    }
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
#pragma unroll
    for (int t = 0; t < R * S; ++t) {
      const uint32_t u[4] = {q[t].x, q[t].y, q[t].z, q[t].w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        acc[2 * i] += __uint_as_float(u[i] << 16);
        acc[2 * i + 1] += __uint_as_float(u[i] & 0xffff0000u);
      }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] *= p.inv_rs;
  }
  const int k0 = blockIdx.y * p.kper;
  const int k1 = min(p.K, k0 + p.kper);
  for (int k = k0; k < k1; ++k) store_vec<OutT, 8>(out + ((long long)k * p.total_v + v) * 8, acc);
  pool_leave(p);
}

template <typename OutT>
cudaError_t pool_launch(void (*kernel)(const __nv_bfloat16*, OutT*, PoolParams), dim3 grid,
                        cudaStream_t stream, const __nv_bfloat16* im, OutT* o, const PoolParams& p) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(256);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = p.overlap ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, im, o, p);
}

template <typename OutT, int R, int S>
cudaError_t launch_pool_window(const void* image, void* out, const PoolParams& p, bool mx, dim3 grid,
                               cudaStream_t stream) {
  const __nv_bfloat16* im = static_cast<const __nv_bfloat16*>(image);
  OutT* o = static_cast<OutT*>(out);
  if (mx) return pool_launch(cconv_pool_window_kernel<OutT, R, S, true>, grid, stream, im, o, p);
  return pool_launch(cconv_pool_window_kernel<OutT, R, S, false>, grid, stream, im, o, p);
}

template <typename OutT, int VEC, bool MAX>
cudaError_t launch_pool_t(const void* image, void* out, const PoolParams& p, int vpb, dim3 grid,
                          cudaStream_t stream) {
  const __nv_bfloat16* im = static_cast<const __nv_bfloat16*>(image);
  OutT* o = static_cast<OutT*>(out);
  if (vpb == 256) return pool_launch(cconv_pool_kernel<OutT, VEC, MAX, 256>, grid, stream, im, o, p);
  if (vpb == 32) return pool_launch(cconv_pool_kernel<OutT, VEC, MAX, 32>, grid, stream, im, o, p);
  return pool_launch(cconv_pool_kernel<OutT, VEC, MAX, 8>, grid, stream, im, o, p);
}

}  // namespace
}  // namespace cconv

using namespace cconv;

extern "C" int cconv_pool_lower_bound(int B, int C, int K, int W, int H, int R, int S, int sw,
                                      int sh, double M_words, double terms_out[3]) {
  if (B <= 0 || C <= 0 || K <= 0 || W <= 0 || H <= 0 || R <= 0 || S <= 0 || sw <= 0 || sh <= 0 ||
      !(M_words > 0) || !terms_out)
    return CCONV_EINVAL;
  const double bwh = double(B) * W * H;
  terms_out[0] = bwh * K;
  terms_out[1] = bwh * C * sw * sh;
  terms_out[2] = bwh * C * K * R * S / M_words;
  return CCONV_OK;
}

extern "C" int cconv_pool_forward(const void* Image, void* Out, int B, int C, int K, int W, int H,
                                  int R, int S, int sw, int sh, int op, int out_dtype,
                                  void* cuda_stream) {
  if (!Image || !Out) return CCONV_EINVAL;
  if (B <= 0 || C <= 0 || K <= 0 || W <= 0 || H <= 0 || R <= 0 || S <= 0 || sw <= 0 || sh <= 0)
    return CCONV_EINVAL;
  if (op != CCONV_POOL_AVG && op != CCONV_POOL_MAX) return CCONV_EINVAL;
  if (out_dtype != CCONV_OUT_BF16 && out_dtype != CCONV_OUT_F32) return CCONV_EINVAL;
  if ((reinterpret_cast<uintptr_t>(Image) & 15u) || (reinterpret_cast<uintptr_t>(Out) & 31u))
    return CCONV_EINVAL;
  const double Wi = double(sw) * (W - 1) + R, Hi = double(sh) * (H - 1) + S;
  if (Wi * Hi * C * B > 9.0e18 || double(K) * H * W * B > 9.0e18 || double(C) * R * S > 2.0e9 ||
      Hi > 2.0e9)
    return CCONV_EINVAL;

  PoolParams p;
  p.B = B; p.C = C; p.K = K; p.W = W; p.H = H; p.R = R; p.S = S; p.sw = sw; p.sh = sh;
  p.Hi = int(Hi);
  const int vec = B % 8 == 0 ? 8 : 1;
  p.nb = B / vec;
  p.total_v = (long long)H * W * p.nb;
  p.terms = C * R * S;
  p.inv_rs = 1.0f / (float(R) * float(S));
  p.overlap = 1;
  if (const char* ov = std::getenv("CCONV_POOL_OVERLAP")) p.overlap = std::atoi(ov) != 0;
  p.wait_prev = 0;
  // Vectors per block: a thread per vector when there is little to share (few terms, few planes);
  // otherwise 32, or 8 when 32 would leave most SMs without a block and the reduction outweighs
  // the writes (8 lanes per plane make 128-byte write runs instead of 512-byte ones).
  int vpb = 256;
  if (p.terms + K >= 64) vpb = ((p.total_v + 31) / 32 >= 1184 || K >= 4 * p.terms) ? 32 : 8;
  const long long blocks_x = (p.total_v + vpb - 1) / vpb;
  if (blocks_x > 0x7fffffffll) return CCONV_EUNSUPPORTED;
  // Few blocks, and writes that outweigh the reduction: split the planes over blockIdx.y (each
  // slice repeats the reduction, whose reads hit L2) until the grid fills the machine a few times.
  int ksplit = 1;
  if (vpb == 32 && blocks_x < 1184) {
    ksplit = int((1184 + blocks_x - 1) / blocks_x);
    ksplit = std::max(1, std::min(ksplit, (K + 63) / 64));
  }
  if (const char* f = std::getenv("CCONV_POOL_FORCE")) {  // diagnostics: "vectors per block,k slices"
    int fv = 0, fk = 0;
    if (std::sscanf(f, "%d,%d", &fv, &fk) == 2 && (fv == 8 || fv == 32 || fv == 256) && fk >= 1 &&
        fk <= 65535 && (p.total_v + fv - 1) / fv <= 0x7fffffffll) {
      vpb = fv;
      ksplit = std::min(fk, K);
    }
  }
  const long long blocks = (p.total_v + vpb - 1) / vpb;
  p.kper = (K + ksplit - 1) / ksplit;
  ksplit = (K + p.kper - 1) / p.kper;
  const dim3 grid{unsigned(blocks), unsigned(ksplit), 1u};
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const bool f32 = out_dtype == CCONV_OUT_F32, mx = op == CCONV_POOL_MAX;
  cudaError_t e;
  if (p.overlap) {
    // stream order against the calls that may still be running: this call's blocks (256 threads of
    // an SM's 2048 each) all stay resident until the kernel in front is complete
    int dev = 0, sm_count = 0;
    e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) {
      set_last_cuda_error(std::string("cconv_pool_forward: ") + cudaGetErrorString(e));
      return CCONV_ECUDA;
    }
    CallSpans spans;
    spans.image.lo = static_cast<const char*>(Image);
    spans.image.hi = spans.image.lo + size_t(Wi * Hi) * size_t(C) * size_t(B) * 2;
    spans.out.lo = static_cast<const char*>(Out);
    spans.out.hi = spans.out.lo + size_t(K) * H * W * size_t(B) * (f32 ? 4 : 2);
    spans.sms_by_threads = double(blocks) * double(ksplit) / 8.0;
    p.wait_prev = note_call(cuda_stream, spans, Overlap::kDeep, sm_count) ? 1 : 0;
  } else {
    note_ordinary_launch(cuda_stream);
  }
  const bool window33 = R == 3 && S == 3, window22 = R == 2 && S == 2;
  if (C == 1 && vec == 8 && vpb == 256 && (window33 || window22) && p.total_v < 0x7fffffffll &&
      !std::getenv("CCONV_POOL_FORCE")) {
    if (window33)
      e = f32 ? launch_pool_window<float, 3, 3>(Image, Out, p, mx, grid, stream)
              : launch_pool_window<__nv_bfloat16, 3, 3>(Image, Out, p, mx, grid, stream);
    else
      e = f32 ? launch_pool_window<float, 2, 2>(Image, Out, p, mx, grid, stream)
              : launch_pool_window<__nv_bfloat16, 2, 2>(Image, Out, p, mx, grid, stream);
  } else if (vec == 8) {
    if (f32) e = mx ? launch_pool_t<float, 8, true>(Image, Out, p, vpb, grid, stream)
                    : launch_pool_t<float, 8, false>(Image, Out, p, vpb, grid, stream);
    else e = mx ? launch_pool_t<__nv_bfloat16, 8, true>(Image, Out, p, vpb, grid, stream)
                : launch_pool_t<__nv_bfloat16, 8, false>(Image, Out, p, vpb, grid, stream);
  } else {
    if (f32) e = mx ? launch_pool_t<float, 1, true>(Image, Out, p, vpb, grid, stream)
                    : launch_pool_t<float, 1, false>(Image, Out, p, vpb, grid, stream);
    else e = mx ? launch_pool_t<__nv_bfloat16, 1, true>(Image, Out, p, vpb, grid, stream)
                : launch_pool_t<__nv_bfloat16, 1, false>(Image, Out, p, vpb, grid, stream);
  }
  if (e != cudaSuccess) {
    set_last_cuda_error(std::string("cconv_pool_kernel launch: ") + cudaGetErrorString(e));
    return CCONV_ECUDA;
  }
  return CCONV_OK;
}
