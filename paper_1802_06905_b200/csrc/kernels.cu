// sm_100a kernels for the seven-nested-loop CNN (Eq. 1, Section 2):
//   Out(k,h,w,b) = sum_{c,r,s} Image(r+sw*w, s+sh*h, c, b) * Filter(k,r,s,c)
// Image [Wi][Hi][C][B], Filter [K][R][S][C], Out [K][H][W][B], bf16, last subscript fastest.
//
// cconv_halo_kernel realises the blocked loop nest of Section 5 on one SM:
//   outer loops  {b,k,w,h}_1 : the persistent tile loop (k innermost so CTAs that run at the same
//                              time share one Image block in L2),
//   outer loop   c_1         : two shared-memory rings: an Image stage per block of b_c channels
//                              (the halo tile b_b x b_c x (sw(b_w-1)+R) x (sh(b_h-1)+S)) and a Filter
//                              stage per group of about nine packed b_k x 16 blocks,
//   inner loops  {b,k,w,h,c,r,s}_2 : tcgen05.mma instructions.  Every (r,s) tap reads the SAME
//                              resident halo tile through a shifted shared-memory descriptor, so
//                              an Image word fetched once serves all R*S taps and all b_k channels
//                              (the reuse behind the fifth term of Theorem 1).
// As a GEMM: D[k][n=(h,w,b)] += A_rs[k][c] * B_rs[c][n]; A = Filter slab, K-major (c contiguous);
// B = Image halo view, MN-major (b contiguous).  Accumulators live in TMEM (fp32).
#include <cuda_bf16.h>

#include "kernels.h"
#include "ptx_sm100.cuh"

namespace cconv {

// ------------------------------------------------------------------------------------------------
// CUDA-core kernel: any shape, any alignment.  One thread = KT output channels of one (h,w,b).
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void store_out(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
__device__ __forceinline__ void store_out(float* p, float v) { *p = v; }

template <int KT, typename OutT>
__global__ void __launch_bounds__(256) cconv_simt_kernel(const __nv_bfloat16* __restrict__ image,
                                                         const __nv_bfloat16* __restrict__ filter,
                                                         OutT* __restrict__ out, Dims d) {
  const long long kq_n = (d.K + KT - 1) / KT;
  const long long total = kq_n * d.H * d.W * d.B;
  const long long Hi = (long long)d.sh * (d.H - 1) + d.S;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int b = int(idx % d.B);
    long long t = idx / d.B;
    const int w = int(t % d.W);
    t /= d.W;
    const int h = int(t % d.H);
    const int k0 = int(t / d.H) * KT;
    float acc[KT];
#pragma unroll
    for (int j = 0; j < KT; ++j) acc[j] = 0.f;
    for (int r = 0; r < d.R; ++r)
      for (int s = 0; s < d.S; ++s) {
        const __nv_bfloat16* ip =
            image + (((long long)(r + d.sw * w) * Hi + (s + d.sh * h)) * d.C) * d.B + b;
        const __nv_bfloat16* fp = filter + (((long long)k0 * d.R + r) * d.S + s) * d.C;
#pragma unroll 4
        for (int c = 0; c < d.C; ++c) {
          const float x = __bfloat162float(ip[(long long)c * d.B]);
#pragma unroll
          for (int j = 0; j < KT; ++j)
            if (k0 + j < d.K)
              acc[j] = fmaf(x, __bfloat162float(fp[(long long)j * d.R * d.S * d.C + c]), acc[j]);
        }
      }
#pragma unroll
    for (int j = 0; j < KT; ++j)
      if (k0 + j < d.K)
        store_out(out + (((long long)(k0 + j) * d.H + h) * d.W + w) * d.B + b, acc[j]);
  }
}

// Tiny problems: the time of the kernel above is one thread's chain of dependent loads (C*R*S of
// them, a few in flight at a time).  Here eight lanes share one output element, lane j taking the
// filter taps j, j+8, ... with all channels of a tap loaded before the first use, and a three-step
// shuffle tree adds the eight partial sums (fixed order: results are reproducible run to run).
template <typename OutT>
__global__ void __launch_bounds__(128) cconv_simt_taps_kernel(const __nv_bfloat16* __restrict__ image,
                                                              const __nv_bfloat16* __restrict__ filter,
                                                              OutT* __restrict__ out, Dims d) {
  const long long total = (long long)d.K * d.H * d.W * d.B;
  const long long Hi = (long long)d.sh * (d.H - 1) + d.S;
  const int sub = threadIdx.x & 7;
  const int RS = d.R * d.S;
  const long long groups_per_grid = (long long)gridDim.x * (blockDim.x >> 3);
  // the loop bound is the same for all lanes of a warp (its four groups are consecutive)
  for (long long base = (blockIdx.x * (long long)blockDim.x + (threadIdx.x & ~31)) >> 3; base < total;
       base += groups_per_grid) {
    const long long idx = base + ((threadIdx.x & 31) >> 3);
    const bool valid = idx < total;
    float acc = 0.f;
    if (valid) {
      const int b = int(idx % d.B);
      long long t = idx / d.B;
      const int w = int(t % d.W);
      t /= d.W;
      const int h = int(t % d.H);
      const int k = int(t / d.H);
      for (int tap = sub; tap < RS; tap += 8) {
        const int r = tap / d.S, s = tap - r * d.S;
        const __nv_bfloat16* ip =
            image + (((long long)(r + d.sw * w) * Hi + (s + d.sh * h)) * d.C) * d.B + b;
        const __nv_bfloat16* fp = filter + ((long long)k * RS + tap) * d.C;
        int c = 0;
        for (; c + 8 <= d.C; c += 8) {
          float x[8], f[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            x[j] = __bfloat162float(ip[(long long)(c + j) * d.B]);
            f[j] = __bfloat162float(fp[c + j]);
          }
#pragma unroll
          for (int j = 0; j < 8; ++j) acc = fmaf(x[j], f[j], acc);
        }
        for (; c < d.C; ++c)
          acc = fmaf(__bfloat162float(ip[(long long)c * d.B]), __bfloat162float(fp[c]), acc);
      }
    }
    acc += __shfl_xor_sync(0xffffffffu, acc, 4);
    acc += __shfl_xor_sync(0xffffffffu, acc, 2);
    acc += __shfl_xor_sync(0xffffffffu, acc, 1);
    if (valid && sub == 0) store_out(out + idx, acc);
  }
}

// Eq. 1 on arrays with explicit element strides per subscript (any layout: column-major storage,
// views of larger arrays, ...).  One thread per output element; consecutive threads run along the
// subscript of Out with the smallest stride, so that stores coalesce whatever the layout.
template <typename OutT>
__global__ void __launch_bounds__(256) cconv_simt_strided_kernel(const __nv_bfloat16* __restrict__ image,
                                                                 const __nv_bfloat16* __restrict__ filter,
                                                                 OutT* __restrict__ out, Dims d,
                                                                 StridedLayout L) {
  const long long total = (long long)d.K * d.H * d.W * d.B;
  // order[0] is the fastest-varying subscript of Out (0 = k, 1 = h, 2 = w, 3 = b)
  const int ext[4] = {d.K, d.H, d.W, d.B};
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    int sub[4];
    long long t = idx;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int a = L.order[j];
      sub[a] = int(t % ext[a]);
      t /= ext[a];
    }
    const int k = sub[0], h = sub[1], w = sub[2], b = sub[3];
    float acc = 0.f;
    for (int r = 0; r < d.R; ++r)
      for (int s = 0; s < d.S; ++s) {
        const __nv_bfloat16* ip = image + (long long)(r + d.sw * w) * L.image[0] +
                                  (long long)(s + d.sh * h) * L.image[1] + (long long)b * L.image[3];
        const __nv_bfloat16* fp = filter + (long long)k * L.filter[0] + (long long)r * L.filter[1] +
                                  (long long)s * L.filter[2];
        for (int c = 0; c < d.C; ++c)
          acc = fmaf(__bfloat162float(ip[(long long)c * L.image[2]]),
                     __bfloat162float(fp[(long long)c * L.filter[3]]), acc);
      }
    store_out(out + (long long)k * L.out[0] + (long long)h * L.out[1] + (long long)w * L.out[2] +
                  (long long)b * L.out[3],
              acc);
  }
}

cudaError_t launch_simt_strided(const void* image, const void* filter, void* out, bool out_f32,
                                const Dims& d, const StridedLayout& L, cudaStream_t stream) {
  const long long total = (long long)d.K * d.H * d.W * d.B;
  long long blocks = (total + 255) / 256;
  if (blocks > 148ll * 64) blocks = 148ll * 64;
  if (blocks < 1) blocks = 1;
  const __nv_bfloat16* im = static_cast<const __nv_bfloat16*>(image);
  const __nv_bfloat16* fl = static_cast<const __nv_bfloat16*>(filter);
  if (out_f32)
    cconv_simt_strided_kernel<float><<<unsigned(blocks), 256, 0, stream>>>(im, fl, static_cast<float*>(out), d, L);
  else
    cconv_simt_strided_kernel<__nv_bfloat16><<<unsigned(blocks), 256, 0, stream>>>(
        im, fl, static_cast<__nv_bfloat16*>(out), d, L);
  return cudaGetLastError();
}

cudaError_t launch_simt(const void* image, const void* filter, void* out, bool out_f32,
                        const Dims& d, cudaStream_t stream) {
  // Four out-channels per thread reuse each Image value four times; problems too small to fill
  // the SMs that way take one out-channel per thread and smaller blocks instead (more threads,
  // shorter dependent chains per thread).
  const long long outputs = (long long)d.K * d.H * d.W * d.B;
  const bool small = outputs < 148ll * 1024 * 4;
  const int KT = small ? 1 : 4;
  const long long total = (long long)((d.K + KT - 1) / KT) * d.H * d.W * d.B;
  const int threads = small ? 64 : 256;
  long long blocks = (total + threads - 1) / threads;
  if (blocks > 148ll * 64) blocks = 148ll * 64;
  if (blocks < 1) blocks = 1;
  const __nv_bfloat16* im = static_cast<const __nv_bfloat16*>(image);
  const __nv_bfloat16* fl = static_cast<const __nv_bfloat16*>(filter);
  // eight lanes per output while that still leaves the SMs room for every thread at once
  if (outputs * 8 <= 148ll * 2048 && d.R * d.S >= 4) {
    const long long tblocks = (outputs * 8 + 127) / 128;
    if (out_f32)
      cconv_simt_taps_kernel<float><<<(unsigned)tblocks, 128, 0, stream>>>(im, fl, static_cast<float*>(out), d);
    else
      cconv_simt_taps_kernel<__nv_bfloat16><<<(unsigned)tblocks, 128, 0, stream>>>(
          im, fl, static_cast<__nv_bfloat16*>(out), d);
    return cudaGetLastError();
  }
  if (small) {
    if (out_f32)
      cconv_simt_kernel<1, float><<<(unsigned)blocks, threads, 0, stream>>>(
          im, fl, static_cast<float*>(out), d);
    else
      cconv_simt_kernel<1, __nv_bfloat16><<<(unsigned)blocks, threads, 0, stream>>>(
          im, fl, static_cast<__nv_bfloat16*>(out), d);
  } else if (out_f32) {
    cconv_simt_kernel<4, float><<<(unsigned)blocks, threads, 0, stream>>>(
        im, fl, static_cast<float*>(out), d);
  } else {
    cconv_simt_kernel<4, __nv_bfloat16><<<(unsigned)blocks, threads, 0, stream>>>(
        im, fl, static_cast<__nv_bfloat16*>(out), d);
  }
  return cudaGetLastError();
}

namespace {

constexpr int kThreads = 288;
// warp 1: MMA issuer, warps 2-5: epilogue, warps 0 and 7: Image producers (TMA), warps 6 and 8:
// Filter producers (bulk copies).  One thread's asynchronous copies run one after the other
// (about 730 cycles each, whatever the size -- measured), so each ring is fed by two threads that
// take alternate stages; that keeps four copies in flight per CTA.
constexpr int kProducersPerRing = 2;

}  // namespace

// ------------------------------------------------------------------------------------------------
// Filter packing: [K][R][S][C] -> [k-tile][16-channel chunk][tap][128 x 16 block].
// Inside a block element (k, c) sits at ((k/8)*2 + c/8)*128 + (k%8)*16 + (c%8)*2 bytes: 8x8 "core
// matrices" of 128 contiguous bytes, K-major, so a block is a ready tcgen05 A operand
// (no swizzle, LBO = 128 B between the two channel halves, SBO = 256 B between 8-row groups).
// Rows k >= K and channels c >= C are zero.  One thread writes 16 bytes.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void pack_filter_slot(const __nv_bfloat16* __restrict__ filter,
                                                 uint4* __restrict__ packed, const Dims& d, int c16,
                                                 long long slot);

__global__ void __launch_bounds__(256)
    cconv_pack_filter_kernel(const __nv_bfloat16* __restrict__ filter, uint4* __restrict__ packed,
                             Dims d, int c16, long long slots) {
  // Let the convolution kernel (launched with programmatic stream serialization) start its set-up
  // and its Image copies while this kernel runs; it waits for our stores before reading them.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const long long slot = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (slot < slots) pack_filter_slot(filter, packed, d, c16, slot);
  // Launched with programmatic stream serialization (overlap_prev), this kernel may run while the
  // kernel in front of it is still executing; it then ends only after that kernel has, so that
  // "this kernel is complete" still implies "everything older in the stream is complete".
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

__device__ __forceinline__ void pack_filter_slot(const __nv_bfloat16* __restrict__ filter,
                                                 uint4* __restrict__ packed, const Dims& d, int c16,
                                                 long long slot) {
  const int RS = d.R * d.S;
  const int j = int(slot & 255);
  long long unit = slot >> 8;
  const int tap = int(unit % RS);
  unit /= RS;
  const int cc = int(unit % c16);
  const int kt = int(unit / c16);
  const int core = j >> 3, row = j & 7;
  const int k = kt * 128 + (core >> 1) * 8 + row;
  const int c0 = cc * 16 + (core & 1) * 8;
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  if (k < d.K && c0 < d.C) {
    const __nv_bfloat16* src = filter + ((long long)k * RS + tap) * d.C + c0;
    if ((d.C & 7) == 0) {
      v = *reinterpret_cast<const uint4*>(src);
    } else {
      unsigned short e[8];
#pragma unroll
      for (int i = 0; i < 8; ++i)
        e[i] = (c0 + i < d.C) ? *reinterpret_cast<const unsigned short*>(src + i) : (unsigned short)0;
      v.x = e[0] | (uint32_t(e[1]) << 16);
      v.y = e[2] | (uint32_t(e[3]) << 16);
      v.z = e[4] | (uint32_t(e[5]) << 16);
      v.w = e[6] | (uint32_t(e[7]) << 16);
    }
  }
  packed[slot] = v;
}

cudaError_t launch_pack_filter(const void* filter, void* packed, const Dims& d, int c16,
                               int tiles_k, bool overlap_prev, cudaStream_t stream) {
  const long long slots = 1ll * tiles_k * c16 * d.R * d.S * (kPackedBlockBytes / 16);
  const long long blocks = (slots + 255) / 256;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(blocks));
  cfg.blockDim = dim3(256);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = overlap_prev ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, cconv_pack_filter_kernel,
                            static_cast<const __nv_bfloat16*>(filter), static_cast<uint4*>(packed), d,
                            c16, slots);
}

// ------------------------------------------------------------------------------------------------
// MMA issuer role (warp 1 of cconv_halo_kernel).
// The whole warp walks the loops (descriptor arithmetic stays warp-uniform) and one fixed lane
// issues the tcgen05 instructions.  BH > 0 fixes b_h at compile time; TAPS = 9 / 1 unrolls 3x3 /
// 1x1 filters (0 = any R x S, offsets advanced arithmetically).
// ------------------------------------------------------------------------------------------------
struct MmaCtx {
  uint32_t bar_ifull, bar_iempty, bar_ffull, bar_fempty, bar_tfull, bar_tempty, bar_drain;
  uint32_t img_ring, filt_ring, tmem_base;
  volatile int* abort_flag;
  int* status;
  uint64_t limit;
  int tile_first, tile_step;  // this CTA's tiles: tile_first, tile_first + tile_step, ...
};

template <int BH>
__device__ __forceinline__ void issue_unit(bool leader, int bh, uint32_t d, uint32_t n_mma,
                                           uint64_t a_desc, uint32_t b_hi, uint32_t b_lo0,
                                           uint32_t b16, uint32_t hstep16, uint32_t idesc,
                                           uint32_t acc) {
  if constexpr (BH > 0) {
#pragma unroll
    for (int hh = 0; hh < BH; ++hh)
      umma_bf16_if(leader, d + uint32_t(hh) * n_mma, a_desc,
                   (uint64_t(b_hi) << 32) | (b_lo0 | (b16 + uint32_t(hh) * hstep16)), idesc, acc);
  } else {
    for (int hh = 0; hh < bh; ++hh, b16 += hstep16, d += n_mma)
      umma_bf16_if(leader, d, a_desc, (uint64_t(b_hi) << 32) | (b_lo0 | b16), idesc, acc);
  }
}

template <int BH, int TAPS>
__device__ __forceinline__ void mma_role(const HaloKernelParams& p, const MmaCtx& cx) {
  const int lane = threadIdx.x & 31;
  const bool leader = elect_one();
  uint32_t is = 0, iph = 0, fs = 0, fph = 0, abuf = 0, aph = 0;
  bool ok = true, first_tile = true;
  const int R = p.R, S = p.S, units = p.units_cta, units_per_img = p.units_per_img;
  const uint32_t slab16 = p.slab_bytes >> 4, row16 = uint32_t(p.halo_w) * slab16;
  uint32_t off9[9];  // 3x3: halo offset of tap (r, s) = r*3 + s, in 16 B units
#pragma unroll
  for (int t = 0; t < 9; ++t) off9[t] = uint32_t(t % 3) * row16 + uint32_t(t / 3) * slab16;
  // Descriptors differ only in their low word (start address >> 4, bits [0,14)); all
  // per-instruction arithmetic below is on 32-bit "address >> 4" quantities.
  const uint32_t a_lo0 = uint32_t(p.a_desc), a_hi = uint32_t(p.a_desc >> 32);
  const uint32_t b_lo0 = uint32_t(p.b_desc), b_hi = uint32_t(p.b_desc >> 32);
  const uint32_t hstep16 = uint32_t(p.sh * p.halo_w) * slab16;  // next output row
  const uint32_t kstep16 = p.b_kstep_bytes >> 4;
  const uint32_t img16 = p.img_stage_bytes >> 4, filt16 = p.filt_stage_bytes >> 4;
  // A descriptor holds address bits [4,18) of the CTA's own window.  In a cluster launch the
  // shared-memory addresses of CTA rank r carry r above bit 24; left in, those bits would run into
  // the descriptor's leading-byte-offset field.
  const uint32_t img_ring16 = (cx.img_ring >> 4) & 0x3FFFu, filt_ring16 = (cx.filt_ring >> 4) & 0x3FFFu;
  const uint32_t idesc = p.idesc, n_mma = uint32_t(p.n_mma);
  const uint32_t n_ist = uint32_t(p.i_stages), n_fst = uint32_t(p.f_stages);
  const int bh = p.bh, uf = p.uf;
  constexpr uint32_t kBlk16 = kPackedBlockBytes >> 4;
  for (int tile = cx.tile_first; tile < p.total_tiles; tile += cx.tile_step) {
    if (!mbar_wait_warp(cx.bar_tempty + 8u * abuf, aph ^ 1u, cx.abort_flag, cx.status,
                        kStatMmaWaitTmem, cx.limit))
      break;
    tc_fence_after();
    const uint32_t d_base = cx.tmem_base + abuf * uint32_t(p.acc_cols);
    uint32_t acc = 0;
    int f_left = 0, i_left = 0;   // units left in the current Filter / Image stage
    int sx = 0, tap_r = 0;
    uint32_t tap_off = 0, col_off = 0;  // halo offset of the current tap, in 16 B units
    uint32_t a16 = 0, img_kk16 = 0;
    int units_left = units;
    long long tw_i = 0, tw_f = 0;
    const long long tl0 = p.trace ? clock64() : 0;
    while (units_left > 0) {
      if (i_left == 0) {
        const long long w0 = p.trace ? clock64() : 0;
        if (!mbar_wait_warp(cx.bar_ifull + 8u * is, iph, cx.abort_flag, cx.status, kStatMmaWaitFull,
                            cx.limit)) {
          ok = false;
          break;
        }
        if (p.trace) tw_i += clock64() - w0;
        tc_fence_after();
        img_kk16 = img_ring16 + is * img16;
        i_left = units_left < units_per_img ? units_left : units_per_img;
      }
      if (f_left == 0) {
        const long long w0 = p.trace ? clock64() : 0;
        if (!mbar_wait_warp(cx.bar_ffull + 8u * fs, fph, cx.abort_flag, cx.status, kStatMmaWaitFull,
                            cx.limit)) {
          ok = false;
          break;
        }
        if (p.trace) tw_f += clock64() - w0;
        tc_fence_after();
        a16 = filt_ring16 + fs * filt16;
        f_left = units_left < uf ? units_left : uf;
      }
      if (first_tile && units_left == units && lane == 0 && p.trace)
        p.trace[blockIdx.x * 16 + 5] = globaltimer_ns();  // operands of the first MMA are resident
      // Issue every unit both resident stages cover, with no barrier work in between.
      // Descriptors are built by the whole warp (uniform values); only the issue is elected.
      const int n = i_left < f_left ? i_left : f_left;
      int issued = 0;
      if (TAPS == 9 && sx == 0 && tap_r == 0) {
        // whole 16-channel steps of a 3x3 filter, the nine tap offsets held in registers
        for (; issued + 9 <= n; issued += 9) {
          if constexpr (BH == 1) {
            umma_taps9_bh1(leader, d_base, a_lo0 | a16, a_hi, b_lo0 | img_kk16, b_hi, idesc, acc, off9);
          } else if constexpr (BH == 2) {
            umma_taps9_bh2(leader, d_base, a_lo0 | a16, a_hi, b_lo0 | img_kk16, b_hi, idesc, acc, off9,
                           hstep16, n_mma);
          } else {
#pragma unroll
            for (int t = 0; t < 9; ++t) {
              const uint64_t a_desc =
                  (uint64_t(a_hi) << 32) | (a_lo0 | (a16 + uint32_t(t) * kBlk16));
              issue_unit<BH>(leader, bh, d_base, n_mma, a_desc, b_hi, b_lo0, img_kk16 + off9[t],
                             hstep16, idesc, acc);
              acc = 1;
            }
          }
          acc = 1;
          a16 += 9u * kBlk16;
          img_kk16 += kstep16;
        }
      } else if (TAPS == 1) {
        // 1x1 filter: one unit per 16 channels, four at a time while both stages last
        if constexpr (BH == 1 || BH == 2) {
          for (; issued + 4 <= n; issued += 4) {
            if constexpr (BH == 1)
              umma_run4_bh1(leader, d_base, a_lo0 | a16, a_hi, b_lo0 | img_kk16, b_hi, idesc, acc,
                            kstep16);
            else
              umma_run4_bh2(leader, d_base, a_lo0 | a16, a_hi, b_lo0 | img_kk16, b_hi, idesc, acc,
                            kstep16, hstep16, n_mma);
            acc = 1;
            a16 += 4u * kBlk16;
            img_kk16 += 4u * kstep16;
          }
        }
        for (; issued < n; ++issued) {
          const uint64_t a_desc = (uint64_t(a_hi) << 32) | (a_lo0 | a16);
          issue_unit<BH>(leader, bh, d_base, n_mma, a_desc, b_hi, b_lo0, img_kk16, hstep16, idesc,
                         acc);
          acc = 1;
          a16 += kBlk16;
          img_kk16 += kstep16;
        }
      }
      for (; issued < n; ++issued) {
        if constexpr (TAPS == 0 && (BH == 1 || BH == 2)) {
          // R x 1 filters: four taps of the filter row (r .. r+3: one halo pixel apart)
          if (S == 1 && tap_r + 4 <= R && issued + 4 <= n) {
            if constexpr (BH == 1)
              umma_run4_bh1(leader, d_base, a_lo0 | a16, a_hi, b_lo0 | (img_kk16 + tap_off), b_hi, idesc,
                            acc, slab16);
            else
              umma_run4_bh2(leader, d_base, a_lo0 | a16, a_hi, b_lo0 | (img_kk16 + tap_off), b_hi, idesc,
                            acc, slab16, hstep16, n_mma);
            acc = 1;
            a16 += 4u * kBlk16;
            issued += 3;
            tap_r += 4;
            col_off += 4u * slab16;
            tap_off = col_off;
            if (tap_r == R) {
              tap_r = 0;
              col_off = 0;
              tap_off = 0;
              img_kk16 += kstep16;
            }
            continue;
          }
          // other filter sizes: four taps of one filter column (s, s+1, s+2, s+3: one halo row
          // apart) per straight-line block while the column and both stages last
          if (sx + 4 <= S && issued + 4 <= n) {
            if constexpr (BH == 1)
              umma_run4_bh1(leader, d_base, a_lo0 | a16, a_hi, b_lo0 | (img_kk16 + tap_off), b_hi, idesc,
                            acc, row16);
            else
              umma_run4_bh2(leader, d_base, a_lo0 | a16, a_hi, b_lo0 | (img_kk16 + tap_off), b_hi, idesc,
                            acc, row16, hstep16, n_mma);
            acc = 1;
            a16 += 4u * kBlk16;
            tap_off += 3u * row16;  // the common tail below adds the fourth step
            sx += 3;
            issued += 3;
          } else {
            const uint64_t a_desc = (uint64_t(a_hi) << 32) | (a_lo0 | a16);
            issue_unit<BH>(leader, bh, d_base, n_mma, a_desc, b_hi, b_lo0, img_kk16 + tap_off, hstep16,
                           idesc, acc);
            acc = 1;
            a16 += kBlk16;
          }
        } else {
          const uint64_t a_desc = (uint64_t(a_hi) << 32) | (a_lo0 | a16);
          issue_unit<BH>(leader, bh, d_base, n_mma, a_desc, b_hi, b_lo0, img_kk16 + tap_off, hstep16,
                         idesc, acc);
          acc = 1;
          a16 += kBlk16;
        }
        // next tap: one halo row down; after S rows, one pixel to the right; after R*S taps, the
        // next 16 channels of the same Image stage
        tap_off += row16;
        if (++sx == S) {
          sx = 0;
          col_off += slab16;
          tap_off = col_off;
          if (++tap_r == R) {
            tap_r = 0;
            col_off = 0;
            tap_off = 0;
            img_kk16 += kstep16;
          }
        }
      }
      i_left -= n;
      f_left -= n;
      units_left -= n;
      if (f_left == 0) {
        // the Filter stage is free once the MMAs issued so far have read it
        if (leader) umma_commit(cx.bar_fempty + 8u * fs);
        if (++fs == n_fst) {
          fs = 0;
          fph ^= 1u;
        }
      }
      if (i_left == 0) {
        if (leader) umma_commit(cx.bar_iempty + 8u * is);
        if (++is == n_ist) {
          is = 0;
          iph ^= 1u;
        }
      }
    }
    if (!ok) break;
    if (first_tile && lane == 0 && p.trace) {
      p.trace[blockIdx.x * 16 + 13] = (unsigned long long)tw_i;
      p.trace[blockIdx.x * 16 + 14] = (unsigned long long)tw_f;
      p.trace[blockIdx.x * 16 + 15] = (unsigned long long)(clock64() - tl0);
    }
    if (leader) umma_commit(cx.bar_tfull + 8u * abuf);  // accumulator complete
    if (first_tile && lane == 0 && p.trace) p.trace[blockIdx.x * 16 + 6] = globaltimer_ns();
    first_tile = false;
    if (++abuf == uint32_t(p.acc_bufs)) {
      abuf = 0;
      aph ^= 1u;
    }
  }
  // All MMAs must have retired before TMEM is released.
  if (lane == 0 && p.trace) p.trace[blockIdx.x * 16 + 7] = globaltimer_ns();
  if (leader) umma_commit(cx.bar_drain);
  const uint64_t t0 = globaltimer_ns();
  while (!mbar_try_wait(cx.bar_drain, 0)) {
    if (globaltimer_ns() - t0 > cx.limit) {
      atomicOr(cx.status, kStatDrainWait);
      break;
    }
  }
}

// 32 consecutive images of one (k, h, w): 64 B (bf16) or 128 B (fp32), written as whole 32-byte
// sectors.
// The same run cut off after `n` images (n a multiple of 8, as B is), in pieces of 8 images.
template <typename OutT>
__device__ __forceinline__ void store_run_partial(OutT* dst, const uint32_t (&v)[32], int n) {
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    if (8 * j < n) {
      if constexpr (sizeof(OutT) == 4) {
        st_global_v8(dst + 8 * j, v[8 * j], v[8 * j + 1], v[8 * j + 2], v[8 * j + 3], v[8 * j + 4],
                     v[8 * j + 5], v[8 * j + 6], v[8 * j + 7]);
      } else {
        *reinterpret_cast<uint4*>(dst + 8 * j) =
            make_uint4(pack_bf16x2(v[8 * j], v[8 * j + 1]), pack_bf16x2(v[8 * j + 2], v[8 * j + 3]),
                       pack_bf16x2(v[8 * j + 4], v[8 * j + 5]), pack_bf16x2(v[8 * j + 6], v[8 * j + 7]));
      }
    }
  }
}

template <typename OutT>
__device__ __forceinline__ void store_run32(OutT* dst, const uint32_t (&v)[32]) {
  if constexpr (sizeof(OutT) == 4) {
#pragma unroll
    for (int j = 0; j < 4; ++j)
      st_global_v8(dst + 8 * j, v[8 * j], v[8 * j + 1], v[8 * j + 2], v[8 * j + 3], v[8 * j + 4],
                   v[8 * j + 5], v[8 * j + 6], v[8 * j + 7]);
  } else {
#pragma unroll
    for (int j = 0; j < 2; ++j)
      st_global_v8(dst + 16 * j, pack_bf16x2(v[16 * j + 0], v[16 * j + 1]),
                   pack_bf16x2(v[16 * j + 2], v[16 * j + 3]),
                   pack_bf16x2(v[16 * j + 4], v[16 * j + 5]),
                   pack_bf16x2(v[16 * j + 6], v[16 * j + 7]),
                   pack_bf16x2(v[16 * j + 8], v[16 * j + 9]),
                   pack_bf16x2(v[16 * j + 10], v[16 * j + 11]),
                   pack_bf16x2(v[16 * j + 12], v[16 * j + 13]),
                   pack_bf16x2(v[16 * j + 14], v[16 * j + 15]));
  }
}

// ------------------------------------------------------------------------------------------------
// Halo-tile tcgen05 kernel
// ------------------------------------------------------------------------------------------------
// BH, TAPS: the issuer's compile-time shape (see mma_role).  One kernel per shape: the issuing loop
// is sensitive to the size of the code around it, so a launch carries only the loops it runs.
template <typename OutT, int BH, int TAPS, bool SB, bool S4>
__global__ void __launch_bounds__(kThreads, 1)
    cconv_halo_kernel(const __grid_constant__ CUtensorMap tm_image,
                      const uint8_t* __restrict__ packed_filter, OutT* __restrict__ out,
                      const HaloKernelParams p, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;  // swizzle atoms need 1024 B
  const uint32_t img_ring = smem0;
  const uint32_t filt_ring = img_ring + uint32_t(p.i_stages) * p.img_stage_bytes;
  const uint32_t bars = filt_ring + uint32_t(p.f_stages) * p.filt_stage_bytes;
  const uint32_t bar_ifull = bars;
  const uint32_t bar_iempty = bar_ifull + 8u * p.i_stages;
  const uint32_t bar_ffull = bar_iempty + 8u * p.i_stages;
  const uint32_t bar_fempty = bar_ffull + 8u * p.f_stages;
  const uint32_t bar_tfull = bar_fempty + 8u * p.f_stages;
  const uint32_t bar_tempty = bar_tfull + 16u;
  const uint32_t bar_drain = bar_tempty + 16u;
  const uint32_t slot_addr = bar_drain + 8u;
  const uint32_t bar_xchg = slot_addr + 8u;  // split launch: the peer's partial sums have arrived
  uint8_t* gen0 = smem_raw + (smem0 - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot =
      reinterpret_cast<volatile uint32_t*>(gen0 + (slot_addr - smem0));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen0 + (slot_addr + 4u - smem0));

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
#define CCONV_TRACE(slot)                                                        \
  do {                                                                           \
    if (p.trace) p.trace[blockIdx.x * 16 + (slot)] = globaltimer_ns();           \
  } while (0)

  if (threadIdx.x == 0) {
    CCONV_TRACE(0);
    for (int s = 0; s < p.i_stages; ++s) {
      mbar_init(bar_ifull + 8u * s, 1);
      mbar_init(bar_iempty + 8u * s, 1);
    }
    for (int s = 0; s < p.f_stages; ++s) {
      mbar_init(bar_ffull + 8u * s, 1);
      mbar_init(bar_fempty + 8u * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull + 8u * a, 1);
      mbar_init(bar_tempty + 8u * a, 4);  // one arrival per epilogue warp
    }
    mbar_init(bar_drain, 1);
    mbar_init(bar_xchg, 1);
    *abort_flag = 0;
    fence_barrier_init();
    // split launch: the peer will copy 128 rows of acc_cols/2 fp32 partial sums into this CTA
    // (four CTAs per tile: each of three peers 128 rows of acc_cols/4)
    if constexpr (S4) {
      mbar_arrive_expect_tx(bar_xchg, 3u * 128u * uint32_t(p.acc_cols >> 2) * 4u);
    } else {
      if (p.split > 1) mbar_arrive_expect_tx(bar_xchg, 128u * uint32_t(p.acc_cols >> 1) * 4u);
    }
    prefetch_tensormap(&tm_image);
  }
  if (warp == 1) {
    tmem_alloc(slot_addr, uint32_t(p.tmem_cols));
    tmem_relinquish();
    tc_fence_before();
  }
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint64_t limit = p.wait_limit_ns;
  const bool wide_rows = (size_t(p.B) * sizeof(OutT)) % 32 == 0;
  if (threadIdx.x == 0) CCONV_TRACE(1);
  // Persistent launch: CTA i takes tiles i, i + grid, ...  Split launch: the two CTAs of cluster i
  // take tile i once, rank r contracting the r-th half of the channels.
  const int crank = p.split > 1 ? int(cluster_ctarank()) : 0;
  const int tile_first = p.split > 1 ? int(blockIdx.x) / p.split : int(blockIdx.x);
  const int tile_step = p.split > 1 ? p.total_tiles : int(gridDim.x);

  // Ring positions advance by increment-and-wrap; a runtime division per stage would cost more
  // single-thread issue time than the stage's tensor-core work.
  if (warp == 0 || warp == 7) {
    // ===================== Image halo producers (TMA) =====================
    // Producer j of the ring issues the stages j, j+2, j+4, ... of the CTA's stage sequence.
    // (A one-stage ring is fed by the first producer alone: with parity waits a thread may be at
    // most one phase ahead of a barrier, and two producers sharing one slot would break that.)
    const uint32_t i_prod = p.i_stages >= 2 ? uint32_t(kProducersPerRing) : 1u;
    if (lane == 0 && ((warp == 0) ? 0u : 1u) < i_prod) {
      const uint32_t me = (warp == 0) ? 0u : 1u;
      const uint32_t n_st = uint32_t(p.i_stages);
      uint32_t seq = 0;             // stages of this CTA so far, both producers count all of them
      uint32_t s = 0, ph = 0;       // ring slot and phase of stage `seq`
      bool ok = true;
      const int cchunks = p.cchunks_cta;
      const int c_first = crank * p.cchunks_cta * p.bc;
      // This kernel may start while the convolution of the call in front of it is still running
      // (that kernel is the only kind that lets its successors start early).  If that call's Out
      // overlaps this call's Image -- the host checks -- nothing is read before it is complete.
      if (p.image_wait) asm volatile("griddepcontrol.wait;" ::: "memory");
      for (int tile = tile_first; ok && tile < p.total_tiles; tile += tile_step) {
        int t = tile / p.tiles_k;
        const int bt = t % p.tiles_b; t /= p.tiles_b;
        const int wt = t % p.tiles_w; t /= p.tiles_w;
        const int ht = t;
        const int b0 = bt * p.bb;
        const int x0 = wt * p.bw * p.sw, y0 = (p.h0 + ht * p.bh) * p.sh;
        for (int cc = 0, c0 = c_first; cc < cchunks; ++cc, c0 += p.bc, ++seq) {
          if ((seq & (i_prod - 1u)) == me) {
            if (!mbar_wait(bar_iempty + 8u * s, ph ^ 1u, abort_flag, status, kStatProducerWait,
                           limit)) {
              ok = false;
              break;
            }
            const uint32_t full = bar_ifull + 8u * s;
            mbar_arrive_expect_tx(full, p.img_stage_bytes);
            tma_load_4d(img_ring + s * p.img_stage_bytes, &tm_image, b0, c0, x0, y0, full);
            if (seq == 0) CCONV_TRACE(2);
          }
          if (++s == n_st) {
            s = 0;
            ph ^= 1u;
          }
        }
      }
      if (me == 0) CCONV_TRACE(3);
      drain_ring(bar_ifull, seq, n_st, status, limit);
    }
  } else if (warp == 6 || warp == 8) {
    // ===================== Filter producers (bulk copies of packed blocks) =====================
    const uint32_t f_prod = p.f_stages >= 2 ? uint32_t(kProducersPerRing) : 1u;
    if (lane == 0 && ((warp == 6) ? 0u : 1u) < f_prod) {
      const uint32_t me = (warp == 6) ? 0u : 1u;
      const uint32_t n_st = uint32_t(p.f_stages);
      uint32_t seq = 0, s = 0, ph = 0;
      bool ok = true;
      // The packed Filter is written by the kernel launched just before this one.  Once that
      // kernel is complete (and with it everything older in the stream), the next packing kernel
      // may start: it writes the other scratch buffer while this kernel runs.
      // (A tail launch starts only after every CTA of the main launch has passed this point, so
      // the packed Filter is known to be complete; it waits at its end instead, see below.)
      if (!p.tail) asm volatile("griddepcontrol.wait;" ::: "memory");
      if (me == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
      for (int tile = tile_first; ok && tile < p.total_tiles; tile += tile_step) {
        const int kt = tile % p.tiles_k;
        const uint8_t* src = packed_filter +
                             ((size_t)kt * p.units + (size_t)crank * p.units_cta) * kPackedBlockBytes;
        for (int left = p.units_cta; left > 0; left -= p.uf, ++seq) {
          const uint32_t bytes = uint32_t(left < p.uf ? left : p.uf) * kPackedBlockBytes;
          if ((seq & (f_prod - 1u)) == me) {
            if (!mbar_wait(bar_fempty + 8u * s, ph ^ 1u, abort_flag, status, kStatFilterWait,
                           limit)) {
              ok = false;
              break;
            }
            const uint32_t full = bar_ffull + 8u * s;
            mbar_arrive_expect_tx(full, bytes);
            bulk_load(filt_ring + s * p.filt_stage_bytes, src, bytes, full);
          }
          src += bytes;
          if (++s == n_st) {
            s = 0;
            ph ^= 1u;
          }
        }
      }
      if (me == 0) CCONV_TRACE(4);
      drain_ring(bar_ffull, seq, n_st, status, limit);
    }
  } else if (warp == 1) {
    // ===================== MMA issuer =====================
    const MmaCtx cx{bar_ifull, bar_iempty, bar_ffull, bar_fempty, bar_tfull, bar_tempty, bar_drain,
                    img_ring, filt_ring, tmem_base, abort_flag, status, limit, tile_first, tile_step};
    mma_role<BH, TAPS>(p, cx);
  } else if (p.split == 1) {
    // ===================== epilogue: TMEM -> registers -> Out =====================
    const int q = warp & 3;  // this warp may touch TMEM lanes [32q, 32q+32)
    uint32_t abuf = 0, aph = 0;
    bool first_tile = true;
    const int chunks = p.bb / 32;
    for (int tile = blockIdx.x; tile < p.total_tiles; tile += gridDim.x) {
      int t = tile;
      const int kt = t % p.tiles_k; t /= p.tiles_k;
      const int bt = t % p.tiles_b; t /= p.tiles_b;
      const int wt = t % p.tiles_w; t /= p.tiles_w;
      const int ht = t;
      const int k = kt * 128 + q * 32 + lane;
      const int b0 = bt * p.bb;
      if (!mbar_wait_warp(bar_tfull + 8u * abuf, aph, abort_flag, status, kStatEpilogueWait, limit))
        break;
      tc_fence_after();
      if (first_tile && threadIdx.x == 64) CCONV_TRACE(8);
      const uint32_t t_base = tmem_base + (uint32_t(q * 32) << 16) + abuf * uint32_t(p.acc_cols);
      if constexpr (SB) {
        // batch blocks of 16 or 8 images: 32 accumulator columns hold 2 or 4 pixels
        const int per = 32 / p.bb;  // pixels per 32 columns
        for (int hh = 0; hh < p.bh; ++hh) {
          const int h = p.h0 + ht * p.bh + hh;
          for (int c0 = 0; c0 < p.n_mma; c0 += 32) {
            uint32_t v[32];
            tmem_ld_32x32b_x32(t_base + uint32_t(hh * p.n_mma + c0), v);
            tmem_ld_wait();
            const int ww0 = c0 / p.bb;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              if (j >= per) break;
              const int w = wt * p.bw + ww0 + j;
              if (!(k < p.K && h < p.H && w < p.W && ww0 + j < p.bw)) continue;
              OutT* dst = out + (((long long)k * p.H + h) * p.W + w) * p.B + b0;
              const int nb = p.B - b0;  // images inside the batch (a multiple of 8)
              // the pixel's images are v[j*bb .. j*bb + bb): 8 (per = 4) or 16 (per = 2) values
#pragma unroll
              for (int g = 0; g < 2; ++g) {
                const int first = (per == 4 ? j * 8 : j * 16 + g * 8);
                if ((per == 4 && g == 1) || g * 8 >= nb) continue;
                OutT* d8 = dst + g * 8;
                if constexpr (sizeof(OutT) == 4) {
                  *reinterpret_cast<uint4*>(d8) = make_uint4(v[first], v[first + 1], v[first + 2], v[first + 3]);
                  *reinterpret_cast<uint4*>(d8 + 4) = make_uint4(v[first + 4], v[first + 5], v[first + 6], v[first + 7]);
                } else {
                  *reinterpret_cast<uint4*>(d8) =
                      make_uint4(pack_bf16x2(v[first], v[first + 1]), pack_bf16x2(v[first + 2], v[first + 3]),
                                 pack_bf16x2(v[first + 4], v[first + 5]), pack_bf16x2(v[first + 6], v[first + 7]));
                }
              }
            }
          }
        }
      } else
      for (int hh = 0; hh < p.bh; ++hh) {
        const int h = p.h0 + ht * p.bh + hh;
        for (int ww = 0; ww < p.bw; ++ww) {
          const int w = wt * p.bw + ww;
          const bool valid = (k < p.K) && (h < p.H) && (w < p.W);
          for (int ch = 0; ch < chunks; ++ch) {
            uint32_t v[32];
            tmem_ld_32x32b_x32(t_base + uint32_t(hh * p.n_mma + ww * p.bb + ch * 32), v);
            tmem_ld_wait();
            if (valid) {
              OutT* dst = out + (((long long)k * p.H + h) * p.W + w) * p.B + b0 + ch * 32;
              const int nb = p.B - (b0 + ch * 32);  // images left in the batch (block padded past B)
              // 32-byte stores need rows of Out that are multiples of 32 bytes (bf16: B % 16 == 0)
              if (nb >= 32 && wide_rows) store_run32(dst, v);
              else if (nb > 0) store_run_partial(dst, v, nb < 32 ? nb : 32);
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty + 8u * abuf);
      if (first_tile && threadIdx.x == 64) CCONV_TRACE(9);
      first_tile = false;
      if (++abuf == uint32_t(p.acc_bufs)) {
        abuf = 0;
        aph ^= 1u;
      }
    }
    if (threadIdx.x == 64) CCONV_TRACE(10);
  }

  // ===================== split launch: exchange partial sums, then store =====================
  // The 2 or 4 CTAs of the cluster each hold a full 128 x acc_cols accumulator over their share of
  // the channels.  Rank r owns the columns [r*half, (r+1)*half), half = acc_cols / split: it receives
  // the peers' partial sums for them in its own shared memory (the rings are idle by then), adds its
  // own and stores.  The partial sums travel as asynchronous shared-memory-to-shared-memory copies
  // (one per epilogue warp and peer), credited to the receiver's mbarrier; single remote stores from
  // 32 lanes to 32 different rows were measured 5x slower.  The order of the additions is fixed
  // (own, then the slices in slot order), so results are reproducible run to run.
  // Every thread of every CTA reaches both cluster barriers, whatever happened before.
  if (p.split > 1) {
    const bool epi = warp >= 2 && warp <= 5;
    const int q = warp & 3;
    bool acc_ok = true;
    if (epi) {
      acc_ok = mbar_wait_warp(bar_tfull, 0, abort_flag, status, kStatEpilogueWait, limit);
      acc_ok = __all_sync(0xffffffffu, acc_ok);  // the TMEM loads below need a uniform decision
      tc_fence_after();
    }
    __syncwarp();
    cluster_sync_all();  // both accumulators complete: neither CTA's rings are read any more
    if (threadIdx.x == 64) CCONV_TRACE(8);
    if constexpr (S4) {
      const int nsp = p.split;                          // CTAs per tile: 2 or 4
      const int half = p.acc_cols / nsp;                // columns per owner, a multiple of 32
      const uint32_t row_bytes = uint32_t(half) * 4u;   // one accumulator row of fp32 partial sums
      const uint32_t t_lane = tmem_base + (uint32_t(q * 32) << 16);
      // Incoming area: one slice of 128 rows per peer, row L = 32q + lane of slice j at
      // smem0 + (j*128 + L)*row_bytes; the outgoing staging slices right behind them, same layout.
      // The sender of rank s writes slice (s - r - 1) mod nsp of the receiver of rank r.  16-byte
      // chunk c of a row is stored at chunk c ^ (lane & 7), so that the eight lanes of a store phase
      // hit eight different bank groups.
      const uint32_t slice_bytes = 128u * row_bytes;
      const uint32_t my_row = uint32_t(q * 32 + lane) * row_bytes;
      const uint32_t out_area = smem0 + uint32_t(nsp - 1) * slice_bytes;
      const uint32_t x7 = uint32_t(lane & 7);
      if (epi && acc_ok) {
        for (int j = 1; j < nsp; ++j) {
          const int peer = (crank + j) % nsp;           // its slot for this CTA's slice is nsp - 1 - j ...
          const uint32_t slot_there = uint32_t(nsp - 1 - j);  // ... = (crank - peer - 1) mod nsp
          const uint32_t out_row = out_area + uint32_t(j - 1) * slice_bytes + my_row;
          const int col0 = peer * half;                 // the peer's columns
          for (int g = 0; g < half; g += 32) {
            uint32_t v[32];
            tmem_ld_32x32b_x32(t_lane + uint32_t(col0 + g), v);
            tmem_ld_wait();
  #pragma unroll
            for (int c = 0; c < 8; ++c)
              st_shared_v4(out_row + ((uint32_t(g / 4 + c) ^ x7) << 4), v[4 * c], v[4 * c + 1],
                           v[4 * c + 2], v[4 * c + 3]);
          }
          fence_proxy_async_shared();  // the copy engine reads these generic-proxy writes
          __syncwarp();
          if (lane == 0) {
            const uint32_t warp_rows = uint32_t(q * 32) * row_bytes;
            bulk_copy_to_peer(cluster_map_shared(smem0 + slot_there * slice_bytes + warp_rows, uint32_t(peer)),
                              out_area + uint32_t(j - 1) * slice_bytes + warp_rows, 32u * row_bytes,
                              cluster_map_shared(bar_xchg, uint32_t(peer)));
          }
        }
      }
      if (threadIdx.x == 64) CCONV_TRACE(9);
      if (epi && acc_ok) {
        acc_ok = mbar_wait_warp(bar_xchg, 0, abort_flag, status, kStatEpilogueWait, limit);
        acc_ok = __all_sync(0xffffffffu, acc_ok);
      }
      if (threadIdx.x == 64) CCONV_TRACE(12);
      if (epi && acc_ok) {
        const int tile = tile_first;
        int t = tile;
        const int kt = t % p.tiles_k; t /= p.tiles_k;
        const int bt = t % p.tiles_b; t /= p.tiles_b;
        const int wt = t % p.tiles_w; t /= p.tiles_w;
        const int ht = t;
        const int k = kt * 128 + q * 32 + lane;
        const int col0 = crank * half;
        for (int g = 0; g < half; g += 32) {
          uint32_t v[32];
          tmem_ld_32x32b_x32(t_lane + uint32_t(col0 + g), v);
          tmem_ld_wait();
          for (int j = 0; j < nsp - 1; ++j) {
            const uint32_t in_row = smem0 + uint32_t(j) * slice_bytes + my_row;
  #pragma unroll
            for (int c = 0; c < 8; ++c) {
              uint32_t a0, a1, a2, a3;
              ld_shared_v4(in_row + ((uint32_t(g / 4 + c) ^ x7) << 4), a0, a1, a2, a3);
              v[4 * c] = __float_as_uint(__uint_as_float(v[4 * c]) + __uint_as_float(a0));
              v[4 * c + 1] = __float_as_uint(__uint_as_float(v[4 * c + 1]) + __uint_as_float(a1));
              v[4 * c + 2] = __float_as_uint(__uint_as_float(v[4 * c + 2]) + __uint_as_float(a2));
              v[4 * c + 3] = __float_as_uint(__uint_as_float(v[4 * c + 3]) + __uint_as_float(a3));
            }
          }
          if constexpr (SB) {
            // column -> (output row, 2 or 4 pixels, 16 or 8 images each), as in the epilogue above
            const int col = col0 + g;
            const int hh = col / p.n_mma, rem = col - hh * p.n_mma;
            const int h = p.h0 + ht * p.bh + hh;
            const int per = 32 / p.bb;
            const int ww0 = rem / p.bb;
  #pragma unroll
            for (int j = 0; j < 4; ++j) {
              if (j >= per) break;
              const int w = wt * p.bw + ww0 + j;
              if (!(k < p.K && h < p.H && w < p.W && ww0 + j < p.bw)) continue;
              OutT* dst = out + (((long long)k * p.H + h) * p.W + w) * p.B + bt * p.bb;
              const int nb = p.B - bt * p.bb;
  #pragma unroll
              for (int g8 = 0; g8 < 2; ++g8) {
                const int first = (per == 4 ? j * 8 : j * 16 + g8 * 8);
                if ((per == 4 && g8 == 1) || g8 * 8 >= nb) continue;
                OutT* d8 = dst + g8 * 8;
                if constexpr (sizeof(OutT) == 4) {
                  *reinterpret_cast<uint4*>(d8) = make_uint4(v[first], v[first + 1], v[first + 2], v[first + 3]);
                  *reinterpret_cast<uint4*>(d8 + 4) = make_uint4(v[first + 4], v[first + 5], v[first + 6], v[first + 7]);
                } else {
                  *reinterpret_cast<uint4*>(d8) =
                      make_uint4(pack_bf16x2(v[first], v[first + 1]), pack_bf16x2(v[first + 2], v[first + 3]),
                                 pack_bf16x2(v[first + 4], v[first + 5]), pack_bf16x2(v[first + 6], v[first + 7]));
                }
              }
            }
          } else {
            // column -> (output row, pixel, 32 images)
            const int col = col0 + g;
            const int hh = col / p.n_mma, rem = col - hh * p.n_mma;
            const int ww = rem / p.bb, ch = (rem - ww * p.bb) >> 5;
            const int h = p.h0 + ht * p.bh + hh, w = wt * p.bw + ww;
            if (k < p.K && h < p.H && w < p.W) {
              OutT* dst = out + (((long long)k * p.H + h) * p.W + w) * p.B + bt * p.bb + ch * 32;
              const int nb = p.B - (bt * p.bb + ch * 32);
              if (nb >= 32 && wide_rows) store_run32(dst, v);
              else if (nb > 0) store_run_partial(dst, v, nb < 32 ? nb : 32);
            }
          }
        }
      }
    } else {
      const int half = p.acc_cols >> 1;                 // columns per owner, a multiple of 32
      const uint32_t row_bytes = uint32_t(half) * 4u;   // one accumulator row of fp32 partial sums
      const uint32_t t_lane = tmem_base + (uint32_t(q * 32) << 16);
      // Incoming area: row L = 32q + lane at smem0 + L*row_bytes; outgoing staging area right behind
      // it, same layout.  16-byte chunk c of a row is stored at chunk c ^ (lane & 7), so that the
      // eight lanes of a store phase hit eight different bank groups.
      const uint32_t in_row = smem0 + uint32_t(q * 32 + lane) * row_bytes;
      const uint32_t out_area = smem0 + 128u * row_bytes;
      const uint32_t out_row = out_area + uint32_t(q * 32 + lane) * row_bytes;
      const uint32_t x7 = uint32_t(lane & 7);
      if (epi && acc_ok) {
        const int col0 = (crank ^ 1) * half;  // the peer's columns
        for (int g = 0; g < half; g += 32) {
          uint32_t v[32];
          tmem_ld_32x32b_x32(t_lane + uint32_t(col0 + g), v);
          tmem_ld_wait();
  #pragma unroll
          for (int c = 0; c < 8; ++c)
            st_shared_v4(out_row + ((uint32_t(g / 4 + c) ^ x7) << 4), v[4 * c], v[4 * c + 1],
                         v[4 * c + 2], v[4 * c + 3]);
        }
        fence_proxy_async_shared();  // the copy engine reads these generic-proxy writes
        __syncwarp();
        if (lane == 0) {
          const uint32_t peer = uint32_t(crank ^ 1);
          const uint32_t warp_rows = uint32_t(q * 32) * row_bytes;
          bulk_copy_to_peer(cluster_map_shared(smem0 + warp_rows, peer), out_area + warp_rows,
                            32u * row_bytes, cluster_map_shared(bar_xchg, peer));
        }
      }
      if (threadIdx.x == 64) CCONV_TRACE(9);
      if (epi && acc_ok) {
        acc_ok = mbar_wait_warp(bar_xchg, 0, abort_flag, status, kStatEpilogueWait, limit);
        acc_ok = __all_sync(0xffffffffu, acc_ok);
      }
      if (threadIdx.x == 64) CCONV_TRACE(12);
      if (epi && acc_ok) {
        const int tile = tile_first;
        int t = tile;
        const int kt = t % p.tiles_k; t /= p.tiles_k;
        const int bt = t % p.tiles_b; t /= p.tiles_b;
        const int wt = t % p.tiles_w; t /= p.tiles_w;
        const int ht = t;
        const int k = kt * 128 + q * 32 + lane;
        const int col0 = crank * half;
        for (int g = 0; g < half; g += 32) {
          uint32_t v[32];
          tmem_ld_32x32b_x32(t_lane + uint32_t(col0 + g), v);
          tmem_ld_wait();
  #pragma unroll
          for (int c = 0; c < 8; ++c) {
            uint32_t a0, a1, a2, a3;
            ld_shared_v4(in_row + ((uint32_t(g / 4 + c) ^ x7) << 4), a0, a1, a2, a3);
            v[4 * c] = __float_as_uint(__uint_as_float(v[4 * c]) + __uint_as_float(a0));
            v[4 * c + 1] = __float_as_uint(__uint_as_float(v[4 * c + 1]) + __uint_as_float(a1));
            v[4 * c + 2] = __float_as_uint(__uint_as_float(v[4 * c + 2]) + __uint_as_float(a2));
            v[4 * c + 3] = __float_as_uint(__uint_as_float(v[4 * c + 3]) + __uint_as_float(a3));
          }
          if constexpr (SB) {
            // column -> (output row, 2 or 4 pixels, 16 or 8 images each), as in the epilogue above
            const int col = col0 + g;
            const int hh = col / p.n_mma, rem = col - hh * p.n_mma;
            const int h = p.h0 + ht * p.bh + hh;
            const int per = 32 / p.bb;
            const int ww0 = rem / p.bb;
  #pragma unroll
            for (int j = 0; j < 4; ++j) {
              if (j >= per) break;
              const int w = wt * p.bw + ww0 + j;
              if (!(k < p.K && h < p.H && w < p.W && ww0 + j < p.bw)) continue;
              OutT* dst = out + (((long long)k * p.H + h) * p.W + w) * p.B + bt * p.bb;
              const int nb = p.B - bt * p.bb;
  #pragma unroll
              for (int g8 = 0; g8 < 2; ++g8) {
                const int first = (per == 4 ? j * 8 : j * 16 + g8 * 8);
                if ((per == 4 && g8 == 1) || g8 * 8 >= nb) continue;
                OutT* d8 = dst + g8 * 8;
                if constexpr (sizeof(OutT) == 4) {
                  *reinterpret_cast<uint4*>(d8) = make_uint4(v[first], v[first + 1], v[first + 2], v[first + 3]);
                  *reinterpret_cast<uint4*>(d8 + 4) = make_uint4(v[first + 4], v[first + 5], v[first + 6], v[first + 7]);
                } else {
                  *reinterpret_cast<uint4*>(d8) =
                      make_uint4(pack_bf16x2(v[first], v[first + 1]), pack_bf16x2(v[first + 2], v[first + 3]),
                                 pack_bf16x2(v[first + 4], v[first + 5]), pack_bf16x2(v[first + 6], v[first + 7]));
                }
              }
            }
          } else {
            // column -> (output row, pixel, 32 images)
            const int col = col0 + g;
            const int hh = col / p.n_mma, rem = col - hh * p.n_mma;
            const int ww = rem / p.bb, ch = (rem - ww * p.bb) >> 5;
            const int h = p.h0 + ht * p.bh + hh, w = wt * p.bw + ww;
            if (k < p.K && h < p.H && w < p.W) {
              OutT* dst = out + (((long long)k * p.H + h) * p.W + w) * p.B + bt * p.bb + ch * 32;
              const int nb = p.B - (bt * p.bb + ch * 32);
              if (nb >= 32 && wide_rows) store_run32(dst, v);
              else if (nb > 0) store_run_partial(dst, v, nb < 32 ? nb : 32);
            }
          }
        }
      }
    }
    if (threadIdx.x == 64) CCONV_TRACE(10);
    // Neither CTA may leave while a copy still reads its staging area or writes its incoming
    // area: both have consumed their incoming rows only past this barrier.
    __syncwarp();
    cluster_sync_all();
  }

  // ===================== teardown =====================
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, uint32_t(p.tmem_cols));
  }
  // A tail launch runs beside the main launch of the same call; it ends only after that one has,
  // so that "the last kernel of a call is complete" implies that the whole call is.
  if (p.tail && threadIdx.x == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
  if (threadIdx.x == 0) CCONV_TRACE(11);
#undef CCONV_TRACE
}

namespace {

// Straight-line issue code for the common shapes (a loop branch costs a lone warp ~20 cycles):
// b_h in {1,2} and 1x1 / 3x3 filters; everything else takes the generic loops.
template <typename OutT>
using HaloFn = void (*)(CUtensorMap, const uint8_t*, OutT*, HaloKernelParams, int*);

template <typename OutT, bool SB>
HaloFn<OutT> halo_fn_sb(int R, int S, int bh) {
  const int b = bh == 1 ? 1 : bh == 2 ? 2 : 0;
  if (R == 3 && S == 3)
    return b == 1 ? cconv_halo_kernel<OutT, 1, 9, SB, false> : b == 2 ? cconv_halo_kernel<OutT, 2, 9, SB, false>
                                                                      : cconv_halo_kernel<OutT, 0, 9, SB, false>;
  if (R * S == 1)
    return b == 1 ? cconv_halo_kernel<OutT, 1, 1, SB, false> : b == 2 ? cconv_halo_kernel<OutT, 2, 1, SB, false>
                                                                      : cconv_halo_kernel<OutT, 0, 1, SB, false>;
  return b == 1 ? cconv_halo_kernel<OutT, 1, 0, SB, false> : b == 2 ? cconv_halo_kernel<OutT, 2, 0, SB, false>
                                                                    : cconv_halo_kernel<OutT, 0, 0, SB, false>;
}

// Four CTAs per tile: 3x3 filters unrolled, every other filter size (1x1 included) on the generic
// tap loop.
template <typename OutT, bool SB>
HaloFn<OutT> halo_fn_s4(int R, int S, int bh) {
  const int b = bh == 1 ? 1 : bh == 2 ? 2 : 0;
  if (R == 3 && S == 3)
    return b == 1 ? cconv_halo_kernel<OutT, 1, 9, SB, true> : b == 2 ? cconv_halo_kernel<OutT, 2, 9, SB, true>
                                                                     : cconv_halo_kernel<OutT, 0, 9, SB, true>;
  return b == 1 ? cconv_halo_kernel<OutT, 1, 0, SB, true> : b == 2 ? cconv_halo_kernel<OutT, 2, 0, SB, true>
                                                                   : cconv_halo_kernel<OutT, 0, 0, SB, true>;
}

// One kernel per issuer shape (b_h, filter size), per batch-block class (32/64 images, or 8/16
// with its own epilogue) and for the four-CTA exchange, so that no instantiation carries another
// one's code.
template <typename OutT>
HaloFn<OutT> halo_fn(int R, int S, int bh, int bb, int split) {
  if (split == 4) return bb < 32 ? halo_fn_s4<OutT, true>(R, S, bh) : halo_fn_s4<OutT, false>(R, S, bh);
  return bb < 32 ? halo_fn_sb<OutT, true>(R, S, bh) : halo_fn_sb<OutT, false>(R, S, bh);
}

template <typename OutT>
cudaError_t prepare_all(int smem_bytes) {
  const int shapes[9][3] = {{3, 3, 1}, {3, 3, 2}, {3, 3, 3}, {1, 1, 1}, {1, 1, 2},
                            {1, 1, 3}, {5, 5, 1}, {5, 5, 2}, {5, 5, 3}};
  for (const auto& sh : shapes) {
    for (int bb : {64, 8}) {
      for (int split : {1, 4}) {
        cudaError_t e = cudaFuncSetAttribute(halo_fn<OutT>(sh[0], sh[1], sh[2], bb, split),
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
        if (e != cudaSuccess) return e;
      }
    }
  }
  return cudaSuccess;
}

}  // namespace

// The attribute is a per-kernel ceiling, and the value set last wins: several plans (and the
// non-allocating entry point) share these kernels, so it is always raised to the device's limit,
// never to one plan's need (a second plan with a smaller tile would otherwise break the first).
cudaError_t halo_kernel_prepare(int smem_bytes) {
  int dev = 0, cap = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&cap, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e != cudaSuccess) return e;
  if (smem_bytes > cap) return cudaErrorInvalidValue;
  e = prepare_all<__nv_bfloat16>(cap);
  if (e != cudaSuccess) return e;
  return prepare_all<float>(cap);
}

cudaError_t launch_halo(const CUtensorMap& tm_image, const void* packed_filter, void* out,
                        bool out_f32, const HaloKernelParams& p, int grid, int smem_bytes,
                        int* status, cudaStream_t stream) {
  const uint8_t* pf = static_cast<const uint8_t*>(packed_filter);
  // Programmatic dependent launch: this kernel may begin while the Filter-packing kernel in front
  // of it is still running; only its Filter producers wait for that kernel's results.
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(grid));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = size_t(smem_bytes);
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (p.split > 1) {
    // the grid is tiles x split CTAs; consecutive CTAs form the cluster that shares a tile
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = unsigned(p.split);
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
  }
  if (out_f32)
    return cudaLaunchKernelEx(&cfg, halo_fn<float>(p.R, p.S, p.bh, p.bb, p.split), tm_image, pf,
                              static_cast<float*>(out), p, status);
  return cudaLaunchKernelEx(&cfg, halo_fn<__nv_bfloat16>(p.R, p.S, p.bh, p.bb, p.split), tm_image, pf,
                            static_cast<__nv_bfloat16*>(out), p, status);
}

}  // namespace cconv
