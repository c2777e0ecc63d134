// sm_100a kernels for the seven-nested-loop CNN (Eq. 1, Section 2):
//   Out(k,h,w,b) = sum_{c,r,s} Image(r+sw*w, s+sh*h, c, b) * Filter(k,r,s,c)
// Image [Wi][Hi][C][B], Filter [K][R][S][C], Out [K][H][W][B], bf16, last subscript fastest.
//
// cconv_halo_kernel realises the blocked loop nest of Section 5 on one SM:
//   outer loops  {b,k,w,h}_1 : the persistent tile loop (k innermost so CTAs that run at the same
//                              time share one Image block in L2),
//   outer loop   c_1         : the shared-memory ring, one stage per block of b_c channels,
//   inner loops  {b,k,w,h,c,r,s}_2 : tcgen05.mma instructions.  One stage holds the Image block
//                              b_b x b_c x (sw(b_w-1)+R) x (sh(b_h-1)+S) -- the halo tile -- and the
//                              Filter block b_k x R x S x b_c.  Every (r,s) tap reads the SAME
//                              resident halo tile through a shifted shared-memory descriptor, so
//                              an Image word fetched once serves all R*S taps and all b_k channels
//                              (the reuse behind the fifth term of Theorem 1).
// As a GEMM: D[k][n=(h,w,b)] += A_rs[k][c] * B_rs[c][n]; A = Filter slab, K-major (c contiguous);
// B = Image halo view, MN-major (b contiguous).  Accumulators live in TMEM (fp32).
#include <cuda_bf16.h>

#include "kernels.h"

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

cudaError_t launch_simt(const void* image, const void* filter, void* out, bool out_f32,
                        const Dims& d, cudaStream_t stream) {
  constexpr int KT = 4;
  const long long total = (long long)((d.K + KT - 1) / KT) * d.H * d.W * d.B;
  const int threads = 256;
  long long blocks = (total + threads - 1) / threads;
  if (blocks > 148ll * 64) blocks = 148ll * 64;
  if (blocks < 1) blocks = 1;
  const __nv_bfloat16* im = static_cast<const __nv_bfloat16*>(image);
  const __nv_bfloat16* fl = static_cast<const __nv_bfloat16*>(filter);
  if (out_f32)
    cconv_simt_kernel<KT, float><<<(unsigned)blocks, threads, 0, stream>>>(
        im, fl, static_cast<float*>(out), d);
  else
    cconv_simt_kernel<KT, __nv_bfloat16><<<(unsigned)blocks, threads, 0, stream>>>(
        im, fl, static_cast<__nv_bfloat16*>(out), d);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// PTX wrappers (sm_100a)
// ------------------------------------------------------------------------------------------------
namespace {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ uint64_t globaltimer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred P1;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 P1, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, P1;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up when another role raised the CTA's abort flag or when the time limit
// passes; on expiry it records `code` in the global status word and raises the abort flag.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int* status, int code, uint64_t limit_ns) {
  uint64_t t0 = 0;
  for (uint32_t i = 0;; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if ((i & 63u) == 63u) {
      const uint64_t t = globaltimer_ns();
      if (t0 == 0) {
        t0 = t;
      } else if (t - t0 > limit_ns) {
        *abort_flag = 1;
        atomicOr(status, code);
        return false;
      }
    }
  }
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, int c0, int c1,
                                            int c2, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(tm)), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, int c0, int c1,
                                            int c2, int c3, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(tm)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* tm) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(tm)) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                          uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives on the mbarrier once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                   bar)
               : "memory");
}
__device__ __forceinline__ void tmem_ld_32x32b_x32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
        "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
        "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]),
        "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]),
        "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() {
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t pack_bf16x2(uint32_t lo_f32_bits, uint32_t hi_f32_bits) {
  const __nv_bfloat162 v =
      __floats2bfloat162_rn(__uint_as_float(lo_f32_bits), __uint_as_float(hi_f32_bits));
  return *reinterpret_cast<const uint32_t*>(&v);
}
// Start-address field of a shared-memory matrix descriptor: bits [0,14) hold (address >> 4).
__device__ __forceinline__ uint64_t desc_at(uint64_t desc0, uint32_t smem_addr) {
  return desc0 | uint64_t((smem_addr >> 4) & 0x3FFFu);
}

constexpr int kThreads = 192;  // warp 0: TMA producer, warp 1: MMA issuer, warps 2-5: epilogue

}  // namespace

// ------------------------------------------------------------------------------------------------
// Halo-tile tcgen05 kernel
// ------------------------------------------------------------------------------------------------
template <typename OutT>
__global__ void __launch_bounds__(kThreads, 1)
    cconv_halo_kernel(const __grid_constant__ CUtensorMap tm_image,
                      const __grid_constant__ CUtensorMap tm_filter, OutT* __restrict__ out,
                      const HaloKernelParams p, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;  // swizzle atoms need 1024 B
  const uint32_t stage_bytes = p.filt_stage_bytes + p.img_stage_bytes;
  const uint32_t bars = smem0 + uint32_t(p.stages) * stage_bytes;
  // barrier block: full[stages], empty[stages], tfull[2], tempty[2], drain, then two 32-bit slots
  const uint32_t bar_full = bars;
  const uint32_t bar_empty = bars + 8u * p.stages;
  const uint32_t bar_tfull = bars + 16u * p.stages;
  const uint32_t bar_tempty = bar_tfull + 16u;
  const uint32_t bar_drain = bar_tempty + 16u;
  const uint32_t slot_addr = bar_drain + 8u;
  uint8_t* gen0 = smem_raw + (smem0 - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot =
      reinterpret_cast<volatile uint32_t*>(gen0 + (slot_addr - smem0));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen0 + (slot_addr + 4u - smem0));

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) {
      mbar_init(bar_full + 8u * s, 1);
      mbar_init(bar_empty + 8u * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull + 8u * a, 1);
      mbar_init(bar_tempty + 8u * a, 4);  // one arrival per epilogue warp
    }
    mbar_init(bar_drain, 1);
    *abort_flag = 0;
    fence_barrier_init();
    prefetch_tensormap(&tm_image);
    prefetch_tensormap(&tm_filter);
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

  if (warp == 0) {
    // ===================== TMA producer =====================
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x) {
        int t = tile;
        const int kt = t % p.tiles_k; t /= p.tiles_k;
        const int bt = t % p.tiles_b; t /= p.tiles_b;
        const int wt = t % p.tiles_w; t /= p.tiles_w;
        const int ht = t;
        const int k0 = kt * 128, b0 = bt * p.bb;
        const int x0 = wt * p.bw * p.sw, y0 = ht * p.bh * p.sh;
        for (int cc = 0; cc < p.cchunks; ++cc, ++it) {
          const uint32_t s = it % uint32_t(p.stages);
          const uint32_t ph = (it / uint32_t(p.stages)) & 1u;
          if (!mbar_wait(bar_empty + 8u * s, ph ^ 1u, abort_flag, status, kStatProducerWait,
                         limit)) {
            ok = false;
            break;
          }
          const uint32_t full = bar_full + 8u * s;
          mbar_arrive_expect_tx(full, stage_bytes);
          const uint32_t dst = smem0 + s * stage_bytes;
          tma_load_3d(dst, &tm_filter, cc * p.bc, k0, 0, full);
          tma_load_4d(dst + p.filt_stage_bytes, &tm_image, b0, cc * p.bc, x0, y0, full);
        }
      }
      // Do not leave while copies may still be landing in this CTA's shared memory.
      const uint32_t back = it < uint32_t(p.stages) ? it : uint32_t(p.stages);
      for (uint32_t j = 0; j < back; ++j) {
        const uint32_t i2 = it - 1 - j;
        const uint32_t s = i2 % uint32_t(p.stages);
        const uint32_t ph = (i2 / uint32_t(p.stages)) & 1u;
        uint64_t t0 = globaltimer_ns();
        while (!mbar_try_wait(bar_full + 8u * s, ph)) {
          if (globaltimer_ns() - t0 > limit) {
            atomicOr(status, kStatDrainWait);
            break;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer =====================
    if (lane == 0) {
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      const uint32_t taps = uint32_t(p.R * p.S);
      const uint32_t ksteps = uint32_t(p.bc / 16);
      for (int tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x, ++tcount) {
        const uint32_t abuf = tcount % uint32_t(p.acc_bufs);
        const uint32_t aph = (tcount / uint32_t(p.acc_bufs)) & 1u;
        if (!mbar_wait(bar_tempty + 8u * abuf, aph ^ 1u, abort_flag, status, kStatMmaWaitTmem,
                       limit)) {
          ok = false;
          break;
        }
        tc_fence_after();
        const uint32_t d_base = tmem_base + abuf * uint32_t(p.acc_cols);
        for (int cc = 0; cc < p.cchunks; ++cc, ++it) {
          const uint32_t s = it % uint32_t(p.stages);
          const uint32_t ph = (it / uint32_t(p.stages)) & 1u;
          if (!mbar_wait(bar_full + 8u * s, ph, abort_flag, status, kStatMmaWaitFull, limit)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t filt = smem0 + s * stage_bytes;
          const uint32_t img = filt + p.filt_stage_bytes;
          for (uint32_t kk = 0; kk < ksteps; ++kk) {
            for (int r = 0; r < p.R; ++r) {
              for (int sx = 0; sx < p.S; ++sx) {
                const uint32_t tap = uint32_t(r * p.S + sx);
                const uint64_t a_desc = desc_at(p.a_desc, filt + tap * p.tap_bytes + kk * 32u);
                const uint32_t acc = (cc | int(kk) | int(tap)) != 0 ? 1u : 0u;
                for (int hh = 0; hh < p.bh; ++hh) {
                  const uint32_t pix = uint32_t((hh * p.sh + sx) * p.halo_w + r);
                  const uint64_t b_desc =
                      desc_at(p.b_desc, img + pix * p.slab_bytes + kk * p.b_kstep_bytes);
                  umma_bf16(d_base + uint32_t(hh * p.n_mma), a_desc, b_desc, p.idesc, acc);
                }
              }
            }
          }
          (void)taps;
          umma_commit(bar_empty + 8u * s);  // stage reusable once these MMAs have read it
        }
        if (ok) umma_commit(bar_tfull + 8u * abuf);  // accumulator complete
      }
      // All MMAs must have retired before TMEM is released.
      umma_commit(bar_drain);
      uint64_t t0 = globaltimer_ns();
      while (!mbar_try_wait(bar_drain, 0)) {
        if (globaltimer_ns() - t0 > limit) {
          atomicOr(status, kStatDrainWait);
          break;
        }
      }
    }
  } else {
    // ===================== epilogue: TMEM -> registers -> bf16 -> global =====================
    const int q = warp & 3;  // this warp may touch TMEM lanes [32q, 32q+32)
    uint32_t tcount = 0;
    bool ok = true;
    const int chunks = p.bb / 32;
    for (int tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x, ++tcount) {
      int t = tile;
      const int kt = t % p.tiles_k; t /= p.tiles_k;
      const int bt = t % p.tiles_b; t /= p.tiles_b;
      const int wt = t % p.tiles_w; t /= p.tiles_w;
      const int ht = t;
      const int k = kt * 128 + q * 32 + lane;
      const int b0 = bt * p.bb;
      const uint32_t abuf = tcount % uint32_t(p.acc_bufs);
      const uint32_t aph = (tcount / uint32_t(p.acc_bufs)) & 1u;
      if (!mbar_wait(bar_tfull + 8u * abuf, aph, abort_flag, status, kStatEpilogueWait, limit)) {
        ok = false;
        break;
      }
      tc_fence_after();
      const uint32_t t_base = tmem_base + (uint32_t(q * 32) << 16) + abuf * uint32_t(p.acc_cols);
      for (int hh = 0; hh < p.bh; ++hh) {
        const int h = ht * p.bh + hh;
        for (int ww = 0; ww < p.bw; ++ww) {
          const int w = wt * p.bw + ww;
          const bool valid = (k < p.K) && (h < p.H) && (w < p.W);
          for (int ch = 0; ch < chunks; ++ch) {
            uint32_t v[32];
            tmem_ld_32x32b_x32(t_base + uint32_t(hh * p.n_mma + ww * p.bb + ch * 32), v);
            tmem_ld_wait();
            if (valid) {
              uint4* dst = reinterpret_cast<uint4*>(
                  out + (((long long)k * p.H + h) * p.W + w) * p.B + b0 + ch * 32);
              if constexpr (sizeof(OutT) == 4) {
#pragma unroll
                for (int j = 0; j < 8; ++j)
                  dst[j] = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
              } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  uint4 o;
                  o.x = pack_bf16x2(v[8 * j + 0], v[8 * j + 1]);
                  o.y = pack_bf16x2(v[8 * j + 2], v[8 * j + 3]);
                  o.z = pack_bf16x2(v[8 * j + 4], v[8 * j + 5]);
                  o.w = pack_bf16x2(v[8 * j + 6], v[8 * j + 7]);
                  dst[j] = o;
                }
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty + 8u * abuf);
    }
  }

  // ===================== teardown =====================
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, uint32_t(p.tmem_cols));
  }
}

cudaError_t halo_kernel_prepare(int smem_bytes) {
  cudaError_t e = cudaFuncSetAttribute(cconv_halo_kernel<__nv_bfloat16>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(cconv_halo_kernel<float>,
                              cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
}

cudaError_t launch_halo(const CUtensorMap& tm_image, const CUtensorMap& tm_filter, void* out,
                        bool out_f32, const HaloKernelParams& p, int grid, int smem_bytes,
                        int* status, cudaStream_t stream) {
  if (out_f32)
    cconv_halo_kernel<float><<<grid, kThreads, smem_bytes, stream>>>(
        tm_image, tm_filter, static_cast<float*>(out), p, status);
  else
    cconv_halo_kernel<__nv_bfloat16><<<grid, kThreads, smem_bytes, stream>>>(
        tm_image, tm_filter, static_cast<__nv_bfloat16*>(out), p, status);
  return cudaGetLastError();
}

}  // namespace cconv
