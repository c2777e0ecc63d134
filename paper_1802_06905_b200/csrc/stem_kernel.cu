// Small-C ("stem") tensor-core kernel for the seven-nested-loop CNN (Eq. 1):
//   Out(k,h,w,b) = sum_{c,r,s} Image(r+sw*w, s+sh*h, c, b) * Filter(k,r,s,c)
// for shapes whose channel count is far below the tensor core's K = 16 (the benchmark's 7x7,
// stride-2, C = 3 layer).  Padding C to 16 would waste 13/16 of every MMA; instead the contraction
// dimension of one MMA runs over the (s, c) pairs of one filter column r, which are CONTIGUOUS rows
// of the Image for a fixed first subscript x: Image[x][y][c][b] viewed as [x][m = y*C + c][b].
// This is the paper's lifting r = sw*r' + r'' turned sideways: the loop that is too short to fill
// a block (c) is merged with its neighbour (s) so that the block is full.
//
// Roles are swapped with respect to the halo kernel:
//   A (MMA rows, M = 128)  = Image: 2 adjacent output pixels x 64 images, MN-major (b contiguous),
//                            TMA-written 128-byte swizzled rows, pixel 2 at +sw columns (LBO);
//   B (MMA cols, N = K)    = Filter column r, K-major, resident in shared memory for the whole
//                            kernel (R x ndelta x kw/16 blocks of n_out x 16);
//   D (TMEM)               = [2 pixels x 64 images][K] fp32, one accumulator per pixel pair.
// An MMA's 16 contraction rows must start on an 8-row swizzle atom, but output row h needs rows
// sh*C*h .. +S*C-1.  So the kernel reads the aligned window that starts delta = (sh*C*h) % 8 rows
// earlier, and the Filter is stored once per distinct delta, shifted by delta rows, zero elsewhere.
#include <cuda_bf16.h>

#include "kernels.h"
#include "ptx_sm100.cuh"

namespace cconv {

namespace {

constexpr int kStemThreads = 192;  // warp 0: producer, warp 1: MMA issuer, warps 2-5: epilogue

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, int c0, int c1,
                                            int c2, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(tm)), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tma_store_4d(const CUtensorMap* tm, int c0, int c1, int c2, int c3,
                                             uint32_t src) {
  asm volatile(
      "cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3, %4}], [%5];" ::
          "l"(reinterpret_cast<uint64_t>(tm)),
      "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(src)
      : "memory");
}
__device__ __forceinline__ void bulk_commit() {
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// until the bulk stores issued so far by this thread have READ their shared-memory source
__device__ __forceinline__ void bulk_wait_read_all() {
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
// until they have completed altogether
__device__ __forceinline__ void bulk_wait_all() {
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

__device__ __forceinline__ void store_scalar(float* p, uint32_t f32_bits) {
  *p = __uint_as_float(f32_bits);
}

}  // namespace

// ------------------------------------------------------------------------------------------------
// Filter packing for the stem kernel.  Block (r, di, kh) holds, for every output channel n and
// window row j = kh*16 + jj, the value Filter[n][r][s][c] with s*C + c = j - di*dstep (zero outside
// 0 .. S*C-1 and for n >= K), as n_out x 16 bf16 in K-major no-swizzle core-matrix order:
// element (n, jj) at ((n/8)*2 + jj/8)*128 + (n%8)*16 + (jj%8)*2 bytes.  One thread writes 16 bytes.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
    cconv_pack_filter_stem_kernel(const __nv_bfloat16* __restrict__ filter,
                                  uint4* __restrict__ packed, Dims d, int n_out, int khalves,
                                  int ndelta, int dstep, long long slots) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const long long slot = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (slot >= slots) return;
  const int per_block = n_out * 2;  // 16-byte slots per block
  const int j = int(slot % per_block);
  long long blk = slot / per_block;
  const int kh = int(blk % khalves);
  blk /= khalves;
  const int di = int(blk % ndelta);
  const int r = int(blk / ndelta);
  const int core = j >> 3, row = j & 7;
  const int n = (core >> 1) * 8 + row;
  const int jj0 = (core & 1) * 8;
  unsigned short e[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int q = kh * 16 + jj0 + i - di * dstep;  // (s, c) index of this window row
    unsigned short v = 0;
    if (n < d.K && q >= 0 && q < d.S * d.C) {
      const int s = q / d.C, c = q - s * d.C;
      v = *reinterpret_cast<const unsigned short*>(
          filter + (((long long)n * d.R + r) * d.S + s) * d.C + c);
    }
    e[i] = v;
  }
  uint4 o;
  o.x = e[0] | (uint32_t(e[1]) << 16);
  o.y = e[2] | (uint32_t(e[3]) << 16);
  o.z = e[4] | (uint32_t(e[5]) << 16);
  o.w = e[6] | (uint32_t(e[7]) << 16);
  packed[slot] = o;
}

cudaError_t launch_pack_filter_stem(const void* filter, void* packed, const Dims& d,
                                    const StemKernelParams& p, cudaStream_t stream) {
  const long long slots = (long long)p.filt_bytes / 16;
  const long long blocks = (slots + 255) / 256;
  cconv_pack_filter_stem_kernel<<<(unsigned)blocks, 256, 0, stream>>>(
      static_cast<const __nv_bfloat16*>(filter), static_cast<uint4*>(packed), d, p.n_out,
      p.khalves, p.ndelta, p.dstep, slots);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// The kernel.  Persistent; tile = (64 images) x (one output row h) x (bw output pixels).
// ------------------------------------------------------------------------------------------------
template <typename OutT>
__global__ void __launch_bounds__(kStemThreads, 1)
    cconv_stem_kernel(const __grid_constant__ CUtensorMap tm_image,
                      const __grid_constant__ CUtensorMap tm_out,
                      const uint8_t* __restrict__ packed_filter, OutT* __restrict__ out,
                      const StemKernelParams p, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t img_ring = smem0;
  const uint32_t filt_smem = img_ring + uint32_t(p.i_stages) * p.img_stage_bytes;
  const uint32_t stage_smem = filt_smem + p.filt_bytes;  // 2 x 4 KB: sources of the TMA stores
  const uint32_t bars = stage_smem + 8192u;
  const uint32_t bar_ifull = bars;
  const uint32_t bar_iempty = bar_ifull + 8u * p.i_stages;
  const uint32_t bar_filt = bar_iempty + 8u * p.i_stages;
  const uint32_t bar_tfull = bar_filt + 8u;
  const uint32_t bar_tempty = bar_tfull + 16u;
  const uint32_t bar_drain = bar_tempty + 16u;
  const uint32_t slot_addr = bar_drain + 8u;
  uint8_t* gen0 = smem_raw + (smem0 - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen0 + (slot_addr - smem0));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen0 + (slot_addr + 4u - smem0));

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.i_stages; ++s) {
      mbar_init(bar_ifull + 8u * s, 1);
      mbar_init(bar_iempty + 8u * s, 1);
    }
    mbar_init(bar_filt, 1);
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull + 8u * a, 1);
      mbar_init(bar_tempty + 8u * a, 4);  // one arrival per epilogue warp
    }
    mbar_init(bar_drain, 1);
    *abort_flag = 0;
    fence_barrier_init();
    prefetch_tensormap(&tm_image);
    prefetch_tensormap(&tm_out);
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
  const int tiles_per_b = p.H * p.tiles_w;
  const int shc = p.sh * p.C;  // Image rows (of the merged (y,c) axis) per output row

  if (warp == 0) {
    // ===================== producer: the Filter once, then one Image slab per tile =====================
    if (lane == 0) {
      uint32_t it = 0, s = 0, ph = 0;
      bool ok = true;
      const uint32_t n_st = uint32_t(p.i_stages);
      for (int tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x, ++it) {
        const int bt = tile / tiles_per_b;
        const int rem = tile - bt * tiles_per_b;
        const int h = rem / p.tiles_w, wt = rem - h * p.tiles_w;
        const int m0 = shc * h - ((shc * h) & 7);  // aligned start of the (s,c) window
        if (!mbar_wait(bar_iempty + 8u * s, ph ^ 1u, abort_flag, status, kStatProducerWait, limit)) {
          ok = false;
          break;
        }
        const uint32_t full = bar_ifull + 8u * s;
        mbar_arrive_expect_tx(full, p.img_stage_bytes);
        tma_load_3d(img_ring + s * p.img_stage_bytes, &tm_image, bt * 64, m0, wt * p.bw * p.sw, full);
        if (it == 0) {
          // the packed Filter is written by the kernel launched just before this one
          asm volatile("griddepcontrol.wait;" ::: "memory");
          mbar_arrive_expect_tx(bar_filt, p.filt_bytes);
          for (uint32_t off = 0; off < p.filt_bytes; off += 16384u) {
            const uint32_t n = p.filt_bytes - off < 16384u ? p.filt_bytes - off : 16384u;
            bulk_load(filt_smem + off, packed_filter + off, n, bar_filt);
          }
        }
        if (++s == n_st) {
          s = 0;
          ph ^= 1u;
        }
      }
      drain_ring(bar_ifull, it, n_st, status, limit);
      if (it > 0) {
        const uint64_t t0 = globaltimer_ns();
        while (!mbar_try_wait(bar_filt, 0)) {
          if (globaltimer_ns() - t0 > limit) {
            atomicOr(status, kStatDrainWait);
            break;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer (whole warp walks, one lane issues) =====================
    const bool leader = elect_one();
    uint32_t is = 0, iph = 0, abuf = 0, aph = 0;
    const uint32_t n_ist = uint32_t(p.i_stages);
    const uint32_t a_lo0 = uint32_t(p.a_desc), a_hi = uint32_t(p.a_desc >> 32);
    const uint32_t b_lo0 = uint32_t(p.b_desc), b_hi = uint32_t(p.b_desc >> 32);
    const uint32_t xslab16 = p.xslab_bytes >> 4, fblk16 = p.fblock_bytes >> 4;
    const uint32_t img16 = p.img_stage_bytes >> 4;
    const uint32_t img_ring16 = img_ring >> 4, filt16 = filt_smem >> 4;
    const uint32_t idesc = p.idesc, n_out = uint32_t(p.n_out);
    const int pairs = p.bw / 2, R = p.R, khalves = p.khalves;
    const uint32_t pair16 = uint32_t(2 * p.sw) * xslab16;  // next pixel pair: 2*sw Image columns
    bool ok = mbar_wait_warp(bar_filt, 0, abort_flag, status, kStatMmaWaitFull, limit);
    tc_fence_after();
    for (int tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x) {
      const int rem = tile % tiles_per_b;
      const int h = rem / p.tiles_w;
      const uint32_t di = uint32_t(((shc * h) & 7) / p.dstep);
      if (!mbar_wait_warp(bar_tempty + 8u * abuf, aph ^ 1u, abort_flag, status, kStatMmaWaitTmem,
                          limit))
        break;
      if (!mbar_wait_warp(bar_ifull + 8u * is, iph, abort_flag, status, kStatMmaWaitFull, limit))
        break;
      tc_fence_after();
      const uint32_t d_base = tmem_base + abuf * uint32_t(p.acc_cols);
      const uint32_t img_s16 = img_ring16 + is * img16;
      uint32_t acc = 0;
      for (int r = 0; r < R; ++r) {
        uint32_t f16 = filt16 + (uint32_t(r) * uint32_t(p.ndelta) + di) * uint32_t(khalves) * fblk16;
        uint32_t a_r16 = img_s16 + uint32_t(r) * xslab16;
        for (int kh = 0; kh < khalves; ++kh, f16 += fblk16, a_r16 += 128u /* 16 rows x 128 B */) {
          const uint64_t b_desc = (uint64_t(b_hi) << 32) | (b_lo0 | f16);
          uint32_t a16 = a_r16, d = d_base;
          for (int g = 0; g < pairs; ++g, a16 += pair16, d += n_out)
            umma_bf16_if(leader, d, (uint64_t(a_hi) << 32) | (a_lo0 | a16), b_desc, idesc, acc);
          acc = 1;
        }
      }
      if (leader) umma_commit(bar_iempty + 8u * is);
      if (leader) umma_commit(bar_tfull + 8u * abuf);
      if (++is == n_ist) {
        is = 0;
        iph ^= 1u;
      }
      abuf ^= 1u;
      if (abuf == 0) aph ^= 1u;
    }
    if (leader) umma_commit(bar_drain);
    const uint64_t t0 = globaltimer_ns();
    while (!mbar_try_wait(bar_drain, 0)) {
      if (globaltimer_ns() - t0 > limit) {
        atomicOr(status, kStatDrainWait);
        break;
      }
    }
  } else {
    // ===================== epilogue: TMEM -> registers -> Out =====================
    // TMEM lane = pixel_in_pair*64 + image; this warp owns lanes [32q, 32q+32).
    const int q = warp & 3;
    const int pix = q >> 1, b_in = (q & 1) * 32 + lane;
    uint32_t abuf = 0, aph = 0;
    const int pairs = p.bw / 2;
    const long long k_stride = (long long)p.H * p.W * p.B;
    for (int tile = blockIdx.x; tile < p.total_tiles; tile += gridDim.x) {
      const int bt = tile / tiles_per_b;
      const int rem = tile - bt * tiles_per_b;
      const int h = rem / p.tiles_w, wt = rem - h * p.tiles_w;
      if (!mbar_wait_warp(bar_tfull + 8u * abuf, aph, abort_flag, status, kStatEpilogueWait, limit))
        break;
      tc_fence_after();
      const uint32_t t_base = tmem_base + (uint32_t(q * 32) << 16) + abuf * uint32_t(p.acc_cols);
      for (int g = 0; g < pairs; ++g) {
        const int w = wt * p.bw + 2 * g + pix;
        for (int k0 = 0; k0 < p.n_out; k0 += 32) {
          uint32_t v[32];
          tmem_ld_32x32b_x32(t_base + uint32_t(g * p.n_out + k0), v);
          tmem_ld_wait();
          if constexpr (sizeof(OutT) == 2) {
            // bf16: the two warps that hold one pixel (images 0-31 and 32-63) transpose their
            // 32 x 32 blocks through a [32 k][64 images] staging buffer, and one TMA store writes
            // it as 32 full 128-byte lines of Out.
            const uint32_t buf = stage_smem + uint32_t(pix) * 4096u;
            const bool issuer = (q & 1) == 0 && lane == 0;
            if (issuer) bulk_wait_read_all();       // the previous store has read the buffer
            named_bar_sync(1 + pix, 64);
            uint8_t* row0 = gen0 + (buf - smem0) + b_in * 2;
#pragma unroll
            for (int j = 0; j < 32; ++j)
              *reinterpret_cast<__nv_bfloat16*>(row0 + j * 128) =
                  __float2bfloat16_rn(__uint_as_float(v[j]));
            fence_proxy_async_smem();
            named_bar_sync(1 + pix, 64);
            if (issuer && w < p.W && k0 < p.K) {
              tma_store_4d(&tm_out, bt * 64, w, h, k0, buf);   // rows k >= K are clipped
              bulk_commit();
            }
          } else {
            if (w < p.W) {
              // fp32: a warp writes 32 consecutive images of one (k, h, w), 128 contiguous bytes
              OutT* dst = out + ((long long)h * p.W + w) * p.B + bt * 64 + b_in;
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (k0 + j < p.K) store_scalar(dst + (long long)(k0 + j) * k_stride, v[j]);
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty + 8u * abuf);
      abuf ^= 1u;
      if (abuf == 0) aph ^= 1u;
    }
    if ((q & 1) == 0 && lane == 0) bulk_wait_all();  // Out is written before the CTA leaves
  }

  // ===================== teardown =====================
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, uint32_t(p.tmem_cols));
  }
}

cudaError_t stem_kernel_prepare(int smem_bytes) {
  cudaError_t e = cudaFuncSetAttribute(cconv_stem_kernel<__nv_bfloat16>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(cconv_stem_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              smem_bytes);
}

cudaError_t launch_stem(const CUtensorMap& tm_image, const CUtensorMap& tm_out,
                        const void* packed_filter, void* out,
                        bool out_f32, const StemKernelParams& p, int grid, int smem_bytes,
                        int* status, cudaStream_t stream) {
  const uint8_t* pf = static_cast<const uint8_t*>(packed_filter);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(grid));
  cfg.blockDim = dim3(kStemThreads);
  cfg.dynamicSmemBytes = size_t(smem_bytes);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (out_f32)
    return cudaLaunchKernelEx(&cfg, cconv_stem_kernel<float>, tm_image, tm_out, pf, static_cast<float*>(out),
                              p, status);
  return cudaLaunchKernelEx(&cfg, cconv_stem_kernel<__nv_bfloat16>, tm_image, tm_out, pf,
                            static_cast<__nv_bfloat16*>(out), p, status);
}

}  // namespace cconv
