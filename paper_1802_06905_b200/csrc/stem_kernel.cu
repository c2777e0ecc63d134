// Small-C ("stem") tensor-core kernel for the seven-nested-loop CNN (Eq. 1):
//   Out(k,h,w,b) = sum_{c,r,s} Image(r+sw*w, s+sh*h, c, b) * Filter(k,r,s,c)
// for shapes whose channel count is far below the tensor core's K = 16 (the benchmark's 7x7,
// stride-2, C = 3 layer).  Padding C to 16 would waste 13/16 of every MMA; instead the contraction
// dimension of one MMA runs over the (s, c) pairs of one filter column r, which are CONTIGUOUS rows
// of the Image for a fixed first subscript x: Image[x][y][c][b] viewed as [x][m = y*C + c][b].
// This is the paper's lifting r = sw*r' + r'' turned sideways: the loop that is too short to fill
// a block (c) is merged with its neighbour (s) so that the block is full.
//
// One MMA (M = 128, N = 64*bw, K = 16):
//   A (rows)  = Filter column r, K-major, repacked by every CTA at its start and resident in
//               shared memory for the whole kernel (no packing kernel, no scratch).  When
//               K <= 64 the 128 rows are STACKED output rows: row j*kpad + k holds filter k shifted
//               down by j*sh*C window rows, so one MMA over one Image window yields the bhm = 128/kpad
//               consecutive output rows h0 .. h0+bhm-1 (their windows overlap almost entirely);
//   B (cols)  = Image window: bw adjacent output pixels x 64 images, MN-major (b contiguous),
//               TMA-written 128-byte swizzled rows; next pixel = +sw Image columns (LBO), next
//               8 window rows = +1024 B (SBO);
//   D (TMEM)  = [stacked row j, out-channel k][pixel, image] fp32, two buffers.
// The window of a tile starts exactly at Image row m0 = sh*C*h0 (a TMA box may start anywhere in
// that coordinate), so shared-memory row 0 is always the first row the MMA needs.  The contraction
// over (r, 16-row slice) is ONE linear walk: the Filter blocks are stored in that order and the
// Image box [x][m][64] has x-slabs of kw rows, so unit u = r*khalves + kh sits at u*4 KB in the
// Filter and at u*2 KB in the Image stage.
//
// Rows of the window that belong to a neighbouring output row meet zero Filter entries; a
// non-finite Image value there would turn that zero product into NaN (the variant assumes finite
// inputs, like any zero-padded tensor-core tiling).
#include <cuda_bf16.h>

#include "kernels.h"
#include "ptx_sm100.cuh"

namespace cconv {

namespace {

// warp 0: producer, warp 1: MMA issuer, warps 2-9: epilogue (two warps per TMEM lane quarter, each
// taking every other pixel of a tile)
constexpr int kStemThreads = 320;
constexpr int kStemEpiThreads = 256;
constexpr uint32_t kStemStagingBytes = 65536;

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
// until all but the newest bulk-store group of this thread have READ their shared-memory source
__device__ __forceinline__ void bulk_wait_read_1() {
  asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
}
// until every bulk store of this thread has completed altogether
__device__ __forceinline__ void bulk_wait_all() {
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c,
                                             uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d)
               : "memory");
}
__device__ __forceinline__ void st_shared_u16(uint32_t addr, unsigned short v) {
  asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_shared_u32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint32_t ld_shared_u16(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}

}  // namespace

// ------------------------------------------------------------------------------------------------
// The kernel.  Persistent; tile = (128 out-channels) x (64 images) x (bhm output rows) x (bw pixels).
// ------------------------------------------------------------------------------------------------
template <typename OutT>
__global__ void __launch_bounds__(kStemThreads, 1)
    cconv_stem_kernel(const __grid_constant__ CUtensorMap tm_image,
                      const __grid_constant__ CUtensorMap tm_out,
                      const unsigned short* __restrict__ filter, const StemKernelParams p,
                      int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t img_ring = smem0;
  const uint32_t filt_smem = img_ring + uint32_t(p.i_stages) * p.img_stage_bytes;
  // 8 epilogue warps x 2 buffers x 4 KB: sources of the TMA stores; before the first tile the same
  // bytes hold the raw Filter while it is repacked
  const uint32_t stage_smem = filt_smem + p.filt_bytes;
  const uint32_t bars = stage_smem + kStemStagingBytes;
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
  // diagnostics: per-CTA row of 16 counters (0 entry ns, 1 exit ns, 2.. cycles spent per role)
  unsigned long long* const tr = p.trace ? p.trace + 16ull * blockIdx.x : nullptr;
  if (tr && threadIdx.x == 0) tr[0] = globaltimer_ns();

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.i_stages; ++s) {
      mbar_init(bar_ifull + 8u * s, 1);
      mbar_init(bar_iempty + 8u * s, 1);
    }
    mbar_init(bar_filt, kStemEpiThreads);  // every thread of the epilogue warps arrives once
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull + 8u * a, 1);
      mbar_init(bar_tempty + 8u * a, kStemEpiThreads / 32);  // one arrival per epilogue warp
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
  const int shc = p.sh * p.C;  // Image rows (of the merged (y,c) axis) per output row

  if (warp == 0) {
    // ===================== producer: one Image window per tile =====================
    if (lane == 0) {
      uint32_t it = 0, s = 0, ph = 0;
      bool ok = true;
      long long t_wait = 0;
      const uint32_t n_st = uint32_t(p.i_stages);
      for (int tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x, ++it) {
        int t = tile / p.tiles_k;
        const int wt = t % p.tiles_w;
        t /= p.tiles_w;
        const int ht = t % p.tiles_h, bt = t / p.tiles_h;
        const long long c0 = tr ? clock64() : 0;
        if (!mbar_wait(bar_iempty + 8u * s, ph ^ 1u, abort_flag, status, kStatProducerWait, limit)) {
          ok = false;
          break;
        }
        if (tr) t_wait += clock64() - c0;
        const uint32_t full = bar_ifull + 8u * s;
        mbar_arrive_expect_tx(full, p.img_stage_bytes);
        tma_load_3d(img_ring + s * p.img_stage_bytes, &tm_image, bt * 64, shc * ht * p.bhm,
                    wt * p.bw * p.sw, full);
        if (++s == n_st) {
          s = 0;
          ph ^= 1u;
        }
      }
      if (tr) tr[2] = (unsigned long long)t_wait;
      drain_ring(bar_ifull, it, n_st, status, limit);
    }
  } else if (warp == 1) {
    // ===================== MMA issuer (whole warp walks, one lane issues) =====================
    const bool leader = elect_one();
    uint32_t is = 0, iph = 0, abuf = 0, aph = 0;
    const uint32_t n_ist = uint32_t(p.i_stages);
    const uint32_t a_lo0 = uint32_t(p.a_desc), a_hi = uint32_t(p.a_desc >> 32);
    const uint32_t b_lo0 = uint32_t(p.b_desc), b_hi = uint32_t(p.b_desc >> 32);
    const uint32_t img16 = p.img_stage_bytes >> 4;
    const uint32_t img_ring16 = img_ring >> 4, filt16 = filt_smem >> 4;
    const uint32_t idesc = p.idesc;
    const int units = p.units;
    const uint32_t kt_step16 = uint32_t(units) * 256u;  // one k-tile of the Filter: units x 4 KB
    long long t_filt = tr ? clock64() : 0, t_wt = 0, t_wi = 0, t_issue = 0, n_tiles = 0;
    bool ok = mbar_wait_warp(bar_filt, 0, abort_flag, status, kStatMmaWaitFull, limit);
    if (tr) t_filt = clock64() - t_filt;
    tc_fence_after();
    for (int tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x) {
      const uint32_t kt = uint32_t(tile % p.tiles_k);
      const long long c0 = tr ? clock64() : 0;
      if (!mbar_wait_warp(bar_tempty + 8u * abuf, aph ^ 1u, abort_flag, status, kStatMmaWaitTmem,
                          limit))
        break;
      const long long c1 = tr ? clock64() : 0;
      if (!mbar_wait_warp(bar_ifull + 8u * is, iph, abort_flag, status, kStatMmaWaitFull, limit))
        break;
      const long long c2 = tr ? clock64() : 0;
      tc_fence_after();
      const uint32_t d = tmem_base + abuf * uint32_t(p.acc_cols);
      uint32_t a16 = a_lo0 | (filt16 + kt * kt_step16);   // +256 per unit (4 KB Filter block)
      uint32_t b16 = b_lo0 | (img_ring16 + is * img16);   // +128 per unit (16 window rows)
      umma_bf16_if(leader, d, (uint64_t(a_hi) << 32) | a16, (uint64_t(b_hi) << 32) | b16, idesc, 0u);
#pragma unroll 2
      for (int u = 1; u < units; ++u) {
        a16 += 256u;
        b16 += 128u;
        umma_bf16_if(leader, d, (uint64_t(a_hi) << 32) | a16, (uint64_t(b_hi) << 32) | b16, idesc,
                     1u);
      }
      if (leader) umma_commit(bar_iempty + 8u * is);
      if (leader) umma_commit(bar_tfull + 8u * abuf);
      if (tr) {
        t_wt += c1 - c0;
        t_wi += c2 - c1;
        t_issue += clock64() - c2;
        ++n_tiles;
      }
      if (++is == n_ist) {
        is = 0;
        iph ^= 1u;
      }
      abuf ^= 1u;
      if (abuf == 0) aph ^= 1u;
    }
    if (tr && lane == 0) {
      tr[3] = (unsigned long long)t_wt;
      tr[4] = (unsigned long long)t_wi;
      tr[5] = (unsigned long long)t_issue;
      tr[8] = (unsigned long long)n_tiles;
      tr[9] = (unsigned long long)t_filt;
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
    // ===================== epilogue warps =====================
    const int q = warp & 3;            // this warp may touch TMEM lanes [32q, 32q+32)
    const int eset = (warp - 2) >> 2;  // 0: even pixels of a tile, 1: odd pixels
    const int et = (warp - 2) * 32 + lane;  // 0..255
    // ---- phase 0: repack the Filter into the resident MMA blocks ----
    // Block (kt, r, kh) holds 128 rows x 16 window rows: row j*kpad + kk, column jj carries
    // Filter[kt*128 + kk][r][s][c] with s*C + c = kh*16 + jj - j*sh*C (zero outside 0 .. S*C-1, for
    // k >= K and for j >= bhm), in K-major no-swizzle core-matrix order: element (row, jj) at
    // ((row/8)*2 + jj/8)*128 + (row%8)*16 + (jj%8)*2 bytes.  Since (s, c) is contiguous in Filter,
    // the value is simply element q = kh*16 + jj - j*sh*C of the run Filter[k][r][.][.].  The raw
    // Filter passes through shared memory in chunks of whole out-channels, every run padded with
    // `lead` zeros in front and zeros behind up to P elements, so that any 8 consecutive window rows
    // of any stacked row are 8 consecutive elements there, with no bounds to test.
    {
      const long long pk0 = tr ? clock64() : 0;
      for (uint32_t off = uint32_t(et) * 16u; off < p.filt_bytes; off += 16u * kStemEpiThreads)
        st_shared_v4(filt_smem + off, 0u, 0u, 0u, 0u);
      const int SC = p.S * p.C;
      const int lead = shc * (p.bhm - 1);
      const int P = (lead + p.kw + 7) & ~7;  // padded run length, elements
      // per out-channel: R raw runs of SC elements and R padded runs of P elements
      const int kc_max = int((kStemStagingBytes - 32u) / (2u * uint32_t(p.R * (SC + P))));  // >= 1
      const int kc = p.K < kc_max ? p.K : kc_max;
      const uint32_t pad_smem = stage_smem;                              // [runs][P]
      const uint32_t raw_base = stage_smem + 2u * uint32_t(kc * p.R * P);  // 16-byte aligned
      for (int k0 = 0; k0 < p.K; k0 += kc) {
        const int nk = p.K - k0 < kc ? p.K - k0 : kc;
        const int runs = nk * p.R;
        named_bar_sync(1, kStemEpiThreads);  // previous chunk no longer read
        // (a) the chunk's raw bytes, as 16-byte vectors; shared and global addresses stay congruent
        //     mod 16 so that the vectors line up
        const unsigned short* g = filter + (long long)k0 * p.R * SC;
        const uint32_t mis = uint32_t(reinterpret_cast<uintptr_t>(g) & 15u);
        const uint32_t raw = raw_base + mis;  // address of element 0 of the chunk
        const int n = runs * SC;
        int head = int(((16u - mis) & 15u) >> 1);
        if (head > n) head = n;
        const int nvec = (n - head) >> 3;
        const int tail0 = head + nvec * 8;
        if (et < head) st_shared_u16(raw + 2u * et, __ldg(g + et));
        const uint4* gv = reinterpret_cast<const uint4*>(g + head);
        for (int i0 = 0; i0 < nvec; i0 += 4 * kStemEpiThreads) {
          uint4 v[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * kStemEpiThreads + et;
            if (i < nvec) v[u] = __ldg(gv + i);
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * kStemEpiThreads + et;
            if (i < nvec) st_shared_v4(raw + 2u * head + 16u * i, v[u].x, v[u].y, v[u].z, v[u].w);
          }
        }
        if (et < n - tail0) st_shared_u16(raw + 2u * (tail0 + et), __ldg(g + tail0 + et));
        // (b) zero the padded runs
        for (uint32_t off = uint32_t(et) * 16u; off < uint32_t(runs * P) * 2u;
             off += 16u * kStemEpiThreads)
          st_shared_v4(pad_smem + off, 0u, 0u, 0u, 0u);
        named_bar_sync(1, kStemEpiThreads);
        if (tr && et == 64) tr[15] = (unsigned long long)(clock64() - pk0);
        // (c) raw run -> padded run, `lead` elements in
        for (int run = et; run < runs; run += kStemEpiThreads) {
          const uint32_t src = raw + 2u * uint32_t(run * SC);
          const uint32_t dst = pad_smem + 2u * uint32_t(run * P + lead);
#pragma unroll 4
          for (int i = 0; i < SC; ++i)
            st_shared_u16(dst + 2u * i, (unsigned short)ld_shared_u16(src + 2u * i));
        }
        named_bar_sync(1, kStemEpiThreads);
        if (tr && et == 64) tr[12] = (unsigned long long)(clock64() - pk0);
        const int combos = nk * p.bhm * 2;
        for (int ci = et; ci < combos; ci += kStemEpiThreads) {
          const int half = ci & 1, rest = ci >> 1;
          const int j = rest / nk, kl = rest - j * nk;
          const int k = k0 + kl;
          const int kt = k >> 7, kk = k & 127;  // kpad is 128 whenever K > 128
          const int row = j * p.kpad + kk;
          uint32_t dst = filt_smem + uint32_t(kt * p.units) * 4096u +
                         uint32_t(((row >> 3) * 2 + half) * 128 + (row & 7) * 16);
          const int qbase = half * 8 - j * shc;  // window row -> element of the run
          const bool even = ((lead + qbase) & 1) == 0;
          uint32_t src_r = pad_smem + 2u * uint32_t(kl * p.R * P + lead + qbase);
          for (int r = 0; r < p.R; ++r, src_r += 2u * P) {
            uint32_t src = src_r;
            for (int kh = 0; kh < p.khalves; ++kh, dst += 4096u, src += 32u) {
              const int q0 = kh * 16 + qbase;
              if (q0 + 8 <= 0 || q0 >= SC) continue;  // stays zero
              if (even) {
                st_shared_v4(dst, ld_shared_u32(src), ld_shared_u32(src + 4u), ld_shared_u32(src + 8u),
                             ld_shared_u32(src + 12u));
              } else {
                uint32_t e[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) e[i] = ld_shared_u16(src + 2u * i);
                st_shared_v4(dst, e[0] | (e[1] << 16), e[2] | (e[3] << 16), e[4] | (e[5] << 16),
                             e[6] | (e[7] << 16));
              }
            }
          }
        }
      }
      fence_proxy_async_smem();  // the MMAs read these generic-proxy writes through the async proxy
      if (tr && et == 64) tr[14] = (unsigned long long)(clock64() - pk0);
      mbar_arrive(bar_filt);
      named_bar_sync(1, kStemEpiThreads);  // the raw area becomes the store staging buffers
    }

    // ---- tiles: TMEM -> registers -> swizzled staging rows -> TMA store ----
    // TMEM lane = j*kpad + kk: stacked output row j (uniform in a warp), out-channel kk (32
    // consecutive ones in a warp).  One staging buffer = [32 out-channels][128 B] = the 64 (bf16) or
    // 32 (fp32) images of one pixel, 16-byte chunks XOR-swizzled by the row as the store's tensor
    // map expects, so that the 8 lanes of a store phase hit 8 different bank groups.
    const int j = (q * 32) / p.kpad;
    const int kk0 = q * 32 - j * p.kpad;
    const uint32_t my_stage = stage_smem + uint32_t(warp - 2) * 8192u;
    const uint32_t row_addr = uint32_t(lane) * 128u, x7 = uint32_t(lane & 7) << 4;
    uint32_t cnt = 0, abuf = 0, aph = 0;
    long long t_wf = 0, t_busy = 0, t_ld = 0, t_rd = 0, t_fence = 0, t_issue = 0;
    auto emit = [&](const uint32_t(&r)[32], bool ok, int b0, int w, int h, int k0) {
      const uint32_t buf = my_stage + (cnt & 1u) * 4096u;
      const long long e0 = tr ? clock64() : 0;
      if (lane == 0) bulk_wait_read_1();  // the store issued two buffers ago has read this one
      __syncwarp();
      if (tr) t_rd += clock64() - e0;
#pragma unroll
      for (int c = 0; c < 8; ++c)
        st_shared_v4(buf + row_addr + (uint32_t(c << 4) ^ x7), r[4 * c], r[4 * c + 1], r[4 * c + 2],
                     r[4 * c + 3]);
      const long long e1 = tr ? clock64() : 0;
      fence_proxy_async_smem();
      __syncwarp();
      const long long e2 = tr ? clock64() : 0;
      if (lane == 0) {
        if (ok) tma_store_4d(&tm_out, b0, w, h, k0, buf);  // rows k >= K are clipped by the map
        bulk_commit();
      }
      if (tr) {
        t_fence += e2 - e1;
        t_issue += clock64() - e2;
      }
      ++cnt;
    };
    for (int tile = blockIdx.x; tile < p.total_tiles; tile += gridDim.x) {
      int t = tile;
      const int kt = t % p.tiles_k;
      t /= p.tiles_k;
      const int wt = t % p.tiles_w;
      t /= p.tiles_w;
      const int ht = t % p.tiles_h, bt = t / p.tiles_h;
      const int k0 = kt * 128 + kk0;
      const int h = ht * p.bhm + j;
      const long long c0 = tr ? clock64() : 0;
      if (!mbar_wait_warp(bar_tfull + 8u * abuf, aph, abort_flag, status, kStatEpilogueWait, limit))
        break;
      const long long c1 = tr ? clock64() : 0;
      tc_fence_after();
      const uint32_t t_base = tmem_base + (uint32_t(q * 32) << 16) + abuf * uint32_t(p.acc_cols);
      const bool row_ok = (k0 < p.K) && (j < p.bhm) && (h < p.H);
      for (int px = eset; px < p.bw; px += 2) {
        uint32_t va[32], vb[32];
        const long long l0 = tr ? clock64() : 0;
        tmem_ld_32x32b_x32(t_base + uint32_t(px * 64), va);
        tmem_ld_32x32b_x32(t_base + uint32_t(px * 64 + 32), vb);
        tmem_ld_wait();
        if (tr) t_ld += clock64() - l0;
        const int w = wt * p.bw + px;
        const bool ok = row_ok && w < p.W;
        if constexpr (sizeof(OutT) == 4) {
          emit(va, ok, bt * 64, w, h, k0);
          emit(vb, ok, bt * 64 + 32, w, h, k0);
        } else {
          uint32_t pk[32];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            pk[i] = pack_bf16x2(va[2 * i], va[2 * i + 1]);
            pk[16 + i] = pack_bf16x2(vb[2 * i], vb[2 * i + 1]);
          }
          emit(pk, ok, bt * 64, w, h, k0);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty + 8u * abuf);
      abuf ^= 1u;
      if (abuf == 0) aph ^= 1u;
      if (tr) {
        t_wf += c1 - c0;
        t_busy += clock64() - c1;
      }
    }
    if (tr && warp == 4 && lane == 0) {
      tr[6] = (unsigned long long)t_wf;
      tr[7] = (unsigned long long)t_busy;
      tr[10] = (unsigned long long)t_ld;
      tr[11] = (unsigned long long)t_rd;
      tr[13] = (unsigned long long)t_issue;
    }
    if (lane == 0) bulk_wait_all();  // Out is written before the CTA leaves
  }

  // ===================== teardown =====================
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, uint32_t(p.tmem_cols));
  }
  if (tr && threadIdx.x == 0) tr[1] = globaltimer_ns();
}

cudaError_t stem_kernel_prepare(int smem_bytes) {
  cudaError_t e = cudaFuncSetAttribute(cconv_stem_kernel<__nv_bfloat16>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(cconv_stem_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              smem_bytes);
}

cudaError_t launch_stem(const CUtensorMap& tm_image, const CUtensorMap& tm_out, const void* filter,
                        bool out_f32, const StemKernelParams& p, int grid, int smem_bytes,
                        int* status, cudaStream_t stream) {
  const unsigned short* f = static_cast<const unsigned short*>(filter);
  if (out_f32)
    cconv_stem_kernel<float><<<grid, kStemThreads, smem_bytes, stream>>>(tm_image, tm_out, f, p, status);
  else
    cconv_stem_kernel<__nv_bfloat16><<<grid, kStemThreads, smem_bytes, stream>>>(tm_image, tm_out, f, p,
                                                                                status);
  return cudaGetLastError();
}

}  // namespace cconv
