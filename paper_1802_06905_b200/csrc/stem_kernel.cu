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
//   A (rows)  = Filter column r, K-major, resident in shared memory for the whole kernel.  When
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
constexpr int kStemEpiThreads = 256;              // 8 warps: two per TMEM lane quarter (16 warps spill: 39 us)
constexpr int kStemThreads = 64 + kStemEpiThreads;
constexpr int kFiltBars = 16;  // 16 KB Filter pieces: at most 14 fit in shared memory
constexpr int kMaxAccBufs = 8;  // accumulator buffers in tensor memory: tmem_cols / acc_cols

}  // namespace

// ------------------------------------------------------------------------------------------------
// Filter packing for the stem kernel.  Block (kt, r, kh) holds 128 rows x 16 window rows: row
// j*kpad + kk, column jj carries Filter[kt*128 + kk][r][s][c] with s*C + c = kh*16 + jj - j*sh*C
// (zero outside 0 .. S*C-1, for k >= K and for j >= bhm), in K-major no-swizzle core-matrix order:
// element (row, jj) at ((row/8)*2 + jj/8)*128 + (row%8)*16 + (jj%8)*2 bytes.  Since (s, c) is
// contiguous in Filter, the value is element q = kh*16 + jj - j*sh*C of the run Filter[k][r][.][.].
// One thread writes 16 bytes.  The kernel lets its dependent (the convolution) start at once and
// does not finish before the kernel in front of it has (see launch_pack_filter).
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
    cconv_pack_filter_stem_kernel(const unsigned short* __restrict__ filter,
                                  uint4* __restrict__ packed, Dims d, int kpad, int bhm, int khalves,
                                  long long slots, unsigned int* __restrict__ ready) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const long long slot = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (slot < slots) {
    const int j16 = int(slot & 255);  // 16-byte slot inside the 4 KB block
    long long blk = slot >> 8;
    const int kh = int(blk % khalves);
    blk /= khalves;
    const int r = int(blk % d.R);
    const int kt = int(blk / d.R);
    const int core = j16 >> 3, row8 = j16 & 7;
    const int row = (core >> 1) * 8 + row8;
    const int jj0 = (core & 1) * 8;
    const int j = row / kpad, kk = row - j * kpad;
    const int k = kt * 128 + kk;
    const int SC = d.S * d.C;
    const int q0 = kh * 16 + jj0 - j * d.sh * d.C;
    unsigned short e[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) e[i] = 0;
    if (k < d.K && j < bhm && q0 + 8 > 0 && q0 < SC) {
      const unsigned short* run = filter + ((long long)k * d.R + r) * SC;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int q = q0 + i;
        if (q >= 0 && q < SC) e[i] = __ldg(run + q);
      }
    }
    uint4 o;
    o.x = e[0] | (uint32_t(e[1]) << 16);
    o.y = e[2] | (uint32_t(e[3]) << 16);
    o.z = e[4] | (uint32_t(e[5]) << 16);
    o.w = e[6] | (uint32_t(e[7]) << 16);
    packed[slot] = o;
  }
  // This block's part of the packed Filter is written: make it visible and count the block in.  The
  // convolution of the same call (already running beside this kernel) reads the Filter once every
  // block has been counted.
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0 && ready != nullptr) atomicAdd(ready, 1u);
  // The kernel ends only after the kernel in front of it has (completion stays in stream order).
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

unsigned int pack_filter_stem_blocks(const StemKernelParams& p) {
  return unsigned(((long long)p.filt_bytes / 16 + 255) / 256);
}

cudaError_t launch_pack_filter_stem(const void* filter, void* packed, const Dims& d,
                                    const StemKernelParams& p, bool overlap_prev,
                                    cudaStream_t stream) {
  const long long slots = (long long)p.filt_bytes / 16;
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
  return cudaLaunchKernelEx(&cfg, cconv_pack_filter_stem_kernel,
                            static_cast<const unsigned short*>(filter), static_cast<uint4*>(packed), d,
                            p.kpad, p.bhm, p.khalves, slots, p.filter_ready);
}

// ------------------------------------------------------------------------------------------------
// The kernel.  Persistent; tile = (128 out-channels) x (64 images) x (bhm output rows) x (bw pixels).
// ------------------------------------------------------------------------------------------------
template <typename OutT>
__global__ void __launch_bounds__(kStemThreads, 1)
    cconv_stem_kernel(const __grid_constant__ CUtensorMap tm_image,
                      const uint8_t* __restrict__ packed_filter, OutT* __restrict__ out,
                      const StemKernelParams p, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem0 = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t img_ring = smem0;
  const uint32_t filt_smem = img_ring + uint32_t(p.i_stages) * p.img_stage_bytes;
  const uint32_t bars = filt_smem + p.filt_bytes;
  const uint32_t bar_ifull = bars;
  const uint32_t bar_iempty = bar_ifull + 8u * p.i_stages;
  const uint32_t bar_filt = bar_iempty + 8u * p.i_stages;
  const uint32_t bar_tfull = bar_filt + 8u * kFiltBars;  // one Filter barrier per 16 KB piece
  const uint32_t bar_tempty = bar_tfull + 8u * kMaxAccBufs;
  const uint32_t bar_drain = bar_tempty + 8u * kMaxAccBufs;
  const uint32_t slot_addr = bar_drain + 8u;
  uint8_t* gen0 = smem_raw + (smem0 - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen0 + (slot_addr - smem0));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen0 + (slot_addr + 4u - smem0));

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // diagnostics: per-CTA row of 16 counters (0 entry ns, 1 exit ns, 2.. cycles spent per role)
  unsigned long long* const tr = p.trace ? p.trace + 16ull * blockIdx.x : nullptr;
  if (tr && threadIdx.x == 0) {
    tr[0] = globaltimer_ns();
    tr[11] = (unsigned long long)clock64();
  }

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.i_stages; ++s) {
      mbar_init(bar_ifull + 8u * s, 1);
      mbar_init(bar_iempty + 8u * s, 1);
    }
    for (int f = 0; f < kFiltBars; ++f) mbar_init(bar_filt + 8u * f, 1);
    for (int a = 0; a < kMaxAccBufs; ++a) {
      mbar_init(bar_tfull + 8u * a, 1);
      mbar_init(bar_tempty + 8u * a, kStemEpiThreads / 32);  // one arrival per epilogue warp
    }
    mbar_init(bar_drain, 1);
    *abort_flag = 0;
    fence_barrier_init();
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
  const bool wide_rows = (size_t(p.B) * sizeof(OutT)) % 32 == 0;  // 32-byte stores stay aligned
  const int shc = p.sh * p.C;  // Image rows (of the merged (y,c) axis) per output row

  if (warp == 0) {
    // ===================== producer: one Image window per tile =====================
    if (lane == 0) {
      uint32_t it = 0, s = 0, ph = 0;
      bool ok = true;
      long long t_wait = 0;
      const uint32_t n_st = uint32_t(p.i_stages);
      // An Image (or Filter) that a call still running may be writing: wait for the stream's
      // earlier work first.  Otherwise this kernel runs beside the kernels in front of it.
      if (p.wait_prev) asm volatile("griddepcontrol.wait;" ::: "memory");
      // The first Image window goes out before the Filter: the first MMA needs both, and one
      // thread's copies are issued one after the other.
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
        if (it == 0) {
          // The packed Filter comes from the packing kernel of this call, which runs beside this
          // kernel: wait (bounded) until all its blocks have counted themselves in, then order the
          // copies below behind that observation.
          if (p.filter_ready != nullptr) {
            const uint64_t t0 = globaltimer_ns();
            unsigned int seen;
            for (;;) {
              asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(p.filter_ready) : "memory");
              if (int(seen - p.ready_target) >= 0) break;
              if (*abort_flag || globaltimer_ns() - t0 > limit) {
                *abort_flag = 1;
                atomicOr(status, kStatFilterWait);
                ok = false;
                break;
              }
              __nanosleep(64);
            }
            if (!ok) break;
            asm volatile("fence.proxy.async;" ::: "memory");
          }
          // the Filter in 16 KB pieces (four 4 KB blocks), each with its own barrier: the MMAs of
          // the first tile start on the first piece while the others are still in flight
          for (uint32_t off = 0, f = 0; off < p.filt_bytes; off += 16384u, ++f) {
            const uint32_t n = p.filt_bytes - off < 16384u ? p.filt_bytes - off : 16384u;
            mbar_arrive_expect_tx(bar_filt + 8u * f, n);
            bulk_load(filt_smem + off, packed_filter + off, n, bar_filt + 8u * f);
          }
        }
      }
      if (tr) tr[2] = (unsigned long long)t_wait;
      drain_ring(bar_ifull, it, n_st, status, limit);
      const uint64_t t0 = globaltimer_ns();
      for (uint32_t f = 0; ok && f < (p.filt_bytes + 16383u) / 16384u; ++f) {
        while (!mbar_try_wait(bar_filt + 8u * f, 0)) {
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
    const uint32_t n_ist = uint32_t(p.i_stages), n_acc = uint32_t(p.acc_bufs);
    const uint32_t a_lo0 = uint32_t(p.a_desc), a_hi = uint32_t(p.a_desc >> 32);
    const uint32_t b_lo0 = uint32_t(p.b_desc), b_hi = uint32_t(p.b_desc >> 32);
    const uint32_t img16 = p.img_stage_bytes >> 4;
    const uint32_t img_ring16 = img_ring >> 4, filt16 = filt_smem >> 4;
    const uint32_t idesc = p.idesc;
    const int units = p.units;
    const uint32_t kt_step16 = uint32_t(units) * 256u;  // one k-tile of the Filter: units x 4 KB
    long long t_filt = 0, t_wt = 0, t_wi = 0, t_issue = 0, n_tiles = 0;
    bool ok = true, filt_ready = false;
    const uint32_t filt_pieces = (p.filt_bytes + 16383u) / 16384u;
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
      if (!filt_ready) {
        // first tile of this CTA: wait for each 16 KB piece of the Filter when its first block is
        // due, then (after the last MMA is issued) for the rest of the Filter
        const long long f0 = tr ? clock64() : 0;
        uint32_t blk = kt * uint32_t(units), waited = 0xffffffffu;
        for (int u = 0; ok && u < units; ++u, ++blk) {
          if ((blk >> 2) != waited) {
            waited = blk >> 2;
            ok = mbar_wait_warp(bar_filt + 8u * waited, 0, abort_flag, status, kStatMmaWaitFull, limit);
            tc_fence_after();
          }
          if (ok)
            umma_bf16_if(leader, d, (uint64_t(a_hi) << 32) | a16, (uint64_t(b_hi) << 32) | b16, idesc,
                         u ? 1u : 0u);
          a16 += 256u;
          b16 += 128u;
        }
        for (uint32_t f = 0; ok && f < filt_pieces; ++f)
          ok = mbar_wait_warp(bar_filt + 8u * f, 0, abort_flag, status, kStatMmaWaitFull, limit);
        tc_fence_after();
        filt_ready = true;
        // The Filter of this CTA is resident: once every CTA is that far, the scratch buffer may be
        // rewritten, so the kernels behind this one may start (the next call's packing kernel and
        // convolution run beside this kernel's remaining tiles).
        if (lane == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        if (tr) t_filt = clock64() - f0;
        if (!ok) break;
      } else {
        umma_bf16_if(leader, d, (uint64_t(a_hi) << 32) | a16, (uint64_t(b_hi) << 32) | b16, idesc, 0u);
#pragma unroll 2
        for (int u = 1; u < units; ++u) {
          a16 += 256u;
          b16 += 128u;
          umma_bf16_if(leader, d, (uint64_t(a_hi) << 32) | a16, (uint64_t(b_hi) << 32) | b16, idesc,
                       1u);
        }
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
      if (++abuf == n_acc) {
        abuf = 0;
        aph ^= 1u;
      }
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
    const int eset = (warp - 2) >> 2;  // which of the quarter's warps: pixels eset, eset + 2, ... of a tile
    // TMEM lane L = j*kpad + kk: stacked output row j, out-channel kk (kpad is a power of two).  A
    // lane reads the 64 images of one pixel of its row; the sectors are then transposed within
    // quads of lanes (quad_transpose_sectors) so that a quad writes whole lines of Out.
    constexpr int kSectorElems = 32 / int(sizeof(OutT));  // images per 32-byte sector: 16 / 8
    constexpr int kPasses = int(sizeof(OutT)) / 2;         // 128-byte row pieces per pixel: 1 / 2
    const int kpad_log2 = 31 - __clz(p.kpad);
    const int sector = lane & 3;                           // the sector this lane stores
    const long long plane_row = (long long)p.W * p.B;      // elements per (k, h) row of Out
    uint32_t abuf = 0, aph = 0;
    const uint32_t n_acc = uint32_t(p.acc_bufs);
    long long t_wf = 0, t_busy = 0, t_ld = 0;
    for (int tile = blockIdx.x; tile < p.total_tiles; tile += gridDim.x) {
      int t = tile;
      const int kt = t % p.tiles_k;
      t /= p.tiles_k;
      const int wt = t % p.tiles_w;
      t /= p.tiles_w;
      const int ht = t % p.tiles_h, bt = t / p.tiles_h;
      // the four rows of this lane's quad: accumulator rows 4*(lane/4) + j of the warp's 32
      OutT* rowp[4];
      uint32_t row_ok = 0;
      const long long tile_off = (long long)(wt * p.bw) * p.B + bt * 64 + sector * kSectorElems;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int L = q * 32 + 4 * (lane >> 2) + j;
        const int jr = L >> kpad_log2, kk = L & (p.kpad - 1);
        const int k = kt * 128 + kk, h = ht * p.bhm + jr;
        if (k < p.K && jr < p.bhm && h < p.H) row_ok |= 1u << j;
        rowp[j] = out + ((long long)k * p.H + h) * plane_row + tile_off;
      }
      const int nb = p.B - bt * 64;  // images left in the batch (the block is padded past B)
      const long long c0 = tr ? clock64() : 0;
      if (!mbar_wait_warp(bar_tfull + 8u * abuf, aph, abort_flag, status, kStatEpilogueWait, limit))
        break;
      const long long c1 = tr ? clock64() : 0;
      tc_fence_after();
      const uint32_t t_base = tmem_base + (uint32_t(q * 32) << 16) + abuf * uint32_t(p.acc_cols);
      for (int px = eset; px < p.bw; px += kStemEpiThreads / 128) {
        uint32_t va[32], vb[32];
        const long long l0 = tr ? clock64() : 0;
        tmem_ld_32x32b_x32(t_base + uint32_t(px * 64), va);
        tmem_ld_32x32b_x32(t_base + uint32_t(px * 64 + 32), vb);
        tmem_ld_wait();
        if (tr) t_ld += clock64() - l0;
        const bool px_ok = wt * p.bw + px < p.W;
#pragma unroll
        for (int pass = 0; pass < kPasses; ++pass) {
          uint32_t sec[4][8];  // this lane's 128-byte row piece as four sectors
          if constexpr (sizeof(OutT) == 2) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              sec[0][i] = pack_bf16x2(va[2 * i], va[2 * i + 1]);
              sec[1][i] = pack_bf16x2(va[16 + 2 * i], va[17 + 2 * i]);
              sec[2][i] = pack_bf16x2(vb[2 * i], vb[2 * i + 1]);
              sec[3][i] = pack_bf16x2(vb[16 + 2 * i], vb[17 + 2 * i]);
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) sec[i >> 3][i & 7] = pass == 0 ? va[i] : vb[i];
          }
          quad_transpose_sectors(sec, lane);
          // first image (within the block of 64) of the sector this lane stores
          const int first = sector * kSectorElems + pass * 32;
          const int left = nb - first;  // images of the sector inside the batch (a multiple of 8)
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            if (!px_ok || !((row_ok >> j) & 1u) || left <= 0) continue;
            OutT* dst = rowp[j] + (long long)px * p.B + pass * 32;
            if (left >= kSectorElems && wide_rows) {
              st_global_v8(dst, sec[j][0], sec[j][1], sec[j][2], sec[j][3], sec[j][4], sec[j][5],
                           sec[j][6], sec[j][7]);
            } else {
              // rows of Out that are not multiples of 32 bytes, or a sector cut by the end of the
              // batch (bf16 only: half a sector = 8 images): 16-byte pieces
              *reinterpret_cast<uint4*>(dst) = make_uint4(sec[j][0], sec[j][1], sec[j][2], sec[j][3]);
              if (left >= kSectorElems)
                *reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(dst) + 16) =
                    make_uint4(sec[j][4], sec[j][5], sec[j][6], sec[j][7]);
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty + 8u * abuf);
      if (++abuf == n_acc) {
        abuf = 0;
        aph ^= 1u;
      }
      if (tr) {
        t_wf += c1 - c0;
        t_busy += clock64() - c1;
      }
    }
    if (tr && warp == 4 && lane == 0) {
      tr[6] = (unsigned long long)t_wf;
      tr[7] = (unsigned long long)t_busy;
      tr[10] = (unsigned long long)t_ld;
    }
  }

  // ===================== teardown =====================
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, uint32_t(p.tmem_cols));
  }
  // This kernel ran beside the kernels in front of it; it ends only after they have.
  if (threadIdx.x == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
  if (tr && threadIdx.x == 0) {
    tr[1] = globaltimer_ns();
    tr[12] = (unsigned long long)clock64();
  }
}

// (The attribute is a per-kernel ceiling and the value set last wins: it is raised to the device's
// limit, never to one plan's need, since several plans share the kernel.)
cudaError_t stem_kernel_prepare(int smem_bytes) {
  int dev = 0, cap = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&cap, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e != cudaSuccess) return e;
  if (smem_bytes > cap) return cudaErrorInvalidValue;
  e = cudaFuncSetAttribute(cconv_stem_kernel<__nv_bfloat16>,
                           cudaFuncAttributeMaxDynamicSharedMemorySize, cap);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(cconv_stem_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              cap);
}

cudaError_t launch_stem(const CUtensorMap& tm_image, const void* packed_filter, void* out,
                        bool out_f32, const StemKernelParams& p, int grid, int smem_bytes,
                        int* status, cudaStream_t stream) {
  const uint8_t* pf = static_cast<const uint8_t*>(packed_filter);
  // Programmatic dependent launch: the kernel may begin while the Filter-packing kernel in front of
  // it is still running; only its producer waits for that kernel's results.
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
    return cudaLaunchKernelEx(&cfg, cconv_stem_kernel<float>, tm_image, pf, static_cast<float*>(out),
                              p, status);
  return cudaLaunchKernelEx(&cfg, cconv_stem_kernel<__nv_bfloat16>, tm_image, pf,
                            static_cast<__nv_bfloat16*>(out), p, status);
}

}  // namespace cconv
