// Direct-Filter tensor-core kernel for the seven-nested-loop CNN (Eq. 1, Section 2):
//   Out(k,h,w,b) = sum_{c,r,s} Image(r+sw*w, s+sh*h, c, b) * Filter(k,r,s,c)
// Image [Wi][Hi][C][B], Filter [K][R][S][C], Out [K][H][W][B], bf16, last subscript fastest.
//
// The blocked loop nest of Section 5 on one SM, as in cconv_halo_kernel, with two differences:
//   * the Filter block b_k x b_c of a tap is fetched straight from [K][R][S][C] by a 3-D TMA box
//     (channels, out-channels, taps) into K-major swizzled rows, so a call is ONE launch with no
//     scratch memory (the halo kernel repacks the Filter in a kernel of its own);
//   * a CTA may own two blocks of 128 out-channels (b_k = 256) that share every staged Image block,
//     which halves the Image words staged per multiply-add.
// Outer loops {b,k,w,h}_1: the tile loop; outer loop c_1: the two shared-memory rings (an Image
// stage = the halo block b_b x b_c x (sw(b_w-1)+R) x (sh(b_h-1)+S), shared by all R*S taps; a Filter
// stage = tg taps of one channel block); inner loops: tcgen05.mma instructions whose B operand is
// the SAME resident halo block seen through a descriptor shifted by (r, s).
// Contraction order inside a tile: channel block -> tap (r major, s minor) -> 16-channel step.
//
// Calls overlap: the kernel lets the next kernel of the stream start at once
// (griddepcontrol.launch_dependents at entry) and ends only after the kernel in front of it has
// (griddepcontrol.wait before exit), so "kernel n complete" still implies "kernels < n complete".
// Small problems therefore use few, large tiles: several calls run side by side on different SMs.
// When an array of this call overlaps an array of a call that may still be running, the host sets
// wait_prev and the producers start with griddepcontrol.wait.
#include <cuda_bf16.h>

#include "direct_issue.cuh"
#include "kernels.h"
#include "ptx_sm100.cuh"

namespace cconv {

namespace {

// warp 0: Image producer (TMA), warp 1: MMA issuer, warps 2-9: epilogue (two per quarter of the TMEM
// lanes, taking alternate 128-byte pieces of a row: the conversion and shuffle chain of one warp hides
// behind the other's), warp 10: Filter producer
constexpr int kEpiWarps = 8;
constexpr int kFilterWarp = 2 + kEpiWarps;
constexpr int kDirectThreads = 32 * (kFilterWarp + 1);

// All MMAs of one tap: NC16 channel steps x KT out-channel blocks x b_h output rows.  Built by the
// whole warp (uniform values), issued by the elected lane.  `acc` applies to the first channel
// step; later steps always accumulate.  ob[c*BH + hh]: offset of channel step c, output row hh in the
// Image operand; od[kt*BH + hh]: column offset of that accumulator (both hoisted out of the loops).
// For b_h of 1 or 2 the tap goes out as one straight-line PTX block (direct_issue.cuh): the issuing
// thread pays several cycles per instruction, and a tcgen05.mma of 128 x N x 16 occupies the tensor
// pipe for max(N/2, 75) cycles only, so every instruction between two MMAs counts.
template <int BH, int KT, int NC16>
__device__ __forceinline__ void direct_issue_tap(bool leader, int bh, uint32_t d, uint32_t n_mma,
                                                 uint32_t a_lo, uint32_t a_hi, uint32_t b_lo,
                                                 uint32_t b_hi, uint32_t idesc, uint32_t acc,
                                                 uint32_t ktile16, uint32_t kstep16, uint32_t hstep16,
                                                 const uint32_t (&ob)[NC16 * (BH > 0 ? BH : 1)],
                                                 const uint32_t (&od)[KT * (BH > 0 ? BH : 1)]) {
#define CCONV_TAP(B_, K_, N_)                                             \
  if constexpr (BH == B_ && KT == K_ && NC16 == N_) {                     \
    direct_tap_##B_##_##K_##_##N_(leader, d, a_lo, a_hi, b_lo, b_hi, idesc, acc, ob, od); \
    return;                                                               \
  }
  CCONV_TAP(1, 1, 1) CCONV_TAP(1, 1, 2) CCONV_TAP(1, 1, 4) CCONV_TAP(1, 2, 1) CCONV_TAP(1, 2, 2)
  CCONV_TAP(1, 2, 4) CCONV_TAP(2, 1, 1) CCONV_TAP(2, 1, 2) CCONV_TAP(2, 1, 4) CCONV_TAP(2, 2, 1)
  CCONV_TAP(2, 2, 2) CCONV_TAP(2, 2, 4)
#undef CCONV_TAP
  if constexpr (BH == 0) {
#pragma unroll
    for (int c = 0; c < NC16; ++c) {
      const uint32_t accc = c == 0 ? acc : 1u;
#pragma unroll
      for (int kt = 0; kt < KT; ++kt) {
        const uint64_t a_desc =
            (uint64_t(a_hi) << 32) | (a_lo + uint32_t(c) * 2u + uint32_t(kt) * ktile16);
        for (int hh = 0; hh < bh; ++hh)
          umma_bf16_if(leader, d + uint32_t(kt * bh + hh) * n_mma, a_desc,
                       (uint64_t(b_hi) << 32) | (b_lo + uint32_t(c) * kstep16 + uint32_t(hh) * hstep16),
                       idesc, accc);
      }
    }
  }
}

template <typename OutT>
__device__ __forceinline__ void direct_store_partial(OutT* dst, const uint32_t (&v)[32], int n) {
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
__device__ __forceinline__ void direct_store32(OutT* dst, const uint32_t (&v)[32]) {
  if constexpr (sizeof(OutT) == 4) {
#pragma unroll
    for (int j = 0; j < 4; ++j)
      st_global_v8(dst + 8 * j, v[8 * j], v[8 * j + 1], v[8 * j + 2], v[8 * j + 3], v[8 * j + 4],
                   v[8 * j + 5], v[8 * j + 6], v[8 * j + 7]);
  } else {
#pragma unroll
    for (int j = 0; j < 2; ++j)
      st_global_v8(dst + 16 * j, pack_bf16x2(v[16 * j + 0], v[16 * j + 1]),
                   pack_bf16x2(v[16 * j + 2], v[16 * j + 3]), pack_bf16x2(v[16 * j + 4], v[16 * j + 5]),
                   pack_bf16x2(v[16 * j + 6], v[16 * j + 7]), pack_bf16x2(v[16 * j + 8], v[16 * j + 9]),
                   pack_bf16x2(v[16 * j + 10], v[16 * j + 11]),
                   pack_bf16x2(v[16 * j + 12], v[16 * j + 13]),
                   pack_bf16x2(v[16 * j + 14], v[16 * j + 15]));
  }
}

}  // namespace

// BH: MMAs per tap, channel step and out-channel block (b_h, or 1 for merged rows) at compile time
// (0 = any); KT: blocks of 128 out-channels per CTA; NC16: 16-channel steps
// per channel block (b_c / 16).
template <typename OutT, int BH, int KT, int NC16>
__global__ void __launch_bounds__(kDirectThreads, 1)
    cconv_direct_kernel(const __grid_constant__ CUtensorMap tm_image,
                        const __grid_constant__ CUtensorMap tm_filter,
                        const __grid_constant__ CUtensorMap tm_out, OutT* __restrict__ out,
                        const DirectKernelParams p, int* __restrict__ status) {
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
  uint8_t* gen0 = smem_raw + (smem0 - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen0 + (slot_addr - smem0));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen0 + (slot_addr + 4u - smem0));

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
#define CCONV_TRACE(slot)                                                \
  do {                                                                   \
    if (p.trace) p.trace[blockIdx.x * 16 + (slot)] = globaltimer_ns();   \
  } while (0)

  // Set-up is spread over three threads, and each producer issues its first stages as soon as its
  // own barriers exist, before the CTA-wide barrier: the first operands are then on their way while
  // tensor memory is allocated and the other roles get ready.
  uint32_t pre_issued = 0;  // stages this thread's ring received before the CTA-wide barrier
  if (threadIdx.x == 0) {
    // The next kernel of the stream may start now: it takes SMs that this grid does not use.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    CCONV_TRACE(0);
    if (p.trace) {
      uint32_t smid;
      asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
      p.trace[blockIdx.x * 16 + 12] = smid;
    }
    for (int s = 0; s < p.i_stages; ++s) {
      mbar_init(bar_ifull + 8u * s, 1);
      mbar_init(bar_iempty + 8u * s, 1);
    }
    fence_barrier_init();
    if (p.wait_prev) asm volatile("griddepcontrol.wait;" ::: "memory");
    if (int(blockIdx.x) < p.total_tiles) {
      int t = int(blockIdx.x) / p.tiles_k;
      const int bt = t % p.tiles_b; t /= p.tiles_b;
      const int wt = t % p.tiles_w; t /= p.tiles_w;
      const int n_pre = p.i_stages < p.cchunks ? p.i_stages : p.cchunks;
      for (int cc = 0; cc < n_pre; ++cc) {
        const uint32_t full = bar_ifull + 8u * cc;
        if (p.diag_mode == 2) {
          mbar_arrive(full);  // diagnostics: no copies, the MMAs run on whatever the ring holds
        } else {
          mbar_arrive_expect_tx(full, p.img_stage_bytes);
          tma_load_4d(img_ring + cc * p.img_stage_bytes, &tm_image, bt * p.bb, cc * p.bc,
                      wt * p.bw * p.sw, t * p.bh * p.sh, full);
        }
        if (cc == 0) CCONV_TRACE(2);
      }
      pre_issued = uint32_t(n_pre);
    }
  } else if (threadIdx.x == kFilterWarp * 32) {
    for (int s = 0; s < p.f_stages; ++s) {
      mbar_init(bar_ffull + 8u * s, 1);
      mbar_init(bar_fempty + 8u * s, 1);
    }
    fence_barrier_init();
    if (p.wait_prev) asm volatile("griddepcontrol.wait;" ::: "memory");
    if (int(blockIdx.x) < p.total_tiles) {
      const int k0 = (int(blockIdx.x) % p.tiles_k) * 128 * KT;
      const int all = p.cchunks * p.fgroups;
      const int n_pre = p.f_stages < all ? p.f_stages : all;
      for (int q = 0, cc = 0, fg = 0; q < n_pre; ++q) {
        const uint32_t full = bar_ffull + 8u * q;
        if (p.diag_mode == 2) {
          mbar_arrive(full);
        } else if (q != p.skip_filter_stage) {
          mbar_arrive_expect_tx(full, p.filt_stage_bytes);
          tma_load_3d(filt_ring + q * p.filt_stage_bytes, &tm_filter, cc * p.bc, k0, fg * p.tg, full);
        }
        if (++fg == p.fgroups) {
          fg = 0;
          ++cc;
        }
      }
      pre_issued = uint32_t(n_pre);
    }
  } else if (threadIdx.x == 64) {
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull + 8u * a, 1);
      mbar_init(bar_tempty + 8u * a, kEpiWarps);  // one arrival per epilogue warp
    }
    mbar_init(bar_drain, 1);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(slot_addr, uint32_t(p.tmem_cols));
    tmem_relinquish();
    tc_fence_before();
  }
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // The MMA issuer's wait for a stage is the one that names the cause when a copy never lands; the
  // waits that depend on the issuer's progress (producers, epilogue) are given four times its
  // limit, and leave as soon as the issuer has raised the abort flag.
  const uint64_t limit = (warp == 1) ? p.wait_limit_ns : 4 * p.wait_limit_ns;
  if (threadIdx.x == 0) CCONV_TRACE(1);

  if (warp == 0) {
    // ===================== Image halo producer (TMA) =====================
    if (lane == 0) {
      const uint32_t n_st = uint32_t(p.i_stages);
      uint32_t seq = 0, s = 0, ph = 0;
      bool ok = true;
      auto coords = [&](int tile, int& b0, int& x0, int& y0) {
        int t = tile / p.tiles_k;
        const int bt = t % p.tiles_b; t /= p.tiles_b;
        const int wt = t % p.tiles_w; t /= p.tiles_w;
        b0 = bt * p.bb;
        x0 = wt * p.bw * p.sw;
        y0 = t * p.bh * p.sh;
      };
      for (int tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x) {
        int b0, x0, y0;
        coords(tile, b0, x0, y0);
        for (int cc = 0, c0 = 0; cc < p.cchunks; ++cc, c0 += p.bc, ++seq) {
          if (seq >= pre_issued) {  // (the first stages went out before the CTA-wide barrier)
            if (!mbar_wait(bar_iempty + 8u * s, ph ^ 1u, abort_flag, status, kStatProducerWait, limit)) {
              ok = false;
              break;
            }
            const uint32_t full = bar_ifull + 8u * s;
            if (p.diag_mode == 2) {
              mbar_arrive(full);
            } else {
              mbar_arrive_expect_tx(full, p.img_stage_bytes);
              tma_load_4d(img_ring + s * p.img_stage_bytes, &tm_image, b0, c0, x0, y0, full);
            }
          }
          if (++s == n_st) {
            s = 0;
            ph ^= 1u;
          }
        }
      }
      CCONV_TRACE(3);
      drain_ring(bar_ifull, seq, n_st, status, limit);
    }
  } else if (warp == kFilterWarp) {
    // ===================== Filter producer (TMA boxes of tg taps) =====================
    if (lane == 0) {
      const uint32_t n_st = uint32_t(p.f_stages);
      uint32_t seq = 0, s = 0, ph = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x) {
        const int k0 = (tile % p.tiles_k) * 128 * KT;
        for (int cc = 0, c0 = 0; ok && cc < p.cchunks; ++cc, c0 += p.bc) {
          for (int fg = 0, t0 = 0; fg < p.fgroups; ++fg, t0 += p.tg, ++seq) {
            if (seq >= pre_issued) {
              if (!mbar_wait(bar_fempty + 8u * s, ph ^ 1u, abort_flag, status, kStatFilterWait, limit)) {
                ok = false;
                break;
              }
              const uint32_t full = bar_ffull + 8u * s;
              if (p.diag_mode == 2) {
                mbar_arrive(full);
              } else if (int(seq) != p.skip_filter_stage) {
                mbar_arrive_expect_tx(full, p.filt_stage_bytes);
                tma_load_3d(filt_ring + s * p.filt_stage_bytes, &tm_filter, c0, k0, t0, full);
              }
            }
            if (++s == n_st) {
              s = 0;
              ph ^= 1u;
            }
          }
        }
      }
      CCONV_TRACE(4);
      // wait for the copies in flight (all but a stage left out on purpose, which never lands)
      {
        const uint32_t back = seq < n_st ? seq : n_st;
        for (uint32_t j = 0; j < back; ++j) {
          const uint32_t i2 = seq - 1 - j;
          if (int(i2) == p.skip_filter_stage) continue;
          const uint32_t t0s = i2 % n_st, phs = (i2 / n_st) & 1u;
          const uint64_t t0 = globaltimer_ns();
          while (!mbar_try_wait(bar_ffull + 8u * t0s, phs)) {
            if (globaltimer_ns() - t0 > limit) {
              atomicOr(status, kStatDrainWait);
              break;
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer =====================
    const bool leader = elect_one();
    const bool issuer = leader && p.diag_mode != 1;  // diagnostics: stages are consumed without MMAs
    uint32_t iph = 0, fph = 0, abuf = 0, aph = 0;
    bool ok = true, first_tile = true;
    const int S = p.S, RS = p.R * p.S;
    const uint32_t slab16 = p.slab_bytes >> 4, row16 = uint32_t(p.halo_w) * slab16;
    const uint32_t a_lo0 = uint32_t(p.a_desc), a_hi = uint32_t(p.a_desc >> 32);
    const uint32_t b_lo0 = uint32_t(p.b_desc), b_hi = uint32_t(p.b_desc >> 32);
    const uint32_t hstep16 = uint32_t(p.sh * p.halo_w) * slab16;  // next output row
    const uint32_t kstep16 = p.b_kstep_bytes >> 4;
    const uint32_t img16 = p.img_stage_bytes >> 4, filt16 = p.filt_stage_bytes >> 4;
    const uint32_t tap16 = p.filt_tap_bytes >> 4, ktile16 = p.filt_ktile_bytes >> 4;
    const uint32_t img_ring16 = (img_ring >> 4) & 0x3FFFu, filt_ring16 = (filt_ring >> 4) & 0x3FFFu;
    const uint32_t idesc = p.idesc, n_mma = uint32_t(p.mma_n);
    const uint32_t n_ist = uint32_t(p.i_stages), n_fst = uint32_t(p.f_stages);
    const int bh = p.mma_rows, tg = p.tg;  // BH is mma_rows at compile time
    uint32_t ob[NC16 * (BH > 0 ? BH : 1)], od[KT * (BH > 0 ? BH : 1)];
#pragma unroll
    for (int c = 0; c < NC16; ++c)
#pragma unroll
      for (int hh = 0; hh < (BH > 0 ? BH : 1); ++hh)
        ob[c * (BH > 0 ? BH : 1) + hh] = uint32_t(c) * kstep16 + uint32_t(hh) * hstep16;
#pragma unroll
    for (int i = 0; i < KT * (BH > 0 ? BH : 1); ++i) od[i] = uint32_t(i) * n_mma;
    // Ring positions are kept as running addresses (no multiplications in the loop), and nothing
    // but the waits, the issue blocks and the commits sits between two MMAs: the tensor pipe queues
    // very little work, so every instruction of this warp between two issue blocks is idle time.
    uint32_t i_addr16 = img_ring16, f_addr16 = filt_ring16;
    uint32_t i_full = bar_ifull, i_empty = bar_iempty, f_full = bar_ffull, f_empty = bar_fempty;
    const uint32_t i_full_end = bar_ifull + 8u * n_ist, f_full_end = bar_ffull + 8u * n_fst;
    for (int tile = blockIdx.x; ok && tile < p.total_tiles; tile += gridDim.x) {
      if (!mbar_wait_warp(bar_tempty + 8u * abuf, aph ^ 1u, abort_flag, status, kStatMmaWaitTmem, limit))
        break;
      tc_fence_after();
      const uint32_t d_base = tmem_base + abuf * uint32_t(p.acc_cols);
      uint32_t acc = 0;
      const long long tl0 = p.trace ? clock64() : 0;
      if (RS == 1) {
        // 1x1 filters: one tap, one Filter stage per channel block -- the leanest loop
        bool stamp = first_tile && lane == 0;
        for (int cc = p.cchunks; cc > 0; --cc) {
          if (!mbar_wait_warp(i_full, iph, abort_flag, status, kStatMmaWaitFull, limit) ||
              !mbar_wait_warp(f_full, fph, abort_flag, status, kStatMmaWaitFull, limit)) {
            ok = false;
            break;
          }
          tc_fence_after();
          if (stamp) {
            CCONV_TRACE(5);
            stamp = false;
          }
          direct_issue_tap<BH, KT, NC16>(issuer, bh, d_base, n_mma, a_lo0 | f_addr16, a_hi,
                                         b_lo0 | i_addr16, b_hi, idesc, acc, ktile16, kstep16, hstep16,
                                         ob, od);
          acc = 1;
          if (leader) {
            umma_commit(f_empty);
            umma_commit(i_empty);
          }
          f_full += 8u;
          f_empty += 8u;
          f_addr16 += filt16;
          if (f_full == f_full_end) {
            f_full = bar_ffull;
            f_empty = bar_fempty;
            f_addr16 = filt_ring16;
            fph ^= 1u;
          }
          i_full += 8u;
          i_empty += 8u;
          i_addr16 += img16;
          if (i_full == i_full_end) {
            i_full = bar_ifull;
            i_empty = bar_iempty;
            i_addr16 = img_ring16;
            iph ^= 1u;
          }
        }
      } else
      for (int cc = 0; cc < p.cchunks; ++cc) {
        if (!mbar_wait_warp(i_full, iph, abort_flag, status, kStatMmaWaitFull, limit)) {
          ok = false;
          break;
        }
        int tap = 0, sx = 0;
        uint32_t tap_off = i_addr16, col_off = i_addr16;  // Image view of the current tap, in 16 B units
        for (int fg = 0; fg < p.fgroups; ++fg) {
          if (!mbar_wait_warp(f_full, fph, abort_flag, status, kStatMmaWaitFull, limit)) {
            ok = false;
            break;
          }
          tc_fence_after();
          if (first_tile && cc == 0 && fg == 0 && lane == 0) CCONV_TRACE(5);
          uint32_t a16 = f_addr16;
          const int ntap = RS - tap < tg ? RS - tap : tg;
          for (int j = 0; j < ntap; ++j) {
            direct_issue_tap<BH, KT, NC16>(issuer, bh, d_base, n_mma, a_lo0 | a16, a_hi, b_lo0 | tap_off,
                                           b_hi, idesc, acc, ktile16, kstep16, hstep16, ob, od);
            acc = 1;
            a16 += tap16;
            // next tap: one halo row down (s); after S rows one halo pixel to the right (r)
            tap_off += row16;
            if (++sx == S) {
              sx = 0;
              col_off += slab16;
              tap_off = col_off;
            }
          }
          tap += ntap;
          if (leader) umma_commit(f_empty);  // free once the MMAs so far have read it
          f_full += 8u;
          f_empty += 8u;
          f_addr16 += filt16;
          if (f_full == f_full_end) {
            f_full = bar_ffull;
            f_empty = bar_fempty;
            f_addr16 = filt_ring16;
            fph ^= 1u;
          }
        }
        if (!ok) break;
        if (leader) umma_commit(i_empty);
        i_full += 8u;
        i_empty += 8u;
        i_addr16 += img16;
        if (i_full == i_full_end) {
          i_full = bar_ifull;
          i_empty = bar_iempty;
          i_addr16 = img_ring16;
          iph ^= 1u;
        }
      }
      if (!ok) break;
      if (first_tile && lane == 0 && p.trace)
        p.trace[blockIdx.x * 16 + 15] = (unsigned long long)(clock64() - tl0);
      if (leader) umma_commit(bar_tfull + 8u * abuf);  // accumulator complete
      if (first_tile && lane == 0) CCONV_TRACE(6);
      first_tile = false;
      if (++abuf == uint32_t(p.acc_bufs)) {
        abuf = 0;
        aph ^= 1u;
      }
    }
    // All MMAs must have retired before TMEM is released.
    if (lane == 0) CCONV_TRACE(7);
    if (leader) umma_commit(bar_drain);
    const uint64_t t0 = globaltimer_ns();
    while (!mbar_try_wait(bar_drain, 0)) {
      if (globaltimer_ns() - t0 > limit) {
        atomicOr(status, kStatDrainWait);
        break;
      }
    }
  } else if (warp >= 2 && warp < 2 + kEpiWarps) {
    // ===================== epilogue: TMEM -> registers -> Out =====================
    const int q = warp & 3;  // this warp may touch TMEM lanes [32q, 32q+32)
    const int part = (warp - 2) >> 2;   // which of the quarter's warps this is
    constexpr int kParts = kEpiWarps / 4;
    uint32_t abuf = 0, aph = 0;
    bool first_tile = true;
    const bool wide_rows = (size_t(p.B) * sizeof(OutT)) % 32 == 0;
    for (int tile = blockIdx.x; tile < p.total_tiles; tile += gridDim.x) {
      int t = tile;
      const int ktile = t % p.tiles_k; t /= p.tiles_k;
      const int bt = t % p.tiles_b; t /= p.tiles_b;
      const int wt = t % p.tiles_w; t /= p.tiles_w;
      const int ht = t;
      const int b0 = bt * p.bb;
      // (every lane polls for itself and checks the abort flag each time; the decision to go on
      // must be the same in all lanes because the TMEM loads below are warp-wide)
      // One lane polls, with pauses: 256 threads polling shared memory while the main loop runs would
      // compete with the tensor core's own operand reads.
      bool got = true;
      if (lane == 0) {
        uint64_t t0 = 0;
        while (!mbar_try_wait(bar_tfull + 8u * abuf, aph)) {
          __nanosleep(256);
          if (*abort_flag) {
            got = false;
            break;
          }
          const uint64_t t = globaltimer_ns();
          if (t0 == 0) {
            t0 = t;
          } else if (t - t0 > limit) {
            *abort_flag = 1;
            atomicOr(status, kStatEpilogueWait);
            got = false;
            break;
          }
        }
      }
      if (!__shfl_sync(0xffffffffu, got, 0)) break;
      tc_fence_after();
      if (first_tile && threadIdx.x == 64) CCONV_TRACE(8);
      const uint32_t t_base = tmem_base + (uint32_t(q * 32) << 16) + abuf * uint32_t(p.acc_cols);
      // A lane holds one out-channel row of the accumulator.  Stored lane by lane, a warp's store
      // instruction would touch 32 different lines (one sector per out-channel plane), which an SM
      // gets rid of at about 20 B/clk; whole 128-byte lines leave at 32 B/clk (measured).  So the
      // four lanes of a quad exchange 32-byte sectors by warp shuffles (a 4x4 transpose) and then
      // write the 128-byte piece of ONE row per store instruction: lane j of the quad stores sector
      // j of the quad's rows 0..3.  A piece is 64 columns (bf16) or 32 columns (fp32).
      constexpr int kPiece = sizeof(OutT) == 2 ? 64 : 32;   // columns per 128-byte piece
      constexpr int kSec = kPiece / 4;                       // columns per 32-byte sector
      const long long plane = (long long)p.H * p.W * p.B;   // elements of one out-channel plane
      const int bb_shift = p.bb == 64 ? 6 : 5;
      const int sj = lane & 3;
      // A CTA with a single tile: the rings are idle by now and serve as staging memory, 8 KB per
      // epilogue warp.
      const bool idle_rings = p.total_tiles <= int(gridDim.x) && uint32_t(kEpiWarps) * 8192u <= bars - smem0;
      const uint32_t stage = smem0 + uint32_t(warp - 2) * 8192u;
      // With a tensor map of Out, every piece is stored by the TMA engine from a swizzled 4 KB
      // buffer (two per warp, so a warp converts its next piece while the last one drains); the
      // engine clips what lies outside Out.  Else the quad's sectors are exchanged -- through the
      // staging memory if there is some, by shuffles otherwise -- and stored by the lanes.
      const bool via_tma = idle_rings && p.out_tma != 0 && p.diag_mode != 3;
      const bool via_smem = idle_rings;
      uint32_t n_stored = 0;  // pieces this warp handed to the TMA engine
#pragma unroll
      for (int kt = 0; kt < KT; ++kt) {
        const int kw = (ktile * KT + kt) * 128 + q * 32;  // first out-channel of this warp's 32 rows
        const int kq = kw + (lane & ~3);                  // first row of this lane's quad
        for (int hh = 0; hh < p.bh; ++hh) {
          const int h = ht * p.bh + hh;
          if (h >= p.H) continue;
          OutT* const roww = out + (((long long)kw * p.H + h) * p.W + wt * p.bw) * p.B + b0;
          OutT* const rowq = roww + (long long)(lane & ~3) * plane;
          const uint32_t col0 = uint32_t((kt * p.bh + hh) * p.n_mma);
          for (int c = part * kPiece; c + kPiece <= p.n_mma; c += kParts * kPiece) {
            uint32_t va[32], sec[4][8];
            if (p.diag_mode != 4) tmem_ld_32x32b_x32(t_base + col0 + uint32_t(c), va);
            if constexpr (sizeof(OutT) == 2) {
              uint32_t vb[32];
              if (p.diag_mode != 4) tmem_ld_32x32b_x32(t_base + col0 + uint32_t(c + 32), vb);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                sec[0][i] = pack_bf16x2(va[2 * i], va[2 * i + 1]);
                sec[1][i] = pack_bf16x2(va[16 + 2 * i], va[17 + 2 * i]);
                sec[2][i] = pack_bf16x2(vb[2 * i], vb[2 * i + 1]);
                sec[3][i] = pack_bf16x2(vb[16 + 2 * i], vb[17 + 2 * i]);
              }
            } else {
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 32; ++i) sec[i >> 3][i & 7] = va[i];
            }
            if (via_tma) {
              const uint32_t buf = stage + (n_stored & 1u) * 4096u;
              if (n_stored >= 2) {  // the store that read this buffer two pieces ago
                if (lane == 0) bulk_wait_group_read<1>();
                __syncwarp();
              }
              // lane = row of the box; its eight 16-byte chunks land XOR-swizzled by the row (the
              // 128-byte swizzle of the tensor map), which also keeps the stores free of conflicts
              const uint32_t rowa = buf + uint32_t(lane) * 128u;
              const uint32_t x = uint32_t(lane & 7);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                st_shared_v4(rowa + (((2u * i) ^ x) << 4), sec[i][0], sec[i][1], sec[i][2], sec[i][3]);
                st_shared_v4(rowa + (((2u * i + 1u) ^ x) << 4), sec[i][4], sec[i][5], sec[i][6], sec[i][7]);
              }
              fence_proxy_async_smem();
              __syncwarp();
              if (lane == 0) {
                const int ww0 = c >> bb_shift, bb0 = c - (ww0 << bb_shift);
                const int w = wt * p.bw + ww0;
                if (p.out_tma == 2) tma_store_4d(&tm_out, buf, w * p.B + b0 + bb0, 0, h, kw);
                else tma_store_4d(&tm_out, buf, b0 + bb0, w, h, kw);
                bulk_commit_group();
              }
              ++n_stored;
              continue;
            }
            // the sector this lane stores: columns cc .. cc + kSec of the run = images b .. of pixel ww
            const int cc = c + kSec * sj;
            const int ww = cc >> bb_shift, b = cc - (ww << bb_shift);
            const int left = p.B - (b0 + b);   // images of the sector inside the batch (a multiple of 8)
            int row0, row_step;                 // this lane stores rows row0 + j*row_step of the warp's 32
            if (via_smem) {
              // The 4x4 exchange of sectors through shared memory (16 vector accesses instead of
              // 64 shuffles and as many selects): every lane parks its 128-byte piece in a row of
              // 144 bytes (the pitch keeps both phases free of bank conflicts), then reads sector sj
              // of rows 8j + lane/4.
              const uint32_t wrow = stage + uint32_t(lane) * 144u;
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                st_shared_v4(wrow + 32u * i, sec[i][0], sec[i][1], sec[i][2], sec[i][3]);
                st_shared_v4(wrow + 32u * i + 16u, sec[i][4], sec[i][5], sec[i][6], sec[i][7]);
              }
              __syncwarp();
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const uint32_t rrow = stage + uint32_t(8 * j + (lane >> 2)) * 144u + 32u * uint32_t(sj);
                ld_shared_v4(rrow, sec[j][0], sec[j][1], sec[j][2], sec[j][3]);
                ld_shared_v4(rrow + 16u, sec[j][4], sec[j][5], sec[j][6], sec[j][7]);
              }
              __syncwarp();
              row0 = lane >> 2;
              row_step = 8;
            } else {
              quad_transpose_sectors(sec, lane);
              row0 = lane & ~3;
              row_step = 1;
            }
            if (wt * p.bw + ww < p.W && left > 0 && p.diag_mode != 3) {
              OutT* const d0 = roww + (long long)row0 * plane + (long long)ww * p.B + b;
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                if (kw + row0 + j * row_step >= p.K) continue;
                OutT* dst = d0 + (long long)(j * row_step) * plane;
                if (left >= kSec && wide_rows) {
                  st_global_v8(dst, sec[j][0], sec[j][1], sec[j][2], sec[j][3], sec[j][4], sec[j][5],
                               sec[j][6], sec[j][7]);
                } else {
                  // rows of Out that are not multiples of 32 bytes, or (bf16) a sector cut in half by
                  // the end of the batch: 16-byte pieces
                  *reinterpret_cast<uint4*>(dst) = make_uint4(sec[j][0], sec[j][1], sec[j][2], sec[j][3]);
                  if (left >= kSec)
                    *reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(dst) + 16) =
                        make_uint4(sec[j][4], sec[j][5], sec[j][6], sec[j][7]);
                }
              }
            }
          }
          const int c = p.n_mma & ~(kPiece - 1);
          if (c < p.n_mma && part == 0) {
            // bf16, n_mma = 32 mod 64: the last 32 columns (one pixel of a 32-image block), lane by lane
            uint32_t v[32];
            tmem_ld_32x32b_x32(t_base + col0 + uint32_t(c), v);
            tmem_ld_wait();
            const int ww = c >> bb_shift, b = c - (ww << bb_shift);
            const int k = kq + sj, nb = p.B - (b0 + b);
            if (k < p.K && wt * p.bw + ww < p.W && nb > 0) {
              OutT* dst = rowq + sj * plane + (long long)ww * p.B + b;
              if (nb >= 32 && wide_rows) direct_store32(dst, v);
              else direct_store_partial(dst, v, nb < 32 ? nb : 32);
            }
          }
        }
      }
      if (via_tma) {  // Out is complete before this CTA reports completion
        if (lane == 0) bulk_wait_group<0>();
        __syncwarp();
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

  // ===================== teardown =====================
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, uint32_t(p.tmem_cols));
  }
  // This kernel may have run beside the kernels in front of it; it ends only after they have.
  if (threadIdx.x == 0) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    CCONV_TRACE(11);
  }
#undef CCONV_TRACE
}

namespace {

template <typename OutT>
using DirectFn = void (*)(CUtensorMap, CUtensorMap, CUtensorMap, OutT*, DirectKernelParams, int*);

template <typename OutT, int KT, int NC16>
DirectFn<OutT> direct_fn_bh(int bh) {
  switch (bh) {
    case 1: return cconv_direct_kernel<OutT, 1, KT, NC16>;
    case 2: return cconv_direct_kernel<OutT, 2, KT, NC16>;
    default: return cconv_direct_kernel<OutT, 0, KT, NC16>;
  }
}

template <typename OutT, int KT>
DirectFn<OutT> direct_fn_nc(int nc16, int bh) {
  switch (nc16) {
    case 1: return direct_fn_bh<OutT, KT, 1>(bh);
    case 2: return direct_fn_bh<OutT, KT, 2>(bh);
    default: return direct_fn_bh<OutT, KT, 4>(bh);
  }
}

template <typename OutT>
DirectFn<OutT> direct_fn(int kt, int nc16, int bh) {
  return kt == 2 ? direct_fn_nc<OutT, 2>(nc16, bh) : direct_fn_nc<OutT, 1>(nc16, bh);
}

template <typename OutT>
cudaError_t direct_prepare_all(int smem_bytes) {
  for (int kt : {1, 2})
    for (int nc : {1, 2, 4})
      for (int bh : {1, 2, 3}) {
        cudaError_t e = cudaFuncSetAttribute(direct_fn<OutT>(kt, nc, bh),
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
        if (e != cudaSuccess) return e;
      }
  return cudaSuccess;
}

}  // namespace

// The dynamic shared-memory ceiling of every instantiation is raised to the device's limit (the
// attribute is per kernel and the last value wins, so it is never set to one plan's need).
cudaError_t direct_kernel_prepare() {
  int dev = 0, cap = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&cap, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e != cudaSuccess) return e;
  e = direct_prepare_all<__nv_bfloat16>(cap);
  if (e != cudaSuccess) return e;
  return direct_prepare_all<float>(cap);
}

cudaError_t launch_direct(const CUtensorMap& tm_image, const CUtensorMap& tm_filter,
                          const CUtensorMap& tm_out, void* out, bool out_f32, const DirectKernelParams& p, int grid, int smem_bytes,
                          int* status, cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(grid));
  cfg.blockDim = dim3(kDirectThreads);
  cfg.dynamicSmemBytes = size_t(smem_bytes);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const int nc16 = p.bc / 16;
  if (out_f32)
    return cudaLaunchKernelEx(&cfg, direct_fn<float>(p.kt, nc16, p.mma_rows), tm_image, tm_filter,
                              tm_out, static_cast<float*>(out), p, status);
  return cudaLaunchKernelEx(&cfg, direct_fn<__nv_bfloat16>(p.kt, nc16, p.mma_rows), tm_image, tm_filter,
                            tm_out, static_cast<__nv_bfloat16*>(out), p, status);
}

}  // namespace cconv
