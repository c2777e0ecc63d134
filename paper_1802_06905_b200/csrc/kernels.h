// Device kernels of the seven-nested-loop CNN (Eq. 1) and their launchers.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "planner.h"

namespace cconv {

// Bits of the device status word (also returned through cconv_plan_status's detail).
enum : int {
  kStatProducerWait = 1,   // Image producer: a stage never became free
  kStatFilterWait = 32,    // Filter producer: a stage never became free
  kStatMmaWaitFull = 2,    // MMA issuer: a stage never filled
  kStatMmaWaitTmem = 4,    // MMA issuer: an accumulator buffer never drained
  kStatEpilogueWait = 8,   // epilogue: an accumulator never completed
  kStatDrainWait = 16,     // teardown: outstanding MMAs / copies did not retire in time
};

// Everything the halo/tcgen05 kernel needs besides the Image tensor map and the pointers.
// A "unit" is one K=16 step of the contraction: 16 channels x one (r,s) tap; units run
// channel-chunk major, tap minor (u = c16_index * R*S + r*S + s).
struct HaloKernelParams {
  int K, H, W, B, C, R, S, sw, sh;
  int bb, bw, bh, bc;           // block sizes b_b, b_w, b_h, b_c (channels per Image stage)
  int halo_w;                   // Image block extent along w: sw*(bw-1)+R
  int c16;                      // 16-channel chunks of C
  int units;                    // c16 * R*S
  int units_per_img;            // (bc/16) * R*S: units served by one Image stage
  int uf;                       // units per Filter stage
  int i_stages, f_stages;       // ring depths
  int tiles_k, tiles_b, tiles_w, tiles_h;
  int total_tiles;
  int split;                    // 1, or 2 / 4: a cluster of that many CTAs shares one tile, each
                                // contracting an equal share of the channels; partial sums are
                                // exchanged through distributed shared memory and each CTA stores
                                // its share of the columns
  int units_cta;                // units one CTA contracts: units / split
  int cchunks_cta;              // Image stages one CTA loads per tile: ceil(C/bc) / split
  int h0;                       // first output row of this launch (tiles_h counts rows from there)
  int tail;                     // 1: second launch of a call, started while the first still runs
  int image_wait;               // 1: Image overlaps the Out of the call in front of this one on the
                                // stream: the Image producers wait for that call to complete
  int n_mma;                    // N of one MMA = bb*bw
  int acc_cols, acc_bufs, tmem_cols;
  uint32_t img_stage_bytes, filt_stage_bytes;
  uint32_t slab_bytes;          // one Image pixel slab: bc*bb*2
  uint32_t b_kstep_bytes;       // 16 channels of an Image slab: 16*bb*2
  uint32_t idesc;               // tcgen05 instruction descriptor
  uint64_t a_desc, b_desc;      // shared-memory descriptors with a zero start address
  uint64_t wait_limit_ns;       // bound of every device-side wait
  unsigned long long* trace;    // optional [grid][16] globaltimer stamps (diagnostics), or null
};

// One packed Filter block: 128 output channels x 16 input channels of one tap, 4 KB, stored in the
// tensor core's K-major no-swizzle core-matrix order.
constexpr int kPackedBlockBytes = 4096;

// Parameters of the small-C ("stem") tensor-core kernel.  The contraction dimension of one MMA
// runs over consecutive (s, c) rows of the Image, which are contiguous in memory for a fixed first
// subscript; MMA rows = (stacked output row j, out-channel), MMA columns = bw pixels x 64 images.
struct StemKernelParams {
  int K, H, W, B, C, R, S, sw, sh;
  int bw;                 // output pixels per tile along w; MMA N = 64*bw
  int kpad, bhm;          // MMA row = j*kpad + k: bhm output rows stacked in M (kpad*bhm <= 128)
  int kw, khalves;        // rows of the (s,c) window (multiple of 16) and kw/16
  int units;              // MMAs per tile: R * khalves
  int halo_w;             // sw*(bw-1)+R Image columns per tile
  int tiles_k, tiles_w, tiles_h, tiles_b, total_tiles;
  int i_stages;
  int acc_cols, tmem_cols;
  int acc_bufs;           // accumulator buffers of acc_cols columns in tensor memory (2..8)
  uint32_t img_stage_bytes, filt_bytes;
  uint32_t idesc;
  uint64_t a_desc, b_desc;
  uint64_t wait_limit_ns;
  // Hand-over of the packed Filter between the packing kernel and the convolution of one call, which
  // run side by side: every block of the packing kernel adds 1 to *filter_ready when its stores are
  // visible, and the convolution reads the Filter once the counter has reached ready_target (the
  // total over all calls that used this scratch buffer so far).
  unsigned int* filter_ready;
  unsigned int ready_target;
  int wait_prev;          // 1: nothing is read before the stream's earlier work is complete
  unsigned long long* trace;
};

// Parameters of the direct-Filter tensor-core kernel (cconv_direct_kernel).  Same blocked nest as
// the halo kernel, but the Filter is staged straight from [K][R][S][C] by TMA (no packing kernel, no
// scratch): a Filter stage holds `tg` taps x kt*128 out-channels x bc channels as K-major swizzled
// rows of bc*2 bytes.  Contraction order: channel chunk (bc) -> tap -> 16-channel step.
struct DirectKernelParams {
  int K, H, W, B, C, R, S, sw, sh;
  int bb, bw, bh, bc;            // block sizes b_b, b_w, b_h; bc = channels per Image stage = per Filter row
  int kt;                        // blocks of 128 out-channels per CTA (1 or 2): b_k = 128*kt
  int halo_w, halo_h;
  int cchunks;                   // ceil(C/bc)
  int tg, fgroups;               // taps per Filter stage; Filter stages per channel chunk = ceil(R*S/tg)
  int i_stages, f_stages;
  int tiles_k, tiles_b, tiles_w, tiles_h, total_tiles;
  int n_mma;                     // columns of one output row of the tile = bb*bw
  int mma_rows, mma_n;           // MMAs per (tap, 16 channels, out-channel block) and the N of each:
                                 // bh of n_mma columns, or, where the rows of a tile lie at one
                                 // pixel pitch in the stage (no halo between them), 1 of n_mma*bh
  int acc_cols;                  // accumulator columns of one tile = n_mma*bh*kt
  int acc_bufs, tmem_cols;
  int wait_prev;                 // 1: an array of this call overlaps one of a call that may still be
                                 // running on the stream: nothing is read before the stream's
                                 // earlier work is complete
  uint32_t img_stage_bytes, filt_stage_bytes;
  uint32_t filt_tap_bytes;       // one tap of a Filter stage: kt*128 rows of bc*2 bytes
  uint32_t filt_ktile_bytes;     // 128 rows of bc*2 bytes
  uint32_t slab_bytes;           // one Image pixel slab: bc*bb*2
  uint32_t b_kstep_bytes;        // 16 channels of an Image slab: 16*bb*2
  uint32_t idesc;
  uint64_t a_desc, b_desc;       // shared-memory descriptors with a zero start address
  uint64_t wait_limit_ns;
  int out_tma;                   // 1: the Out tensor map is valid and CTAs with a single tile store
                                 // their 128-byte row pieces with TMA tensor stores from shared memory;
                                 // 2: the same, and the map's first coordinate is w*B + b
  int diag_mode;                 // diagnostics (results are meaningless): 1 = stage operands but
                                 // issue no MMA, 2 = issue the MMAs but copy nothing, 3 = the
                                 // epilogue stores nothing, 4 = the epilogue loads no accumulators
  int skip_filter_stage;         // diagnostics: the Filter producer leaves out the stage with this
                                 // sequence number (-1 = none), so that a bounded wait runs out
  unsigned long long* trace;     // optional [grid][16] time stamps, or null
};

cudaError_t direct_kernel_prepare();
cudaError_t launch_direct(const CUtensorMap& tm_image, const CUtensorMap& tm_filter,
                          const CUtensorMap& tm_out, void* out,
                          bool out_f32, const DirectKernelParams& p, int grid, int smem_bytes,
                          int* status, cudaStream_t stream);

cudaError_t launch_simt(const void* image, const void* filter, void* out, bool out_f32,
                        const Dims& d, cudaStream_t stream);

// Element strides of the four subscripts of each array, in the paper's subscript order:
// Image(x, y, c, b), Filter(k, r, s, c), Out(k, h, w, b); `order` lists Out's subscripts
// (0 = k, 1 = h, 2 = w, 3 = b) from the smallest stride to the largest.
struct StridedLayout {
  long long image[4], filter[4], out[4];
  int order[4];
};
cudaError_t launch_simt_strided(const void* image, const void* filter, void* out, bool out_f32,
                                const Dims& d, const StridedLayout& L, cudaStream_t stream);

// Filter [K][R][S][C] -> packed [k-tile][16-channel chunk][tap][4 KB block], zero padded.
// overlap_prev: launch with programmatic stream serialization, so that the packing may run while
// the kernel in front of it in the stream (normally the previous convolution, which signals early)
// is still executing.  Only for callers that alternate between two `packed` buffers: the previous
// convolution still reads the other one.  The packing kernel always ends after its predecessor.
cudaError_t launch_pack_filter(const void* filter, void* packed, const Dims& d, int c16,
                               int tiles_k, bool overlap_prev, cudaStream_t stream);

// Filter [K][R][S][C] -> stem blocks [k-tile][r][16-row slice][128 x 16], the (s,c) run of each r
// repeated once per stacked output row, shifted by that row's window offset, zero padded.
// overlap_prev: as for launch_pack_filter (callers alternate between two buffers); off when the
// Filter may still be being written by the call in front.
cudaError_t launch_pack_filter_stem(const void* filter, void* packed, const Dims& d,
                                    const StemKernelParams& p, bool overlap_prev,
                                    cudaStream_t stream);
// Blocks of that launch (each adds 1 to StemKernelParams::filter_ready).
unsigned int pack_filter_stem_blocks(const StemKernelParams& p);
// Blocks of that launch (each adds 1 to StemKernelParams::filter_ready).
unsigned int pack_filter_stem_blocks(const StemKernelParams& p);
cudaError_t stem_kernel_prepare(int smem_bytes);
cudaError_t launch_stem(const CUtensorMap& tm_image, const void* packed_filter, void* out,
                        bool out_f32, const StemKernelParams& p, int grid, int smem_bytes,
                        int* status, cudaStream_t stream);

cudaError_t halo_kernel_prepare(int smem_bytes);
cudaError_t launch_halo(const CUtensorMap& tm_image, const void* packed_filter, void* out,
                        bool out_f32, const HaloKernelParams& p, int grid, int smem_bytes,
                        int* status, cudaStream_t stream);

}  // namespace cconv
