// Host-side tile planner: Theorem 1 evaluation, the Section-5 tiling LP, and the hardware legaliser
// that turns the LP's continuous block sizes into a tile the sm_100a kernels can run.
#pragma once
#include <cstdint>

namespace cconv {

struct Dims {
  int B, C, K, W, H, R, S, sw, sh;
  int Wi() const { return sw * (W - 1) + R; }
  int Hi() const { return sh * (H - 1) + S; }
  double macs() const { return double(B) * C * K * W * H * R * S; }
  bool positive() const {
    return B > 0 && C > 0 && K > 0 && W > 0 && H > 0 && R > 0 && S > 0 && sw > 0 && sh > 0;
  }
};

// How the tensor-core kernels see the Image.  A 1x1 filter with strides touches only every sw-th
// column and sh-th row, so those kernels run the unstrided problem `dk` on a strided view of the
// array (same Filter, same Out) and never fetch the skipped pixels.  Strides are in elements,
// between consecutive view rows (the h direction) and view columns (the w direction).
struct ImageView {
  Dims dk;
  long long stride_h, stride_w;
  long long stride_c;  // between consecutive channels (B for a dense Image; b itself is contiguous)
};
inline ImageView image_view(const Dims& d) {
  ImageView v{d, (long long)d.C * d.B, (long long)d.Hi() * d.C * d.B, (long long)d.B};
  if (d.R == 1 && d.S == 1 && (d.sw > 1 || d.sh > 1)) {
    v.stride_h *= d.sh;
    v.stride_w *= d.sw;
    v.dk.sw = v.dk.sh = 1;
  }
  return v;
}

// What the device offers; filled from cudaGetDeviceProperties (or defaults for a B200 when a plan
// is only inspected on a machine without a GPU).
struct Machine {
  int sm_count = 148;
  int smem_optin_bytes = 232448;  // 227 KB
  int tmem_cols = 512;
  int l2_bytes = 126 * 1024 * 1024;
};

// Integer tile of the halo/tcgen05 kernel.  Names follow the paper's block sizes b_x.
//
// The contraction over (c, r, s) is cut into "units": one unit = 16 channels x one (r,s) tap, i.e.
// one K=16 step of the tensor core.  Units are ordered channel-chunk major, tap minor.  Two
// shared-memory rings feed them:
//   * the Image ring: one stage = the halo block b_b x b_c x (sw(b_w-1)+R) x (sh(b_h-1)+S),
//     shared by all R*S taps of its b_c channels;
//   * the Filter ring: one stage = `uf` consecutive units of the packed Filter (b_k x 16 each).
struct HaloTile {
  int bb = 0;      // b_b: images per tile (32 or 64; one swizzled shared-memory row)
  int bw = 0;      // b_w: output pixels along w; the N extent of one MMA is bb*bw
  int bh = 0;      // b_h: output pixels along h, one MMA per row
  int bk = 128;    // b_k: output channels per tile = MMA M
  int bc = 0;      // b_c: channels per Image stage (16, 32 or 64)
  int halo_w = 0, halo_h = 0;
  int i_stages = 0;   // Image ring depth
  int f_stages = 0;   // Filter ring depth
  int uf = 0;         // units per Filter stage
  int acc_bufs = 1;   // TMEM accumulator buffers (2 when two fit in 512 columns)
  int split = 1;      // 2 or 4: the CTAs of a cluster share each tile, an equal share of the channels each
  int tmem_cols = 0;
  int c16 = 0;        // 16-channel chunks: ceil(C/16)
  int cchunks = 0;    // Image stages per tile: ceil(C/bc)
  int tiles_k = 0, tiles_b = 0, tiles_w = 0, tiles_h = 0;
  long long tiles = 0;
  int grid = 0;
  uint32_t img_stage_bytes = 0, filt_stage_bytes = 0;
  long long packed_filter_bytes = 0;  // scratch: tiles_k * c16 * R*S blocks of 4 KB
  int smem_bytes = 0;
  double est_cycles = 0;   // cost-model estimate for the whole problem, SM cycles
  double model_cycles = 0; // the same before the HBM floor is applied
  double tile_cycles = 0;  // cost-model estimate for one tile on one SM
  double words_smem = 0;   // words staged into shared memory over the whole problem + |Out|
};

// Tile of the small-C ("stem") kernel: 128 MMA rows = bhm stacked output rows x kpad out-channels,
// bw pixels, 64 images; the whole (shifted, zero-padded) Filter stays in shared memory.
struct StemTile {
  int bw = 0, kpad = 0, bhm = 0, kw = 0, khalves = 0, halo_w = 0;
  int i_stages = 2, tmem_cols = 0;
  int tiles_k = 0, tiles_w = 0, tiles_h = 0, tiles_b = 0;
  long long tiles = 0;
  int grid = 0;
  uint32_t img_stage_bytes = 0, filt_bytes = 0;
  long long packed_filter_bytes = 0;
  int smem_bytes = 0;
  double words_smem = 0;
};

// Integer tile of the direct-Filter kernel.  As HaloTile, plus kt (b_k = 128*kt) and the Filter
// stage shape; the Filter needs no scratch.
struct DirectTile {
  int bb = 0, bw = 0, bh = 0, bc = 0, kt = 1;
  int halo_w = 0, halo_h = 0;
  int tg = 1, fgroups = 1;
  int i_stages = 0, f_stages = 0;
  int acc_bufs = 1, tmem_cols = 0;
  int cchunks = 0;
  int tiles_k = 0, tiles_b = 0, tiles_w = 0, tiles_h = 0;
  long long tiles = 0;
  int grid = 0;
  uint32_t img_stage_bytes = 0, filt_stage_bytes = 0;
  int smem_bytes = 0;
  double tile_cycles = 0;   // cost-model estimate for the main loop of one tile
  double cta_cycles = 0;    // lifetime of one CTA: what a call that runs alone takes
  double sm_cycles = 0;     // grid * cta_cycles: SM time of one call
  double est_cycles = 0;    // period of a stream of such calls (calls overlap on the SMs)
  double words_smem = 0;
};

// True when the direct-Filter kernel can run this shape: B % 8 == 0 and C % 8 == 0 (16-byte TMA
// strides of both tensor maps).
bool direct_supported(const Dims& d, const char** why);
// Enumerate legal tiles and keep the one with the least estimated SM time per call.  `force` may
// carry "bb,bw,bh,kt,bc,tg,i_stages,f_stages,grid" (0 = free) from CCONV_FORCE_DIRECT.
bool choose_direct_tile(const Dims& d, const Machine& m, const int force[9], DirectTile* out);

void theorem1_terms(const Dims& d, double M, double t[5]);

// Theorem 2 (Appendix A; strides 1): which expression of Theorem 1 is attainable.  Returns the leaf
// of the decision tree as the digits of its name (1, 21, 221, 2221, 2222) and stores the attainable
// lower bound in words.
int theorem2_leaf(const Dims& d, double M, double* alb_words);

// Section 8, "Parallel Algorithm": p processors behind one shared memory of M words, the output cut
// into a[0] x a[1] x a[2] x a[3] = aB x aK x aH x aW equal blocks, one per processor.  The bound is p
// times Theorem 1 on a block, i.e. the Image term times aK and the Filter term times aB*aH*aW.
void parallel_terms(const Dims& d, double M, const int a[4], double t[5]);
// The cut with aX <= X and product <= p that uses the most processors, then has the smallest
// bound, then the least replicated traffic (terms 2 + 3), then is lexicographically smallest.
// Returns false for p < 1 or p > 65536.
bool choose_partition(const Dims& d, double M, int p, int a_out[4], double* bound_out);

// Dense primal simplex on the LP of Section 5 in log_M space.  tiles[9] in the order
// b_b,b_c,b_k,b_w,b_h,b_r',b_r'',b_s',b_s''.  Returns false on non-positive arguments.
bool tiling_lp(const Dims& d, double M, bool pooling, double tiles[9], double* G, double* words);

// True when the halo/tcgen05 kernel can run this shape at all.
bool halo_supported(const Dims& d, const char** why);

// Enumerate legal tiles and keep the one with the least estimated time (ties: fewer staged words).
// `force` may carry "bw,bh,bc,stages,bb,split" (0 = free) from the CCONV_FORCE_TILE environment
// variable; split: 1 = never split the channels over a CTA pair, 2 = always.
bool choose_halo_tile(const Dims& d, const Machine& m, const int force[6], HaloTile* out);

// Wave quantisation: when the tiles of the best tiling fill the last wave of the persistent grid
// only partly, the last output rows may be cheaper as a second launch with a smaller tile whose
// CTAs fill the SMs that the first launch leaves idle.  Returns true and sets *main_tiles_h (rows of
// tiles the main tiling keeps, counted from h = 0) and *tail (tiling of the remaining output rows,
// planned as a problem with H = the remaining rows) when the model predicts a gain; `main` is the
// whole-problem tile from choose_halo_tile.
bool choose_halo_tail(const Dims& d, const Machine& m, const HaloTile& main, int* main_tiles_h,
                      HaloTile* tail);

// The stem kernel needs B % 8 == 0 and the resident Filter plus two Image windows to fit in shared
// memory.
bool choose_stem_tile(const Dims& d, const Machine& m, StemTile* out, int force_bw = 0);

}  // namespace cconv
