// Host-side helpers shared by the entry points (see host_setup.h).
#include "host_setup.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cstdlib>
#include <map>
#include <mutex>

#include "../../include/cconv.h"

namespace cconv {

namespace {

thread_local std::string g_last_cuda_error;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver is reached through the runtime so that the library loads on machines without one.
EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) !=
            cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

int env_int(const char* name, int dflt) {
  const char* v = std::getenv(name);
  return (v && *v) ? std::atoi(v) : dflt;
}

uint64_t make_smem_desc(uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout_type) {
  // tcgen05 shared-memory matrix descriptor: start address [0,14) (set on the device),
  // leading byte offset [16,30), stride byte offset [32,46), version=1 [46,48),
  // base offset [49,52)=0, layout type [61,64).  Offsets are stored >> 4.
  uint64_t d = 0;
  d |= uint64_t((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= uint64_t((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= uint64_t(1) << 46;
  d |= uint64_t(layout_type & 7u) << 61;
  return d;
}

}  // namespace

void build_halo_params(const Dims& d, const HaloTile& t, HaloKernelParams* out) {
  HaloKernelParams& p = *out;
  p.K = d.K; p.H = d.H; p.W = d.W; p.B = d.B; p.C = d.C;
  p.R = d.R; p.S = d.S; p.sw = d.sw; p.sh = d.sh;
  p.bb = t.bb; p.bw = t.bw; p.bh = t.bh; p.bc = t.bc;
  p.halo_w = t.halo_w;
  p.c16 = t.c16;
  p.units = t.c16 * d.R * d.S;
  p.units_per_img = (t.bc / 16) * d.R * d.S;
  p.uf = t.uf;
  p.i_stages = t.i_stages; p.f_stages = t.f_stages;
  p.tiles_k = t.tiles_k; p.tiles_b = t.tiles_b; p.tiles_w = t.tiles_w; p.tiles_h = t.tiles_h;
  p.total_tiles = int(t.tiles);
  p.split = t.split;
  p.units_cta = p.units / t.split;
  p.cchunks_cta = t.cchunks / t.split;
  p.h0 = 0;
  p.tail = 0;
  p.image_wait = 0;
  p.n_mma = t.bb * t.bw;
  p.acc_cols = p.n_mma * t.bh;
  p.acc_bufs = t.acc_bufs;
  p.tmem_cols = t.tmem_cols;
  p.img_stage_bytes = t.img_stage_bytes;
  p.filt_stage_bytes = t.filt_stage_bytes;
  p.slab_bytes = uint32_t(t.bc) * t.bb * 2;
  p.b_kstep_bytes = 16u * t.bb * 2;
  // instruction descriptor: D=f32 [4,6)=1, A=bf16 [7,10)=1, B=bf16 [10,13)=1, A K-major [15]=0,
  // B MN-major [16]=1, N>>3 [17,23), M>>4 [24,29)
  p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) |
            (uint32_t(p.n_mma >> 3) << 17) | (uint32_t(128 >> 4) << 24);
  // A = one packed Filter block [128 rows][16 channels], K-major, no swizzle (layout type 0):
  // 8x8 core matrices of 128 B; LBO = 128 B between the two channel halves, SBO = 256 B between
  // groups of 8 rows.
  p.a_desc = make_smem_desc(128, 256, 0);
  // B = Image halo view [channels][n = (w, b)], MN-major; row = bb*2 bytes = the swizzle span
  // (layout type 2 = 128B swizzle, 4 = 64B).  SBO: from one group of 8 channels to the next;
  // LBO: from one pixel's bb images to the next pixel along w, sw halo pixels further.
  // (layout type 6 = 32B swizzle for blocks of 16 images, 0 = none for blocks of 8: 16-byte rows)
  const uint32_t b_row = uint32_t(t.bb) * 2;
  const uint32_t b_layout = b_row == 128 ? 2u : b_row == 64 ? 4u : b_row == 32 ? 6u : 0u;
  // (Without a swizzle the two offsets change roles: the stride field then steps along n, from
  // pixel to pixel, and the leading field from one group of 8 channels to the next.)
  p.b_desc = b_layout != 0u ? make_smem_desc(uint32_t(d.sw) * p.slab_bytes, 8 * b_row, b_layout)
                            : make_smem_desc(8 * b_row, uint32_t(d.sw) * p.slab_bytes, 0u);
  p.wait_limit_ns = uint64_t(env_int("CCONV_WAIT_LIMIT_MS", 1000)) * 1000000ull;
  p.trace = nullptr;
}

int encode_image_map(const ImageView& v, const HaloTile& t, const void* image, CUtensorMap* tm) {
  const Dims& d = v.dk;
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) {
    set_last_cuda_error("cuTensorMapEncodeTiled is not available from this driver");
    return CCONV_ECUDA;
  }
  // Image viewed as (b, c, x, y): b fastest; x is the w-direction subscript (slowest in memory).
  // A box lands in shared memory as [y][x][c][b]: one slab of b_c x b_b per halo pixel.
  const cuuint64_t dims[4] = {cuuint64_t(d.B), cuuint64_t(d.C), cuuint64_t(d.Wi()),
                              cuuint64_t(d.Hi())};
  const cuuint64_t strides[3] = {cuuint64_t(v.stride_c) * 2, cuuint64_t(v.stride_w) * 2,
                                 cuuint64_t(v.stride_h) * 2};
  const cuuint32_t box[4] = {cuuint32_t(t.bb), cuuint32_t(t.bc), cuuint32_t(t.halo_w),
                             cuuint32_t(t.halo_h)};
  const cuuint32_t es[4] = {1, 1, 1, 1};
  const CUtensorMapSwizzle sw = t.bb == 64   ? CU_TENSOR_MAP_SWIZZLE_128B
                                : t.bb == 32 ? CU_TENSOR_MAP_SWIZZLE_64B
                                : t.bb == 16 ? CU_TENSOR_MAP_SWIZZLE_32B
                                             : CU_TENSOR_MAP_SWIZZLE_NONE;
  CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(image),
                   dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_last_cuda_error("cuTensorMapEncodeTiled(Image) failed with CUresult " +
                        std::to_string(int(r)));
    return CCONV_ECUDA;
  }
  return CCONV_OK;
}

void build_direct_params(const Dims& d, const DirectTile& t, DirectKernelParams* out) {
  DirectKernelParams& p = *out;
  p.K = d.K; p.H = d.H; p.W = d.W; p.B = d.B; p.C = d.C;
  p.R = d.R; p.S = d.S; p.sw = d.sw; p.sh = d.sh;
  p.bb = t.bb; p.bw = t.bw; p.bh = t.bh; p.bc = t.bc; p.kt = t.kt;
  p.halo_w = t.halo_w; p.halo_h = t.halo_h;
  p.cchunks = t.cchunks;
  p.tg = t.tg; p.fgroups = t.fgroups;
  p.i_stages = t.i_stages; p.f_stages = t.f_stages;
  p.tiles_k = t.tiles_k; p.tiles_b = t.tiles_b; p.tiles_w = t.tiles_w; p.tiles_h = t.tiles_h;
  p.total_tiles = int(t.tiles);
  p.n_mma = t.bb * t.bw;
  p.acc_cols = p.n_mma * t.bh * t.kt;
  p.acc_bufs = t.acc_bufs;
  p.tmem_cols = t.tmem_cols;
  p.wait_prev = 0;
  p.img_stage_bytes = t.img_stage_bytes;
  p.filt_stage_bytes = t.filt_stage_bytes;
  p.filt_ktile_bytes = 128u * uint32_t(t.bc) * 2u;
  p.filt_tap_bytes = uint32_t(t.kt) * p.filt_ktile_bytes;
  p.slab_bytes = uint32_t(t.bc) * t.bb * 2;
  p.b_kstep_bytes = 16u * t.bb * 2;
  // instruction descriptor: D=f32, A=B=bf16, A K-major [15]=0, B MN-major [16]=1, N>>3, M=128>>4
  // Output rows whose pixels continue at the same pitch in the stage (no halo columns between
  // the rows: R = S = 1 at stride 1) form one operand of n_mma*bh columns: one MMA instead of bh
  // reads the Filter block from shared memory once instead of bh times.
  const bool rows_merge = t.bh > 1 && d.sh * t.halo_w == t.bw * d.sw && p.n_mma * t.bh <= 256 &&
                          (p.n_mma * t.bh) % 16 == 0 && env_int("CCONV_DIRECT_MERGE_ROWS", 1) != 0;
  p.mma_rows = rows_merge ? 1 : t.bh;
  p.mma_n = rows_merge ? p.n_mma * t.bh : p.n_mma;
  p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) |
            (uint32_t(p.mma_n >> 3) << 17) | (uint32_t(128 >> 4) << 24);
  // A = Filter rows [128 out-channels][bc channels], K-major, one swizzle span per row (bc*2 = 128,
  // 64 or 32 bytes: layout type 2, 4, 6); SBO = 8 rows; the leading offset is not used by swizzled
  // K-major operands.  A 16-channel step advances the start address by 32 bytes inside the row.
  const uint32_t a_row = uint32_t(t.bc) * 2;
  const uint32_t a_layout = a_row == 128 ? 2u : a_row == 64 ? 4u : 6u;
  p.a_desc = make_smem_desc(16, 8 * a_row, a_layout);
  // B = Image halo view, as in the halo kernel: MN-major rows of bb*2 bytes (128- or 64-byte swizzle);
  // SBO from one group of 8 channels to the next, LBO from one pixel to the next along w.
  const uint32_t b_row = uint32_t(t.bb) * 2;
  const uint32_t b_layout = b_row == 128 ? 2u : 4u;
  p.b_desc = make_smem_desc(uint32_t(d.sw) * p.slab_bytes, 8 * b_row, b_layout);
  p.wait_limit_ns = uint64_t(env_int("CCONV_WAIT_LIMIT_MS", 1000)) * 1000000ull;
  p.diag_mode = env_int("CCONV_DIAG_MODE", 0);
  p.out_tma = 0;  // set per call when the Out tensor map could be built
  p.skip_filter_stage = -1;
  p.trace = nullptr;
}

int encode_direct_image_map(const ImageView& v, const DirectTile& t, const void* image, CUtensorMap* tm) {
  HaloTile h;
  h.bb = t.bb; h.bc = t.bc; h.halo_w = t.halo_w; h.halo_h = t.halo_h;
  return encode_image_map(v, h, image, tm);
}

int encode_direct_filter_map(const Dims& d, const DirectTile& t, const void* filter, CUtensorMap* tm) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) {
    set_last_cuda_error("cuTensorMapEncodeTiled is not available from this driver");
    return CCONV_ECUDA;
  }
  // Filter[k][r][s][c] viewed as (c, k, tap = r*S + s): a box lands as [tap][k][bc channels].
  // Rows past K and channels past C are zero filled.
  const cuuint64_t dims[3] = {cuuint64_t(d.C), cuuint64_t(d.K), cuuint64_t(d.R) * d.S};
  const cuuint64_t strides[2] = {cuuint64_t(d.R) * d.S * d.C * 2, cuuint64_t(d.C) * 2};
  const cuuint32_t box[3] = {cuuint32_t(t.bc), cuuint32_t(128 * t.kt), cuuint32_t(t.tg)};
  const cuuint32_t es[3] = {1, 1, 1};
  const CUtensorMapSwizzle sw = t.bc == 64   ? CU_TENSOR_MAP_SWIZZLE_128B
                                : t.bc == 32 ? CU_TENSOR_MAP_SWIZZLE_64B
                                             : CU_TENSOR_MAP_SWIZZLE_32B;
  CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(filter), dims, strides,
                   box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_last_cuda_error("cuTensorMapEncodeTiled(Filter) failed with CUresult " + std::to_string(int(r)));
    return CCONV_ECUDA;
  }
  return CCONV_OK;
}

int encode_direct_out_map(const Dims& d, const DirectTile& t, bool out_f32, void* out, CUtensorMap* tm,
                          int* merged_wb) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) {
    set_last_cuda_error("cuTensorMapEncodeTiled is not available from this driver");
    return CCONV_ECUDA;
  }
  // A piece is 128 bytes of one accumulator row (64 bf16 / 32 fp32 columns, images fastest) and
  // must be 128 contiguous bytes of Out, so that the box's inner extent is the swizzle span:
  // one pixel's 64 images (bf16) or half of them (fp32), a 32-image block in fp32, or -- bf16 with
  // b_b = B = 32 -- two neighbouring pixels, addressed through the merged subscript w*B + b.
  const cuuint64_t es = out_f32 ? 4 : 2;
  const bool merged = !out_f32 && t.bb == 32 && d.B == 32;
  if (!merged && uint64_t(t.bb) * es < 128) return CCONV_EUNSUPPORTED;
  *merged_wb = merged ? 1 : 0;
  const cuuint64_t row = cuuint64_t(d.W) * d.B * es;
  const cuuint64_t dims[4] = {merged ? cuuint64_t(d.W) * d.B : cuuint64_t(d.B),
                              merged ? cuuint64_t(1) : cuuint64_t(d.W), cuuint64_t(d.H), cuuint64_t(d.K)};
  const cuuint64_t strides[3] = {merged ? row : cuuint64_t(d.B) * es, row, cuuint64_t(d.H) * row};
  const cuuint32_t box[4] = {cuuint32_t(128 / es), 1, 1, 32};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = enc(tm, out_f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4,
                   out, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_last_cuda_error("cuTensorMapEncodeTiled(Out) failed with CUresult " + std::to_string(int(r)));
    return CCONV_ECUDA;
  }
  return CCONV_OK;
}

void build_stem_params(const Dims& d, const StemTile& t, StemKernelParams* out) {
  StemKernelParams& p = *out;
  p.K = d.K; p.H = d.H; p.W = d.W; p.B = d.B; p.C = d.C;
  p.R = d.R; p.S = d.S; p.sw = d.sw; p.sh = d.sh;
  p.bw = t.bw; p.kpad = t.kpad; p.bhm = t.bhm; p.kw = t.kw; p.khalves = t.khalves;
  p.units = d.R * t.khalves;
  p.halo_w = t.halo_w;
  p.tiles_k = t.tiles_k; p.tiles_w = t.tiles_w; p.tiles_h = t.tiles_h; p.tiles_b = t.tiles_b;
  p.total_tiles = int(t.tiles);
  p.i_stages = t.i_stages;
  p.acc_cols = 64 * t.bw;
  p.tmem_cols = t.tmem_cols;
  p.acc_bufs = std::min(8, t.tmem_cols / p.acc_cols);
  p.img_stage_bytes = t.img_stage_bytes;
  p.filt_bytes = t.filt_bytes;
  // instruction descriptor: D=f32, A=B=bf16, A K-major [15]=0, B MN-major [16]=1, N = 64*bw, M = 128
  p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) |
            (uint32_t((64 * t.bw) >> 3) << 17) | (uint32_t(128 >> 4) << 24);
  // A = Filter block [128 rows][16], K-major, no swizzle: LBO = 128 B, SBO = 256 B.
  p.a_desc = make_smem_desc(128, 256, 0);
  // B = Image window [16 rows][bw pixels x 64 images], MN-major, 128-byte swizzle (layout type 2):
  // SBO = 1024 B from one group of 8 rows to the next; LBO = from one pixel's 64 images to the next
  // pixel's, sw Image columns (of kw rows x 128 B) further.
  p.b_desc = make_smem_desc(uint32_t(d.sw) * uint32_t(t.kw) * 128u, 1024, 2);
  p.wait_limit_ns = uint64_t(env_int("CCONV_WAIT_LIMIT_MS", 1000)) * 1000000ull;
  p.filter_ready = nullptr;
  p.ready_target = 0;
  p.wait_prev = 0;
  p.trace = nullptr;
}

int encode_stem_image_map(const Dims& d, const StemTile& t, const void* image, CUtensorMap* tm) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) {
    set_last_cuda_error("cuTensorMapEncodeTiled is not available from this driver");
    return CCONV_ECUDA;
  }
  // Image[x][y][c][b] viewed as (b, m, x) with m = y*C + c: for a fixed x the (y,c) rows are
  // contiguous, B images each.  A box lands as [x][m][64 images].
  const cuuint64_t dims[3] = {cuuint64_t(d.B), cuuint64_t(d.Hi()) * d.C, cuuint64_t(d.Wi())};
  const cuuint64_t strides[2] = {cuuint64_t(d.B) * 2, cuuint64_t(d.Hi()) * d.C * d.B * 2};
  const cuuint32_t box[3] = {64u, cuuint32_t(t.kw), cuuint32_t(t.halo_w)};
  const cuuint32_t es[3] = {1, 1, 1};
  CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(image), dims, strides,
                   box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_last_cuda_error("cuTensorMapEncodeTiled(Image, stem view) failed with CUresult " +
                        std::to_string(int(r)));
    return CCONV_ECUDA;
  }
  return CCONV_OK;
}


namespace {
constexpr int kMaxTracked = 160;
struct StreamCalls {
  CallSpans calls[kMaxTracked];
  int n = 0;
};
std::map<void*, StreamCalls> g_inflight;
std::mutex g_inflight_mu;
}  // namespace

CallSpans spans_of(const Dims& d, int out_dtype, const void* Image, const void* Filter, const void* Out) {
  CallSpans c;
  c.image.lo = static_cast<const char*>(Image);
  c.image.hi = c.image.lo + size_t(d.Wi()) * d.Hi() * d.C * d.B * 2;
  c.filter.lo = static_cast<const char*>(Filter);
  c.filter.hi = c.filter.lo + size_t(d.K) * d.R * d.S * d.C * 2;
  c.out.lo = static_cast<const char*>(Out);
  c.out.hi = c.out.lo + size_t(d.K) * d.H * d.W * d.B * (out_dtype == CCONV_OUT_F32 ? 4 : 2);
  return c;
}

bool note_call(void* stream, const CallSpans& c, Overlap how, int sm_count) {
  return note_call_hazards(stream, c, how, sm_count) != 0;
}

int note_call_hazards(void* stream, const CallSpans& c, Overlap how, int sm_count) {
  std::lock_guard<std::mutex> lk(g_inflight_mu);
  StreamCalls& sc = g_inflight[stream];
  if (how == Overlap::kNone) {
    sc.n = 0;  // starts after, and is complete before, its neighbours
    return 0;
  }
  // forget the calls that must be complete by the time this one starts: walking back from the
  // latest call, everything behind more than sm_count SMs' worth of resident CTAs
  {
    double sms = 0, sms_by_threads = 0;
    int keep = 0;
    for (int i = sc.n - 1; i >= 0; --i) {
      ++keep;
      sms += sc.calls[i].sms;
      sms_by_threads += sc.calls[i].sms_by_threads;
      // no SM left on which an older call could still have a CTA
      if (sms >= double(sm_count) || sms_by_threads >= double(sm_count)) break;
    }
    if (keep < sc.n) {
      for (int i = 0; i < keep; ++i) sc.calls[i] = sc.calls[sc.n - keep + i];
      sc.n = keep;
    }
  }
  // (a full list counts as both kinds: a waiting call completes everything before it)
  int hazards = sc.n >= kMaxTracked ? (kHazardInputs | kHazardOut) : 0;
  for (int i = 0; i < sc.n && hazards != (kHazardInputs | kHazardOut); ++i) {
    const CallSpans& e = sc.calls[i];
    if (e.out.meets(c.image) || e.out.meets(c.filter)) hazards |= kHazardInputs;
    if (how == Overlap::kDeep &&
        (e.out.meets(c.out) || e.image.meets(c.out) || e.filter.meets(c.out)))
      hazards |= kHazardOut;
  }
  if (hazards || how == Overlap::kInputsEarly) sc.n = 0;
  sc.calls[sc.n++] = c;
  return hazards;
}

void note_ordinary_launch(void* stream) {
  std::lock_guard<std::mutex> lk(g_inflight_mu);
  auto it = g_inflight.find(stream);
  if (it != g_inflight.end()) it->second.n = 0;
}

void set_last_cuda_error(const std::string& msg) { g_last_cuda_error = msg; }
const char* last_cuda_error() { return g_last_cuda_error.c_str(); }

}  // namespace cconv
