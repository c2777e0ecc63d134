// C ABI of libcconv (declared in include/cconv.h): argument checking, plans, TMA descriptors,
// launches.  No compute happens on the host; there is no CPU fallback.
#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <string>
#include <tuple>

#include "../../include/cconv.h"
#include "host_setup.h"
#include "kernels.h"
#include "planner.h"

using namespace cconv;

namespace {

int cuda_fail(cudaError_t e, const char* what) {
  set_last_cuda_error(std::string(what) + ": " + cudaGetErrorString(e));
  return CCONV_ECUDA;
}
#define CCONV_CUDA(call)                                  \
  do {                                                    \
    cudaError_t e_ = (call);                              \
    if (e_ != cudaSuccess) return cuda_fail(e_, #call);   \
  } while (0)

int env_int(const char* name, int dflt) {
  const char* v = std::getenv(name);
  return (v && *v) ? std::atoi(v) : dflt;
}

// Out of the most recent tensor-core convolution launched through a plan, and its stream (see
// cconv_forward_planned).
// What a padded plan runs on (see cconv_plan): Image [Wi][Hi][C][B] -> [Wi][Hir][C][Bp], where image
// b' = band * B + b of the copy holds the rows of image b that output rows band*Hr .. band*Hr+Hr-1
// need (Hir = sh*(Hr-1)+S of them, starting at row band*Hr*sh); rows past Hi, bands past `bands`
// and the images that round Bp up to a multiple of 8 are zero.  bands == 1: batch padding alone.
struct BandGeom {
  long long Wi, Hi, Hir, C;  // Image extents of the caller's problem and rows of the banded copy
  int B, Bp, bands;
  int Hr, sh;                // output rows per band, stride along h
};

// (one thread per 16 bytes of the copy: 8 images of one (x, y, c))
// Launched behind the Filter-packing kernel of the same call with programmatic stream
// serialisation, so that the two (which share no data) run side by side; it ends with a dependency
// wait, so that "this kernel is complete" implies that the packing kernel is, which is what the
// convolution behind it relies on.  `wait_first`: the caller's Image may still be being written by
// the kernel in front (the host's overlap check), so nothing is read before that one is complete.
__global__ void __launch_bounds__(256) cconv_pad_bands_kernel(const unsigned short* __restrict__ src,
                                                              uint4* __restrict__ dst, BandGeom g,
                                                              int wait_first) {
  if (wait_first) asm volatile("griddepcontrol.wait;" ::: "memory");
  const int gpb = g.Bp / 8;
  const long long n = g.Wi * g.Hir * g.C * gpb;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
       i += (long long)gridDim.x * blockDim.x) {
    long long t = i / gpb;
    const int grp = int(i - t * gpb);
    const long long c = t % g.C;
    t /= g.C;
    const long long yr = t % g.Hir;
    const long long x = t / g.Hir;
    uint32_t e[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int bp = grp * 8 + j;
      const int band = bp / g.B, b = bp - band * g.B;
      const long long y = (long long)band * g.Hr * g.sh + yr;
      e[j] = (band < g.bands && y < g.Hi) ? uint32_t(src[((x * g.Hi + y) * g.C + c) * g.B + b]) : 0u;
    }
    dst[i] = make_uint4(e[0] | (e[1] << 16), e[2] | (e[3] << 16), e[4] | (e[5] << 16),
                        e[6] | (e[7] << 16));
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

// The way back: Out [K][H][W][B] of the caller from [K][Hr][W][Bp] of the banded run (T = bf16 bits
// or fp32); output row h is row h % Hr of band h / Hr.  One thread per 8 images of the banded Out:
// consecutive threads hold consecutive w, so that the stores of one band run along an output row.
template <typename T>
__global__ void __launch_bounds__(256) cconv_compact_bands_kernel(const T* __restrict__ src,
                                                                  T* __restrict__ dst, long long K,
                                                                  long long H, long long W,
                                                                  BandGeom g) {
  // launched with programmatic stream serialisation: resident early, working once the convolution
  // in front is complete
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int gpb = g.Bp / 8;
  const long long n = K * g.Hr * W * gpb;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
       i += (long long)gridDim.x * blockDim.x) {
    const int grp = int(i % gpb);
    long long t = i / gpb;
    const long long w = t % W;
    t /= W;
    const long long hr = t % g.Hr;
    const long long k = t / g.Hr;
    T v[8];
    const T* s8 = src + ((k * g.Hr + hr) * W + w) * g.Bp + grp * 8;
    if constexpr (sizeof(T) == 2) {
      *reinterpret_cast<uint4*>(v) = *reinterpret_cast<const uint4*>(s8);
    } else {
      *reinterpret_cast<uint4*>(v) = *reinterpret_cast<const uint4*>(s8);
      *reinterpret_cast<uint4*>(v + 4) = *reinterpret_cast<const uint4*>(s8 + 4);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int bp = grp * 8 + j;
      const int band = bp / g.B, b = bp - band * g.B;
      const long long h = (long long)band * g.Hr + hr;
      if (band < g.bands && h < H) dst[((k * H + h) * W + w) * g.B + b] = v[j];
    }
  }
}

// Eq. 1's "+=" on an Out that already holds values: Out <- Out + Conv, Conv in fp32 from the plan's
// fp32 twin, one rounding to Out's type
template <typename T>
__device__ __forceinline__ T add_round(T old, float conv);
template <>
__device__ __forceinline__ float add_round<float>(float old, float conv) { return old + conv; }
template <>
__device__ __forceinline__ __nv_bfloat16 add_round<__nv_bfloat16>(__nv_bfloat16 old, float conv) {
  return __float2bfloat16_rn(__bfloat162float(old) + conv);
}
template <typename T>
__global__ void __launch_bounds__(256) cconv_accumulate_kernel(T* __restrict__ out,
                                                               const float* __restrict__ conv,
                                                               long long n) {
  // four elements per thread and step (Out is 32-byte aligned, the fp32 array 256), the last n % 4
  // one by one
  const long long n4 = n >> 2;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n4;
       i += (long long)gridDim.x * blockDim.x) {
    const float4 c = reinterpret_cast<const float4*>(conv)[i];
    T* o = out + 4 * i;
    if constexpr (sizeof(T) == 4) {
      float4 v = *reinterpret_cast<float4*>(o);
      v.x += c.x; v.y += c.y; v.z += c.z; v.w += c.w;
      *reinterpret_cast<float4*>(o) = v;
    } else {
      uint2 raw = *reinterpret_cast<uint2*>(o);
      __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&raw.x);
      __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162*>(&raw.y);
      a = __floats2bfloat162_rn(__low2float(a) + c.x, __high2float(a) + c.y);
      b = __floats2bfloat162_rn(__low2float(b) + c.z, __high2float(b) + c.w);
      raw.x = *reinterpret_cast<uint32_t*>(&a);
      raw.y = *reinterpret_cast<uint32_t*>(&b);
      *reinterpret_cast<uint2*>(o) = raw;
    }
  }
  for (long long i = 4 * n4 + blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
       i += (long long)gridDim.x * blockDim.x)
    out[i] = add_round<T>(out[i], conv[i]);
}

unsigned grid_for(long long n) {
  const long long blocks = (n + 255) / 256;
  return unsigned(std::max<long long>(1, std::min<long long>(blocks, 148ll * 32)));
}

}  // namespace

struct cconv_plan {
  Dims d{};
  // What the tensor-core kernels run.  They need B % 8 == 0 (16-byte TMA strides, 16-byte pieces of
  // Out): for any other batch size they run `drun` = `d` with B rounded up to a multiple of 8 on
  // plan-owned zero-padded copies of Image and Out (`d_img_pad`, `d_out_pad`); a padding kernel in
  // front and a compaction kernel behind move the real images in and out.
  // Fewer than 8 images: instead of padding with up to 7 zero images, the output rows are cut into
  // `bands` bands of drun.H rows, and each band of each image becomes one image of `drun` (Eq. 1 has
  // no dependence between output rows; a band only needs S - sh more Image rows than it owns, which
  // the padding kernel copies twice).  One image then fills a block of 8 with real work.
  Dims drun{};
  bool padded = false;
  int bands = 1;
  void* d_img_pad = nullptr;
  void* d_out_pad = nullptr;
  // cconv_plan_reserve_accumulate: the same plan with fp32 Out and an fp32 array of Out's shape
  cconv_plan* acc_twin = nullptr;
  // AUTO plans that took the direct kernel (tiled for a stream of independent calls): the same
  // problem planned for the halo kernel, whose many small tiles finish one call sooner.  A call
  // that has to wait for the stream's earlier work cannot run beside it and takes this plan.
  cconv_plan* wait_twin = nullptr;
  float* d_acc = nullptr;
  ImageView view{};  // `drun`, or its unstrided equivalent for 1x1 filters with strides
  bool strided_image = false;     // the Image is a view with explicit strides (cconv_forward_strided)
  size_t image_span_bytes = 0;    // bytes from the Image's first to one past its last element
  int device = -1;
  int variant = CCONV_VARIANT_SIMT;
  int out_dtype = CCONV_OUT_BF16;
  Machine m{};
  double M_words = 0;
  double terms[5] = {0, 0, 0, 0, 0};
  double lp_tile[9] = {0};
  double lp_G = 0, lp_words = 0;
  HaloTile tile{};
  HaloKernelParams kp{};
  // Optional second launch of a call: the last output rows with a smaller tile, filling the SMs
  // that the last wave of the main launch leaves idle.
  bool has_tail = false;
  HaloTile tail{};
  HaloKernelParams kp_tail{};
  StemTile stile{};
  StemKernelParams skp{};
  DirectTile dtile{};
  DirectKernelParams dkp{};
  mutable int diag_skip_once = -1;  // diagnostics: Filter stage the first call leaves out
  int* d_status = nullptr;
  // Scratch: the packed Filter, rewritten by every forward call.  Two buffers, used alternately:
  // the packing kernel of call n+1 may run while the convolution of call n still reads its buffer.
  void* d_packed = nullptr;  // 2 x packed_bytes
  size_t packed_bytes = 0;
  mutable unsigned calls = 0;
  mutable unsigned stem_uses[2] = {0, 0};  // calls that used each packed-Filter buffer (stem kernel)
  unsigned long long* d_trace = nullptr;  // diagnostics: [grid][16] device time stamps
  int trace_rows = 0;
  // host-buffer entry point: device staging owned by the plan
  void* st_image = nullptr;
  void* st_filter = nullptr;
  void* st_out = nullptr;
  // cconv_forward_host_async: two sets of staging arrays, a copy stream per direction, and per set
  // the events "inputs copied", "kernels done", "Out copied back"
  bool pipe_ready = false;
  unsigned pipe_calls = 0;
  void* pp_image[2] = {nullptr, nullptr};
  void* pp_filter[2] = {nullptr, nullptr};
  void* pp_out[2] = {nullptr, nullptr};
  cudaStream_t pp_h2d = nullptr, pp_h2d_f = nullptr, pp_d2h = nullptr;
  cudaEvent_t ev_in_f[2] = {nullptr, nullptr};
  cudaEvent_t ev_in[2] = {nullptr, nullptr}, ev_run[2] = {nullptr, nullptr}, ev_out[2] = {nullptr, nullptr};
  // the tensor map is rebuilt only when the base pointer changes
  mutable std::mutex mu;
  mutable const void* tm_image_ptr = nullptr;
  mutable CUtensorMap tm_image{};
  mutable CUtensorMap tm_image_tail{};
  // direct kernel: tensor maps of the latest base pointers (callers rotate through a few buffers;
  // encoding a map costs more host time than the rest of a call)
  struct MapSlot {
    const void* ptr = nullptr;
    CUtensorMap tm{};
  };
  static constexpr int kMapSlots = 64;
  mutable MapSlot img_maps[kMapSlots];
  mutable MapSlot flt_maps[kMapSlots];
  mutable MapSlot out_maps[kMapSlots];
  bool direct_tma_store = false;  // single-tile CTAs store Out through the TMA engine
  int direct_tma_mode = 1;        // DirectKernelParams::out_tma of such calls
  static int map_slot(const void* p) {
    return int((reinterpret_cast<uintptr_t>(p) >> 8) * 0x9E3779B97F4A7C15ull >> 58);
  }
};

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

std::mutex g_cache_mu;
std::map<std::tuple<int, void*, int, int, int, int, int, int, int, int, int, int>, cconv_plan*> g_cache;
std::map<std::tuple<int, void*, int, int, int, int, int, int, int, int, int, int, long long, long long, long long>, cconv_plan*>
    g_cache_strided;

}  // namespace

// The tensor-core launches of one forward call (Image and Out already padded if need be).
// `pad` (padded plans): the caller's Image is copied into the plan's padded array between the
// packing kernel and the convolution, and `Image` is that array.
static cudaError_t launch_pad(const void* user_image, void* padded, const BandGeom& g, bool wait_first,
                              cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid_for(g.Wi * g.Hir * g.C * (g.Bp / 8)));
  cfg.blockDim = dim3(256);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, cconv_pad_bands_kernel, static_cast<const unsigned short*>(user_image),
                            static_cast<uint4*>(padded), g, wait_first ? 1 : 0);
}

static int launch_tensor_core(const cconv_plan* pl, const void* Image, const void* Filter, void* Out,
                              bool inputs_hazard, cudaStream_t stream,
                              const BandGeom* pad = nullptr, const void* user_image = nullptr) {
  CUtensorMap tmi, tmi_tail;
  void* packed = nullptr;
  {
    // the tensor map is rebuilt only when the Image pointer changes
    std::lock_guard<std::mutex> lk(pl->mu);
    if (pl->tm_image_ptr != Image) {
      int rc = pl->variant == CCONV_VARIANT_STEM
                   ? encode_stem_image_map(pl->drun, pl->stile, Image, &pl->tm_image)
                   : encode_image_map(pl->view, pl->tile, Image, &pl->tm_image);
      if (rc == CCONV_OK && pl->has_tail)
        rc = encode_image_map(pl->view, pl->tail, Image, &pl->tm_image_tail);
      if (rc != CCONV_OK) return rc;
      pl->tm_image_ptr = Image;
    }
    tmi = pl->tm_image;
    if (pl->has_tail) tmi_tail = pl->tm_image_tail;
    packed = static_cast<char*>(pl->d_packed) + (pl->calls++ & 1u) * pl->packed_bytes;
  }
  if (pl->variant == CCONV_VARIANT_STEM) {
    // The packing kernel and the convolution of a call run side by side (and beside the previous
    // call's last tiles); the packed Filter is handed over through a counter in plan-owned memory,
    // one per scratch buffer (see StemKernelParams::filter_ready).
    StemKernelParams skp = pl->skp;
    {
      std::lock_guard<std::mutex> lk(pl->mu);
      const unsigned buf = (pl->calls - 1u) & 1u;  // the buffer `packed` points to
      skp.filter_ready = reinterpret_cast<unsigned int*>(pl->d_status) + 16 + 16 * buf;
      skp.ready_target = ++pl->stem_uses[buf] * pack_filter_stem_blocks(skp);
    }
    skp.wait_prev = (inputs_hazard || pad) ? 1 : 0;
    cudaError_t es = launch_pack_filter_stem(Filter, packed, pl->d, skp, !inputs_hazard, stream);
    if (es != cudaSuccess) return cuda_fail(es, "launch_pack_filter_stem");
    if (pad) {
      es = launch_pad(user_image, pl->d_img_pad, *pad, inputs_hazard, stream);
      if (es != cudaSuccess) return cuda_fail(es, "cconv_pad_bands_kernel");
    }
    es = launch_stem(tmi, packed, Out, pl->out_dtype == CCONV_OUT_F32, skp, pl->stile.grid,
                     pl->stile.smem_bytes, pl->d_status, stream);
    return es == cudaSuccess ? CCONV_OK : cuda_fail(es, "launch_stem");
  }
  HaloKernelParams kp = pl->kp;
  // (a padded Image is written by the kernel right in front of the convolution)
  kp.image_wait = (inputs_hazard || pad) ? 1 : 0;
  // (a Filter that the call in front may still be writing is not read before that call is complete)
  cudaError_t e = launch_pack_filter(Filter, packed, pl->d, pl->tile.c16, pl->tile.tiles_k,
                                     /*overlap_prev=*/!inputs_hazard, stream);
  if (e != cudaSuccess) return cuda_fail(e, "launch_pack_filter");
  if (pad) {
    e = launch_pad(user_image, pl->d_img_pad, *pad, inputs_hazard, stream);
    if (e != cudaSuccess) return cuda_fail(e, "cconv_pad_bands_kernel");
  }
  e = launch_halo(tmi, packed, Out, pl->out_dtype == CCONV_OUT_F32, kp, pl->tile.grid,
                  pl->tile.smem_bytes, pl->d_status, stream);
  if (e == cudaSuccess && pl->has_tail)
    e = launch_halo(tmi_tail, packed, Out, pl->out_dtype == CCONV_OUT_F32, pl->kp_tail,
                    pl->tail.grid, pl->tail.smem_bytes, pl->d_status, stream);
  return e == cudaSuccess ? CCONV_OK : cuda_fail(e, "launch_halo");
}

extern "C" {

int cconv_version(void) { return 100; }

const char* cconv_strerror(int code) {
  switch (code) {
    case CCONV_OK: return "ok";
    case CCONV_EINVAL: return "invalid argument";
    case CCONV_EUNSUPPORTED: return "unsupported shape or device for the requested variant";
    case CCONV_ECUDA: return "CUDA error";
    case CCONV_EDEVICE_TIMEOUT: return "a bounded device-side wait expired";
    case CCONV_ENOMEM: return "out of memory";
    case CCONV_ETOOLARGE:
      return "the repacked Filter does not fit the fixed scratch array of cconv_forward_noalloc";
    default: return "unknown error";
  }
}

const char* cconv_last_cuda_error(void) { return last_cuda_error(); }

int cconv_lower_bound(int B, int C, int K, int W, int H, int R, int S, int sw, int sh,
                      double M_words, double terms_out[5]) {
  const Dims d{B, C, K, W, H, R, S, sw, sh};
  if (!d.positive() || !(M_words > 0) || !terms_out) return CCONV_EINVAL;
  theorem1_terms(d, M_words, terms_out);
  return CCONV_OK;
}

int cconv_theorem2_case(int B, int C, int K, int W, int H, int R, int S, double M_words,
                        int* leaf_out, double* alb_words_out) {
  const Dims d{B, C, K, W, H, R, S, 1, 1};
  if (!d.positive() || !(M_words > 0) || !leaf_out) return CCONV_EINVAL;
  *leaf_out = theorem2_leaf(d, M_words, alb_words_out);
  return CCONV_OK;
}

int cconv_parallel_lower_bound(int B, int C, int K, int W, int H, int R, int S, int sw, int sh,
                               double M_words, int aB, int aK, int aH, int aW, double terms_out[5]) {
  const Dims d{B, C, K, W, H, R, S, sw, sh};
  if (!d.positive() || !(M_words > 0) || !terms_out) return CCONV_EINVAL;
  if (aB < 1 || aK < 1 || aH < 1 || aW < 1 || aB > B || aK > K || aH > H || aW > W) return CCONV_EINVAL;
  const int a[4] = {aB, aK, aH, aW};
  parallel_terms(d, M_words, a, terms_out);
  return CCONV_OK;
}

int cconv_parallel_partition(int B, int C, int K, int W, int H, int R, int S, int sw, int sh,
                             double M_words, int p, int a_out[4], double* bound_out) {
  const Dims d{B, C, K, W, H, R, S, sw, sh};
  if (!d.positive() || !(M_words > 0) || !a_out) return CCONV_EINVAL;
  return choose_partition(d, M_words, p, a_out, bound_out) ? CCONV_OK : CCONV_EINVAL;
}

int cconv_tiling_lp(int B, int C, int K, int W, int H, int R, int S, int sw, int sh,
                    double M_words, int pooling, double tiles_out[9], double* G_out,
                    double* words_out) {
  const Dims d{B, C, K, W, H, R, S, sw, sh};
  if (!d.positive() || !(M_words > 1.0) || !tiles_out || !G_out || !words_out) return CCONV_EINVAL;
  return tiling_lp(d, M_words, pooling != 0, tiles_out, G_out, words_out) ? CCONV_OK : CCONV_EINVAL;
}

// `image_strides` (may be null): element strides of Image's subscripts (x, y, c, b) with b contiguous;
// the tensor-core kernels then read the Image through a strided tensor map (no padded copies).
static int plan_create_impl(cconv_plan** plan_out, int B, int C, int K, int W, int H, int R, int S,
                            int sw, int sh, int device, double M_words, int variant, int out_dtype,
                            const long long* image_strides) {
  if (!plan_out) return CCONV_EINVAL;
  *plan_out = nullptr;
  const Dims d{B, C, K, W, H, R, S, sw, sh};
  if (!d.positive()) return CCONV_EINVAL;
  if (variant < CCONV_VARIANT_AUTO || variant > CCONV_VARIANT_DIRECT) return CCONV_EINVAL;
  if (out_dtype != CCONV_OUT_BF16 && out_dtype != CCONV_OUT_F32) return CCONV_EINVAL;
  // element counts must fit the kernels' index arithmetic
  const double lim = 9.0e18;
  if (double(d.Wi()) * d.Hi() * C * B > lim || double(K) * H * W * B > lim ||
      double(K) * R * S * C > lim)
    return CCONV_EINVAL;
  cconv_plan* pl = new (std::nothrow) cconv_plan();
  if (!pl) return CCONV_ENOMEM;
  pl->d = d;
  pl->drun = d;
  if (d.B < 8) {
    int want = env_int("CCONV_BANDS", 0);
    if (want < 1) want = 8 / d.B;
    want = std::max(1, std::min(want, d.H));
    pl->drun.H = (d.H + want - 1) / want;
    pl->bands = (d.H + pl->drun.H - 1) / pl->drun.H;  // no empty band
  }
  pl->drun.B = (d.B * pl->bands + 7) / 8 * 8;
  pl->padded = pl->drun.B != d.B || pl->bands > 1;
  pl->view = image_view(pl->drun);
  pl->image_span_bytes = size_t(d.Wi()) * d.Hi() * d.C * d.B * 2;
  if (image_strides) {
    if (pl->padded) {
      delete pl;
      return CCONV_EUNSUPPORTED;
    }
    // (a strided 1x1 filter is already planned on a subsampled view: compose the two)
    pl->view.stride_w = image_strides[0] * (pl->view.dk.sw != d.sw ? d.sw : 1);
    pl->view.stride_h = image_strides[1] * (pl->view.dk.sh != d.sh ? d.sh : 1);
    pl->view.stride_c = image_strides[2];
    pl->strided_image = true;
    pl->image_span_bytes = size_t((d.Wi() - 1) * image_strides[0] + (d.Hi() - 1) * image_strides[1] +
                                  (d.C - 1) * image_strides[2] + d.B) * 2;
  }
  const Dims& dk = pl->view.dk;
  pl->device = device;
  pl->out_dtype = out_dtype;
  if (device >= 0) {
    // device < 0: a plan for a nominal B200, for inspection only (no CUDA call is made)
    cudaDeviceProp prop;
    cudaError_t e = cudaGetDeviceProperties(&prop, device);
    if (e != cudaSuccess) {
      delete pl;
      return cuda_fail(e, "cudaGetDeviceProperties");
    }
    pl->m.sm_count = prop.multiProcessorCount;
    pl->m.smem_optin_bytes = int(prop.sharedMemPerBlockOptin);
    pl->m.l2_bytes = prop.l2CacheSize;
    if (prop.major != 10 && variant >= CCONV_VARIANT_HALO) {
      delete pl;
      return CCONV_EUNSUPPORTED;
    }
  }
  pl->M_words = M_words > 0 ? M_words : pl->m.smem_optin_bytes / 2.0;
  theorem1_terms(d, pl->M_words, pl->terms);
  if (pl->M_words > 1.0) tiling_lp(d, pl->M_words, false, pl->lp_tile, &pl->lp_G, &pl->lp_words);

  int force[6] = {0, 0, 0, 0, 0, 0};
  if (const char* f = std::getenv("CCONV_FORCE_TILE"))
    std::sscanf(f, "%d,%d,%d,%d,%d,%d", &force[0], &force[1], &force[2], &force[3], &force[4],
                &force[5]);
  const int env_variant = env_int("CCONV_VARIANT", 0);
  if (variant == CCONV_VARIANT_AUTO && env_variant >= 1 && env_variant <= 4) variant = env_variant;
  int dforce[9] = {0, 0, 0, 0, 0, 0, 0, 0, 0};
  if (const char* f = std::getenv("CCONV_FORCE_DIRECT"))
    std::sscanf(f, "%d,%d,%d,%d,%d,%d,%d,%d,%d", &dforce[0], &dforce[1], &dforce[2], &dforce[3],
                &dforce[4], &dforce[5], &dforce[6], &dforce[7], &dforce[8]);

  bool want_wait_twin = false;
  const bool halo_ok = halo_supported(dk, nullptr) && choose_halo_tile(dk, pl->m, force, &pl->tile);
  // (the stem kernel reads the Image through a map of its own that needs the dense layout)
  const bool stem_ok = !image_strides &&
                       choose_stem_tile(pl->drun, pl->m, &pl->stile, env_int("CCONV_STEM_BW", 0));
  // the direct-Filter kernel runs on the caller's arrays only (no padded copies)
  const bool direct_ok = !pl->padded && direct_supported(dk, nullptr) &&
                         choose_direct_tile(dk, pl->m, dforce, &pl->dtile);
  if ((variant == CCONV_VARIANT_HALO && !halo_ok) || (variant == CCONV_VARIANT_STEM && !stem_ok) ||
      (variant == CCONV_VARIANT_DIRECT && !direct_ok)) {
    delete pl;
    return CCONV_EUNSUPPORTED;
  }
  if (variant == CCONV_VARIANT_AUTO) {
    // Fewer than 8 channels: a 16-channel K step of the halo kernel is mostly zero padding, so
    // the kernel that folds (s, c) into the contraction wins where it applies.
    if (stem_ok && d.C < 8) variant = CCONV_VARIANT_STEM;
    else variant = halo_ok ? CCONV_VARIANT_HALO : CCONV_VARIANT_SIMT;
    // Problems whose tiles fit the SMs as one wave: the direct-Filter kernel (one launch, large
    // tiles on few SMs, calls side by side) has about twice the throughput of the halo kernel in a
    // stream of calls (measured on 16 layer shapes; it loses on problems of several waves).  A
    // single call then takes longer (one CTA lifetime): CCONV_OBJECTIVE=latency keeps the halo
    // kernel's many small tiles.
    const char* objective = std::getenv("CCONV_OBJECTIVE");
    const bool want_latency = objective && std::strcmp(objective, "latency") == 0;
    if (variant == CCONV_VARIANT_HALO && direct_ok && !want_latency &&
        pl->dtile.tiles <= pl->m.sm_count && d.macs() >= 4.0e6) {
      variant = CCONV_VARIANT_DIRECT;
      want_wait_twin = device >= 0 && env_int("CCONV_WAIT_TWIN", 1) != 0;
    }
    // A padded batch costs two more kernels (about 15 us per call in all, measured) and two scratch
    // arrays: worth it unless the problem is tiny (the CUDA-core kernel needs 8 us for 0.5 M
    // multiply-adds, 25-50 us for 7-15 M), and only within 4 GiB of scratch.
    if (pl->padded && variant != CCONV_VARIANT_SIMT) {
      const double scratch = 2.0 * pl->drun.Wi() * pl->drun.Hi() * d.C * pl->drun.B +
                             double(d.K) * pl->drun.H * d.W * pl->drun.B * (out_dtype == CCONV_OUT_F32 ? 4 : 2);
      if (d.macs() < 4.0e6 || scratch > 4.0 * 1024 * 1024 * 1024) variant = CCONV_VARIANT_SIMT;
    }
  }
  if (image_strides && variant != CCONV_VARIANT_HALO && variant != CCONV_VARIANT_DIRECT) {
    delete pl;
    return CCONV_EUNSUPPORTED;  // the caller falls back to the CUDA-core kernel for any strides
  }
  pl->variant = variant;
  if (variant == CCONV_VARIANT_HALO) {
    const bool forced = force[0] || force[1] || force[2] || force[3] || force[4] || force[5];
    int keep = 0;
    bool tail_ok = !forced && !env_int("CCONV_NO_TAIL", 0) &&
                   choose_halo_tail(dk, pl->m, pl->tile, &keep, &pl->tail);
    if (const char* f = std::getenv("CCONV_FORCE_TAIL")) {
      // diagnostics: "rows of tiles kept,bw,bh,bc,stages,bb" for the tail
      int tf[6] = {0, 0, 0, 0, 0, 1};
      tail_ok = false;
      if (std::sscanf(f, "%d,%d,%d,%d,%d,%d", &keep, &tf[0], &tf[1], &tf[2], &tf[3], &tf[4]) >= 1 &&
          keep >= 1 && keep < pl->tile.tiles_h) {
        Dims dr = dk;
        dr.H = dk.H - keep * pl->tile.bh;
        tail_ok = dr.H > 0 && choose_halo_tile(dr, pl->m, tf, &pl->tail);
      }
    }
    if (tail_ok) {
      pl->has_tail = true;
      const long long per_row = pl->tile.tiles / pl->tile.tiles_h;
      pl->tile.tiles_h = keep;
      pl->tile.tiles = per_row * keep;
      pl->tile.grid = int(std::min<long long>(pl->tile.tiles, pl->m.sm_count));
      build_halo_params(dk, pl->tail, &pl->kp_tail);
      pl->kp_tail.h0 = keep * pl->tile.bh;
      pl->kp_tail.tail = 1;
    }
    build_halo_params(dk, pl->tile, &pl->kp);
  }
  if (variant == CCONV_VARIANT_STEM) build_stem_params(pl->drun, pl->stile, &pl->skp);
  if (variant == CCONV_VARIANT_DIRECT) {
    build_direct_params(dk, pl->dtile, &pl->dkp);
    pl->diag_skip_once = env_int("CCONV_DIAG_SKIP_FILTER_STAGE", -1);
    // (the staging buffers of the TMA-store epilogue live in the rings of a CTA with a single tile)
    pl->direct_tma_store = pl->dtile.tiles <= pl->dtile.grid && env_int("CCONV_DIRECT_TMA_STORE", 1) != 0;
    if (pl->direct_tma_store) {  // is a piece 128 contiguous bytes of Out?  (same rule as the encoder's)
      const bool f32 = out_dtype == CCONV_OUT_F32;
      const bool merged = !f32 && pl->dtile.bb == 32 && dk.B == 32;
      pl->direct_tma_mode = merged ? 2 : 1;
      if (!merged && pl->dtile.bb * (f32 ? 4 : 2) < 128) pl->direct_tma_store = false;
    }
  }

  if (device >= 0) {
    int prev = 0;
    cudaGetDevice(&prev);
    cudaError_t e = cudaSetDevice(device);
    if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&pl->d_status), 256);
    if (e == cudaSuccess) e = cudaMemset(pl->d_status, 0, 256);
    if (e == cudaSuccess && variant == CCONV_VARIANT_HALO)
      e = halo_kernel_prepare(std::max(pl->tile.smem_bytes, pl->has_tail ? pl->tail.smem_bytes : 0));
    if (variant == CCONV_VARIANT_HALO) pl->packed_bytes = size_t(pl->tile.packed_filter_bytes);
    if (variant == CCONV_VARIANT_STEM) pl->packed_bytes = size_t(pl->stile.packed_filter_bytes);
    pl->packed_bytes = (pl->packed_bytes + 255) & ~size_t(255);
    if (e == cudaSuccess && (variant == CCONV_VARIANT_HALO || variant == CCONV_VARIANT_STEM))
      e = cudaMalloc(&pl->d_packed, 2 * pl->packed_bytes);
    if (e == cudaSuccess && variant == CCONV_VARIANT_DIRECT) e = direct_kernel_prepare();
    if (e == cudaSuccess && variant >= CCONV_VARIANT_HALO && pl->padded) {
      const Dims& r = pl->drun;
      e = cudaMalloc(&pl->d_img_pad, size_t(r.Wi()) * r.Hi() * r.C * r.B * 2);
      if (e == cudaSuccess)
        e = cudaMalloc(&pl->d_out_pad, size_t(r.K) * r.H * r.W * r.B * (out_dtype == CCONV_OUT_F32 ? 4 : 2));
    }
    if (e == cudaSuccess && variant == CCONV_VARIANT_STEM)
      e = stem_kernel_prepare(pl->stile.smem_bytes);
    if (e == cudaSuccess && variant >= CCONV_VARIANT_HALO && env_int("CCONV_TRACE", 0)) {
      pl->trace_rows = (variant == CCONV_VARIANT_HALO     ? pl->tile.grid
                        : variant == CCONV_VARIANT_DIRECT ? pl->dtile.grid
                                                          : pl->stile.grid) + 16;
      e = cudaMalloc(reinterpret_cast<void**>(&pl->d_trace), size_t(pl->trace_rows) * 16 * 8);
      if (e == cudaSuccess) e = cudaMemset(pl->d_trace, 0, size_t(pl->trace_rows) * 16 * 8);
      pl->kp.trace = pl->d_trace;
      pl->skp.trace = pl->d_trace;
      pl->dkp.trace = pl->d_trace;
    }
    cudaSetDevice(prev);
    if (e != cudaSuccess) {
      if (pl->d_status) cudaFree(pl->d_status);
      if (pl->d_packed) cudaFree(pl->d_packed);
      if (pl->d_img_pad) cudaFree(pl->d_img_pad);
      if (pl->d_out_pad) cudaFree(pl->d_out_pad);
      delete pl;
      return cuda_fail(e, "plan device setup");
    }
  }
  if (env_int("CCONV_LOG", 0) && variant == CCONV_VARIANT_STEM) {
    const StemTile& t = pl->stile;
    std::fprintf(stderr,
                 "[cconv] B%d C%d K%d W%d H%d R%d S%d s%dx%d variant=3 tile bw=%d bhm=%d kpad=%d "
                 "kw=%d i_stages=%d tmem=%d tiles=%lld grid=%d smem=%d filt=%u\n",
                 B, C, K, W, H, R, S, sw, sh, t.bw, t.bhm, t.kpad, t.kw, t.i_stages, t.tmem_cols,
                 t.tiles, t.grid, t.smem_bytes, t.filt_bytes);
  } else if (env_int("CCONV_LOG", 0) && variant == CCONV_VARIANT_DIRECT) {
    const DirectTile& t = pl->dtile;
    std::fprintf(stderr,
                 "[cconv] B%d C%d K%d W%d H%d R%d S%d s%dx%d variant=4 tile bb=%d bw=%d bh=%d kt=%d bc=%d "
                 "tg=%d i_stages=%d f_stages=%d acc_bufs=%d tmem=%d tiles=%lld grid=%d smem=%d est_cyc=%.0f\n",
                 B, C, K, W, H, R, S, sw, sh, t.bb, t.bw, t.bh, t.kt, t.bc, t.tg, t.i_stages, t.f_stages,
                 t.acc_bufs, t.tmem_cols, t.tiles, t.grid, t.smem_bytes, t.est_cycles);
  } else if (env_int("CCONV_LOG", 0)) {
    const HaloTile& t = pl->tile;
    std::fprintf(stderr,
                 "[cconv] B%d C%d K%d W%d H%d R%d S%d s%dx%d variant=%d tile bb=%d bw=%d bh=%d "
                 "bc=%d split=%d i_stages=%d f_stages=%d uf=%d acc_bufs=%d tmem=%d tiles=%lld grid=%d smem=%d "
                 "est_cyc=%.0f\n",
                 B, C, K, W, H, R, S, sw, sh, variant, t.bb, t.bw, t.bh, t.bc, t.split, t.i_stages,
                 t.f_stages, t.uf, t.acc_bufs, t.tmem_cols, t.tiles, t.grid, t.smem_bytes,
                 t.est_cycles);
    if (pl->has_tail)
      std::fprintf(stderr, "[cconv]   tail from h=%d: tile bb=%d bw=%d bh=%d bc=%d i_stages=%d tiles=%lld "
                           "grid=%d smem=%d\n",
                   pl->kp_tail.h0, pl->tail.bb, pl->tail.bw, pl->tail.bh, pl->tail.bc,
                   pl->tail.i_stages, pl->tail.tiles, pl->tail.grid, pl->tail.smem_bytes);
  }
  if (want_wait_twin && pl->variant == CCONV_VARIANT_DIRECT) {
    // (a plan without it still works: waiting calls then run the direct kernel)
    cconv_plan* twin = nullptr;
    if (plan_create_impl(&twin, B, C, K, W, H, R, S, sw, sh, device, M_words, CCONV_VARIANT_HALO,
                         out_dtype, image_strides) == CCONV_OK)
      pl->wait_twin = twin;
  }
  *plan_out = pl;
  return CCONV_OK;
}

int cconv_plan_create(cconv_plan** plan_out, int B, int C, int K, int W, int H, int R, int S,
                      int sw, int sh, int device, double M_words, int variant, int out_dtype) {
  return plan_create_impl(plan_out, B, C, K, W, H, R, S, sw, sh, device, M_words, variant, out_dtype,
                          nullptr);
}

int cconv_plan_info_get(const cconv_plan* pl, cconv_plan_info* o) {
  if (!pl || !o) return CCONV_EINVAL;
  std::memset(o, 0, sizeof(*o));
  int arg = 0;
  for (int i = 0; i < 5; ++i) {
    o->term[i] = pl->terms[i];
    if (pl->terms[i] > pl->terms[arg]) arg = i;
  }
  o->bound_words = pl->terms[arg];
  o->bound_argmax = arg + 1;
  o->M_words = pl->M_words;
  for (int i = 0; i < 9; ++i) o->lp_tile[i] = pl->lp_tile[i];
  o->lp_G = pl->lp_G;
  o->lp_words = pl->lp_words;
  o->variant = pl->variant;
  o->wait_variant = pl->wait_twin ? pl->wait_twin->variant : pl->variant;
  o->out_dtype = pl->out_dtype;
  const Dims& d = pl->d;
  o->tail_h0 = pl->view.dk.H;
  o->run_B = pl->drun.B;
  o->run_H = pl->drun.H;
  o->bands = pl->bands;
  o->split = pl->variant == CCONV_VARIANT_HALO ? pl->tile.split : 1;
  o->compulsory_words =
      double(d.Wi()) * d.Hi() * d.C * d.B + double(d.K) * d.R * d.S * d.C + double(d.K) * d.H * d.W * d.B;
  if (pl->variant == CCONV_VARIANT_STEM) {
    const StemTile& t = pl->stile;
    o->bb = 64; o->bc = d.C; o->bk = t.kpad; o->bw = t.bw; o->bh = t.bhm;
    o->halo_w = t.halo_w; o->halo_h = d.sh * (t.bhm - 1) + d.S;
    o->stages = t.i_stages; o->filter_stages = 1; o->grid = t.grid; o->tiles = int(t.tiles);
    o->smem_bytes = t.smem_bytes; o->tmem_cols = t.tmem_cols;
    o->tile_words_smem = t.words_smem;
    o->scratch_bytes = double(t.packed_filter_bytes);
  }
  if (pl->variant == CCONV_VARIANT_DIRECT) {
    const DirectTile& t = pl->dtile;
    o->bb = t.bb; o->bc = t.bc; o->bk = 128 * t.kt; o->bw = t.bw; o->bh = t.bh;
    o->halo_w = t.halo_w; o->halo_h = t.halo_h;
    o->stages = t.i_stages; o->filter_stages = t.f_stages; o->grid = t.grid; o->tiles = int(t.tiles);
    o->smem_bytes = t.smem_bytes; o->tmem_cols = t.tmem_cols;
    o->tile_words_smem = t.words_smem;
    o->scratch_bytes = pl->wait_twin ? double(pl->wait_twin->tile.packed_filter_bytes) : 0.0;
    o->filter_taps = t.tg;
    o->est_cta_cycles = t.cta_cycles;
    o->est_period_cycles = t.est_cycles;
  }
  if (pl->variant == CCONV_VARIANT_HALO) {
    const HaloTile& t = pl->tile;
    o->bb = t.bb; o->bc = t.bc; o->bk = t.bk; o->bw = t.bw; o->bh = t.bh;
    o->halo_w = t.halo_w; o->halo_h = t.halo_h;
    o->stages = t.i_stages; o->filter_stages = t.f_stages; o->grid = t.grid; o->tiles = int(t.tiles);
    o->smem_bytes = t.smem_bytes; o->tmem_cols = t.tmem_cols;
    o->tile_words_smem = t.words_smem;
    o->scratch_bytes = double(t.packed_filter_bytes);
    if (pl->has_tail) {
      const HaloTile& u = pl->tail;
      o->tail_h0 = pl->kp_tail.h0;
      o->tail_bb = u.bb; o->tail_bc = u.bc; o->tail_bw = u.bw; o->tail_bh = u.bh;
      o->tail_tiles = int(u.tiles); o->tail_grid = u.grid;
      // rows kept by the main tiling: scale its staged words; then add the tail's (minus the Out
      // words both estimates include)
      const Dims& r = pl->view.dk;  // what the kernels run
      const double out_words = double(r.K) * r.H * r.W * r.B;
      o->tile_words_smem = double(t.tiles) * ((t.words_smem - out_words) /
                                              (double(t.tiles) / t.tiles_h * ((r.H + t.bh - 1) / t.bh))) +
                           (u.words_smem - double(r.K) * (r.H - pl->kp_tail.h0) * r.W * r.B) + out_words;
    }
  }
  if (o->bb > 0 && pl->variant != CCONV_VARIANT_STEM) {
    o->tile_G = double(o->bb) * o->bc * o->bk * o->bw * o->bh * d.R * d.S;
    o->tile_G_over_lp_G = pl->lp_G > 0 ? o->tile_G / pl->lp_G : 0.0;
  }
  return CCONV_OK;
}

void cconv_plan_destroy(cconv_plan* pl) {
  if (!pl) return;
  if (pl->device >= 0) {
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(pl->device);
    if (pl->d_status) cudaFree(pl->d_status);
    if (pl->d_packed) cudaFree(pl->d_packed);
    if (pl->d_trace) cudaFree(pl->d_trace);
    if (pl->d_img_pad) cudaFree(pl->d_img_pad);
    if (pl->d_out_pad) cudaFree(pl->d_out_pad);
    if (pl->st_image) cudaFree(pl->st_image);
    if (pl->st_filter) cudaFree(pl->st_filter);
    if (pl->st_out) cudaFree(pl->st_out);
    if (pl->d_acc) cudaFree(pl->d_acc);
    if (pl->pp_d2h) cudaStreamSynchronize(pl->pp_d2h);
    if (pl->pp_h2d) cudaStreamSynchronize(pl->pp_h2d);
    if (pl->pp_h2d_f) cudaStreamSynchronize(pl->pp_h2d_f);
    for (int i = 0; i < 2; ++i) {
      if (pl->ev_in_f[i]) cudaEventDestroy(pl->ev_in_f[i]);
      if (pl->pp_image[i]) cudaFree(pl->pp_image[i]);
      if (pl->pp_filter[i]) cudaFree(pl->pp_filter[i]);
      if (pl->pp_out[i]) cudaFree(pl->pp_out[i]);
      if (pl->ev_in[i]) cudaEventDestroy(pl->ev_in[i]);
      if (pl->ev_run[i]) cudaEventDestroy(pl->ev_run[i]);
      if (pl->ev_out[i]) cudaEventDestroy(pl->ev_out[i]);
    }
    if (pl->pp_h2d) cudaStreamDestroy(pl->pp_h2d);
    if (pl->pp_h2d_f) cudaStreamDestroy(pl->pp_h2d_f);
    if (pl->pp_d2h) cudaStreamDestroy(pl->pp_d2h);
    cudaSetDevice(prev);
  }
  if (pl->acc_twin) cconv_plan_destroy(pl->acc_twin);
  if (pl->wait_twin) cconv_plan_destroy(pl->wait_twin);
  delete pl;
}

int cconv_plan_reserve_accumulate(cconv_plan* pl) {
  if (!pl || pl->device < 0) return CCONV_EINVAL;
  if (pl->acc_twin) return CCONV_OK;
  const Dims& d = pl->d;
  cconv_plan* twin = nullptr;
  const int rc = cconv_plan_create(&twin, d.B, d.C, d.K, d.W, d.H, d.R, d.S, d.sw, d.sh, pl->device,
                                   pl->M_words, pl->variant, CCONV_OUT_F32);
  if (rc != CCONV_OK) return rc;
  int prev = 0;
  cudaGetDevice(&prev);
  cudaError_t e = cudaSetDevice(pl->device);
  if (e == cudaSuccess)
    e = cudaMalloc(reinterpret_cast<void**>(&pl->d_acc), size_t(d.K) * d.H * d.W * d.B * sizeof(float));
  cudaSetDevice(prev);
  if (e != cudaSuccess) {
    cconv_plan_destroy(twin);
    pl->d_acc = nullptr;
    return cuda_fail(e, "cconv_plan_reserve_accumulate");
  }
  pl->acc_twin = twin;
  return CCONV_OK;
}

int cconv_forward_accumulate(const cconv_plan* pl, const void* Image, const void* Filter, void* Out,
                             void* cuda_stream) {
  if (!pl || !Image || !Filter || !Out) return CCONV_EINVAL;
  if (!pl->acc_twin || !pl->d_acc) return CCONV_EINVAL;  // not reserved
  if (reinterpret_cast<uintptr_t>(Out) & 31u) return CCONV_EINVAL;
  const int rc = cconv_forward_planned(pl->acc_twin, Image, Filter, pl->d_acc, cuda_stream);
  if (rc != CCONV_OK) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const Dims& d = pl->d;
  const long long n = (long long)d.K * d.H * d.W * d.B;
  if (pl->out_dtype == CCONV_OUT_F32)
    cconv_accumulate_kernel<float><<<grid_for((n + 3) / 4), 256, 0, stream>>>(static_cast<float*>(Out), pl->d_acc, n);
  else
    cconv_accumulate_kernel<__nv_bfloat16><<<grid_for((n + 3) / 4), 256, 0, stream>>>(
        static_cast<__nv_bfloat16*>(Out), pl->d_acc, n);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "cconv_accumulate_kernel");
  // an ordinary launch: nothing behind it starts before it is complete
  note_ordinary_launch(cuda_stream);
  return CCONV_OK;
}

int cconv_forward_planned(const cconv_plan* pl, const void* Image, const void* Filter, void* Out,
                          void* cuda_stream) {
  if (!pl || !Image || !Filter || !Out) return CCONV_EINVAL;
  if (pl->device < 0) return CCONV_EINVAL;  // inspection-only plan
  int cur = -1;
  if (cudaGetDevice(&cur) != cudaSuccess || cur != pl->device) return CCONV_EINVAL;  // wrong current device
  if (!aligned16(Image) || !aligned16(Filter) || (reinterpret_cast<uintptr_t>(Out) & 31u))
    return CCONV_EINVAL;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  CallSpans spans = spans_of(pl->d, pl->out_dtype, Image, Filter, Out);
  spans.image.hi = spans.image.lo + pl->image_span_bytes;
  if (pl->variant == CCONV_VARIANT_SIMT) {
    note_call(cuda_stream, spans, Overlap::kNone, pl->m.sm_count);
    cudaError_t e = launch_simt(Image, Filter, Out, pl->out_dtype == CCONV_OUT_F32, pl->d, stream);
    return e == cudaSuccess ? CCONV_OK : cuda_fail(e, "launch_simt");
  }
  if (pl->variant == CCONV_VARIANT_DIRECT) {
    // SMs' worth of resident CTAs: CTAs that need more than half of an SM's shared memory or tensor
    // memory have an SM each (under-counting only keeps calls on the list for longer)
    spans.sms = double(pl->dtile.grid) /
                std::max(1, std::min(pl->m.smem_optin_bytes / std::max(pl->dtile.smem_bytes, 1),
                                     pl->m.tmem_cols / std::max(pl->dtile.tmem_cols, 1)));
    const int hazards = note_call_hazards(cuda_stream, spans, Overlap::kDeep, pl->m.sm_count);
    const bool hazard = hazards != 0;
    if (hazard && pl->wait_twin) {
      // The call starts only when the stream's earlier work is complete, so it cannot run beside
      // other calls: the halo kernel's tiling gives it the whole GPU.  That kernel writes Out only
      // after every earlier kernel is complete; its inputs wait when they are what conflicts.
      return launch_tensor_core(pl->wait_twin, Image, Filter, Out, (hazards & kHazardInputs) != 0, stream);
    }
    CUtensorMap tmi, tmf, tmo{};
    {
      std::lock_guard<std::mutex> lk(pl->mu);
      cconv_plan::MapSlot& si = pl->img_maps[cconv_plan::map_slot(Image)];
      if (si.ptr != Image) {
        const int rc = encode_direct_image_map(pl->view, pl->dtile, Image, &si.tm);
        if (rc != CCONV_OK) return rc;
        si.ptr = Image;
      }
      cconv_plan::MapSlot& sf = pl->flt_maps[cconv_plan::map_slot(Filter)];
      if (sf.ptr != Filter) {
        const int rc = encode_direct_filter_map(pl->view.dk, pl->dtile, Filter, &sf.tm);
        if (rc != CCONV_OK) return rc;
        sf.ptr = Filter;
      }
      tmi = si.tm;
      tmf = sf.tm;
      if (pl->direct_tma_store) {
        cconv_plan::MapSlot& so = pl->out_maps[cconv_plan::map_slot(Out)];
        if (so.ptr != Out) {
          int merged = 0;
          const int rc = encode_direct_out_map(pl->view.dk, pl->dtile, pl->out_dtype == CCONV_OUT_F32, Out,
                                               &so.tm, &merged);
          if (rc != CCONV_OK) return rc;
          so.ptr = Out;
        }
        tmo = so.tm;
      }
    }
    DirectKernelParams kp = pl->dkp;
    {
      std::lock_guard<std::mutex> lk(pl->mu);
      kp.skip_filter_stage = pl->diag_skip_once;
      pl->diag_skip_once = -1;
    }
    kp.wait_prev = hazard ? 1 : 0;
    kp.out_tma = pl->direct_tma_store ? pl->direct_tma_mode : 0;
    cudaError_t e = launch_direct(tmi, tmf, tmo, Out, pl->out_dtype == CCONV_OUT_F32, kp, pl->dtile.grid,
                                  pl->dtile.smem_bytes, pl->d_status, stream);
    return e == cudaSuccess ? CCONV_OK : cuda_fail(e, "launch_direct");
  }
  // (the stem kernel's calls overlap like the direct kernel's: reads and writes beside earlier calls)
  if (pl->variant == CCONV_VARIANT_STEM) spans.sms = double(pl->stile.grid);
  const bool inputs_hazard =
      note_call(cuda_stream, spans,
                pl->variant == CCONV_VARIANT_STEM ? Overlap::kDeep : Overlap::kInputsEarly, pl->m.sm_count);
  // Batch sizes that are not multiples of 8: the kernels run on zero-padded copies (see cconv_plan).
  void* const user_out = Out;
  const void* const user_image = Image;
  BandGeom g{};
  if (pl->padded) {
    const Dims& r = pl->drun;
    g = BandGeom{pl->d.Wi(), pl->d.Hi(), r.Hi(), pl->d.C, pl->d.B, r.B, pl->bands, r.H, pl->d.sh};
    Image = pl->d_img_pad;
    Out = pl->d_out_pad;
  }
  const int rc_run = launch_tensor_core(pl, Image, Filter, Out, inputs_hazard, stream,
                                        pl->padded ? &g : nullptr, user_image);
  if (rc_run != CCONV_OK || !pl->padded) return rc_run;
  {
    const Dims& d = pl->d;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid_for((long long)d.K * g.Hr * d.W * (g.Bp / 8)));
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t ec;
    if (pl->out_dtype == CCONV_OUT_F32)
      ec = cudaLaunchKernelEx(&cfg, cconv_compact_bands_kernel<float>, static_cast<const float*>(Out),
                              static_cast<float*>(user_out), (long long)d.K, (long long)d.H,
                              (long long)d.W, g);
    else
      ec = cudaLaunchKernelEx(&cfg, cconv_compact_bands_kernel<unsigned short>,
                              static_cast<const unsigned short*>(Out),
                              static_cast<unsigned short*>(user_out), (long long)d.K, (long long)d.H,
                              (long long)d.W, g);
    if (ec != cudaSuccess) return cuda_fail(ec, "cconv_compact_bands_kernel");
    // the compaction kernel never releases its dependents early: nothing behind it starts before it
    // is complete
    note_ordinary_launch(cuda_stream);
  }
  return CCONV_OK;
}

int cconv_forward(const void* Image, const void* Filter, void* Out, int B, int C, int K, int W,
                  int H, int R, int S, int sw, int sh, int out_dtype, void* cuda_stream) {
  int dev = 0;
  CCONV_CUDA(cudaGetDevice(&dev));
  cconv_plan* pl = nullptr;
  {
    std::lock_guard<std::mutex> lk(g_cache_mu);
    auto key = std::make_tuple(dev, cuda_stream, B, C, K, W, H, R, S, sw, sh, out_dtype);
    auto it = g_cache.find(key);
    if (it == g_cache.end()) {
      int rc = cconv_plan_create(&pl, B, C, K, W, H, R, S, sw, sh, dev, 0.0, CCONV_VARIANT_AUTO,
                                 out_dtype);
      if (rc != CCONV_OK) return rc;
      g_cache[key] = pl;
    } else {
      pl = it->second;
    }
  }
  return cconv_forward_planned(pl, Image, Filter, Out, cuda_stream);
}

int cconv_forward_strided(const void* Image, const int64_t image_strides[4], const void* Filter,
                          const int64_t filter_strides[4], void* Out, const int64_t out_strides[4],
                          int B, int C, int K, int W, int H, int R, int S, int sw, int sh,
                          int out_dtype, void* cuda_stream) {
  if (!Image || !Filter || !Out || !image_strides || !filter_strides || !out_strides) return CCONV_EINVAL;
  const Dims d{B, C, K, W, H, R, S, sw, sh};
  if (!d.positive()) return CCONV_EINVAL;
  if (out_dtype != CCONV_OUT_BF16 && out_dtype != CCONV_OUT_F32) return CCONV_EINVAL;
  for (int i = 0; i < 4; ++i)
    if (image_strides[i] <= 0 || filter_strides[i] <= 0 || out_strides[i] <= 0) return CCONV_EINVAL;
  const size_t oel = out_dtype == CCONV_OUT_F32 ? 4 : 2;
  if ((reinterpret_cast<uintptr_t>(Image) & 1u) || (reinterpret_cast<uintptr_t>(Filter) & 1u) ||
      (reinterpret_cast<uintptr_t>(Out) & (oel - 1)))
    return CCONV_EINVAL;
  const int64_t dense_i[4] = {int64_t(d.Hi()) * C * B, int64_t(C) * B, B, 1};
  const int64_t dense_f[4] = {int64_t(R) * S * C, int64_t(S) * C, C, 1};
  const int64_t dense_o[4] = {int64_t(H) * W * B, int64_t(W) * B, B, 1};
  bool img_dense = true, flt_dense = true, out_dense = true;
  for (int i = 0; i < 4; ++i) {
    // (the stride of a subscript with a single value is never used)
    const int ext_i[4] = {d.Wi(), d.Hi(), C, B}, ext_f[4] = {K, R, S, C}, ext_o[4] = {K, H, W, B};
    img_dense = img_dense && (ext_i[i] == 1 || image_strides[i] == dense_i[i]);
    flt_dense = flt_dense && (ext_f[i] == 1 || filter_strides[i] == dense_f[i]);
    out_dense = out_dense && (ext_o[i] == 1 || out_strides[i] == dense_o[i]);
  }
  const bool aligned = aligned16(Image) && aligned16(Filter) && !(reinterpret_cast<uintptr_t>(Out) & 31u);
  // 1. the ABI's own dense layout: the planned path
  if (img_dense && flt_dense && out_dense && aligned)
    return cconv_forward(Image, Filter, Out, B, C, K, W, H, R, S, sw, sh, out_dtype, cuda_stream);
  // 2. a strided view of the Image whose images are contiguous and whose other strides keep 16-byte
  //    alignment (a window of a larger array, padded rows, a channel slice), Filter and Out dense:
  //    the tensor-core kernels read it through a tensor map built from the strides
  const bool img_tma = (B == 1 || image_strides[3] == 1) && image_strides[0] % 8 == 0 &&
                       image_strides[1] % 8 == 0 && image_strides[2] % 8 == 0 && B % 8 == 0;
  if (img_tma && flt_dense && out_dense && aligned) {
    int dev = 0;
    CCONV_CUDA(cudaGetDevice(&dev));
    cconv_plan* pl = nullptr;
    int rc = CCONV_OK;
    {
      std::lock_guard<std::mutex> lk(g_cache_mu);
      auto key = std::make_tuple(dev, cuda_stream, B, C, K, W, H, R, S, sw, sh, out_dtype,
                                 (long long)image_strides[0], (long long)image_strides[1],
                                 (long long)image_strides[2]);
      auto it = g_cache_strided.find(key);
      if (it == g_cache_strided.end()) {
        const long long ist[4] = {image_strides[0], image_strides[1], image_strides[2], 1};
        rc = plan_create_impl(&pl, B, C, K, W, H, R, S, sw, sh, dev, 0.0, CCONV_VARIANT_AUTO, out_dtype, ist);
        g_cache_strided[key] = rc == CCONV_OK ? pl : nullptr;  // remember a refusal too
      } else {
        pl = it->second;
        if (!pl) rc = CCONV_EUNSUPPORTED;
      }
    }
    if (rc == CCONV_OK) return cconv_forward_planned(pl, Image, Filter, Out, cuda_stream);
    if (rc != CCONV_EUNSUPPORTED) return rc;
  }
  // 3. any other strides (column-major storage, transposed arrays, ...): the CUDA-core kernel
  StridedLayout L;
  for (int i = 0; i < 4; ++i) {
    L.image[i] = image_strides[i];
    L.filter[i] = filter_strides[i];
    L.out[i] = out_strides[i];
    L.order[i] = i;
  }
  std::sort(L.order, L.order + 4, [&](int a, int b) { return out_strides[a] < out_strides[b]; });
  note_ordinary_launch(cuda_stream);
  cudaError_t e = launch_simt_strided(Image, Filter, Out, out_dtype == CCONV_OUT_F32, d, L,
                                      static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? CCONV_OK : cuda_fail(e, "launch_simt_strided");
}

int cconv_forward_host(cconv_plan* pl, const void* hImage, const void* hFilter, void* hOut,
                       void* cuda_stream) {
  if (!pl || !hImage || !hFilter || !hOut || pl->device < 0) return CCONV_EINVAL;
  const Dims& d = pl->d;
  const size_t ni = size_t(d.Wi()) * d.Hi() * d.C * d.B * 2;
  const size_t nf = size_t(d.K) * d.R * d.S * d.C * 2;
  const size_t no = size_t(d.K) * d.H * d.W * d.B * (pl->out_dtype == CCONV_OUT_F32 ? 4 : 2);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (!pl->st_image) {
    CCONV_CUDA(cudaMalloc(&pl->st_image, ni));
    CCONV_CUDA(cudaMalloc(&pl->st_filter, nf));
    CCONV_CUDA(cudaMalloc(&pl->st_out, no));
  }
  CCONV_CUDA(cudaMemcpyAsync(pl->st_image, hImage, ni, cudaMemcpyHostToDevice, stream));
  CCONV_CUDA(cudaMemcpyAsync(pl->st_filter, hFilter, nf, cudaMemcpyHostToDevice, stream));
  int rc = cconv_forward_planned(pl, pl->st_image, pl->st_filter, pl->st_out, cuda_stream);
  if (rc != CCONV_OK) return rc;
  CCONV_CUDA(cudaMemcpyAsync(hOut, pl->st_out, no, cudaMemcpyDeviceToHost, stream));
  int detail = 0;
  return cconv_plan_status(pl, cuda_stream, &detail);
}

int cconv_forward_host_async(cconv_plan* pl, const void* hImage, const void* hFilter, void* hOut,
                             void* cuda_stream) {
  if (!pl || !hImage || !hFilter || !hOut || pl->device < 0) return CCONV_EINVAL;
  int cur = -1;
  if (cudaGetDevice(&cur) != cudaSuccess || cur != pl->device) return CCONV_EINVAL;
  const Dims& d = pl->d;
  const size_t ni = size_t(d.Wi()) * d.Hi() * d.C * d.B * 2;
  const size_t nf = size_t(d.K) * d.R * d.S * d.C * 2;
  const size_t no = size_t(d.K) * d.H * d.W * d.B * (pl->out_dtype == CCONV_OUT_F32 ? 4 : 2);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (!pl->pipe_ready) {
    CCONV_CUDA(cudaStreamCreateWithFlags(&pl->pp_h2d, cudaStreamNonBlocking));
    CCONV_CUDA(cudaStreamCreateWithFlags(&pl->pp_h2d_f, cudaStreamNonBlocking));
    CCONV_CUDA(cudaStreamCreateWithFlags(&pl->pp_d2h, cudaStreamNonBlocking));
    for (int i = 0; i < 2; ++i) {
      CCONV_CUDA(cudaEventCreateWithFlags(&pl->ev_in_f[i], cudaEventDisableTiming));
      CCONV_CUDA(cudaMalloc(&pl->pp_image[i], ni));
      CCONV_CUDA(cudaMalloc(&pl->pp_filter[i], nf));
      CCONV_CUDA(cudaMalloc(&pl->pp_out[i], no));
      CCONV_CUDA(cudaEventCreateWithFlags(&pl->ev_in[i], cudaEventDisableTiming));
      CCONV_CUDA(cudaEventCreateWithFlags(&pl->ev_run[i], cudaEventDisableTiming));
      CCONV_CUDA(cudaEventCreateWithFlags(&pl->ev_out[i], cudaEventDisableTiming));
    }
    pl->pipe_ready = true;
  }
  const int set = int(pl->pipe_calls++ & 1u);
  // inputs: this set's arrays are free once the kernels of the call two back have run
  // (Image and Filter on a stream each: a copy of this size is mostly fixed cost)
  CCONV_CUDA(cudaStreamWaitEvent(pl->pp_h2d, pl->ev_run[set], 0));
  CCONV_CUDA(cudaStreamWaitEvent(pl->pp_h2d_f, pl->ev_run[set], 0));
  CCONV_CUDA(cudaMemcpyAsync(pl->pp_image[set], hImage, ni, cudaMemcpyHostToDevice, pl->pp_h2d));
  CCONV_CUDA(cudaMemcpyAsync(pl->pp_filter[set], hFilter, nf, cudaMemcpyHostToDevice, pl->pp_h2d_f));
  CCONV_CUDA(cudaEventRecord(pl->ev_in[set], pl->pp_h2d));
  CCONV_CUDA(cudaEventRecord(pl->ev_in_f[set], pl->pp_h2d_f));
  // kernels: after the inputs have landed and this set's Out of two calls back has been copied out
  CCONV_CUDA(cudaStreamWaitEvent(stream, pl->ev_in[set], 0));
  CCONV_CUDA(cudaStreamWaitEvent(stream, pl->ev_in_f[set], 0));
  CCONV_CUDA(cudaStreamWaitEvent(stream, pl->ev_out[set], 0));
  const int rc = cconv_forward_planned(pl, pl->pp_image[set], pl->pp_filter[set], pl->pp_out[set], cuda_stream);
  if (rc != CCONV_OK) return rc;
  CCONV_CUDA(cudaEventRecord(pl->ev_run[set], stream));
  // Out: back to the host on the other copy stream
  CCONV_CUDA(cudaStreamWaitEvent(pl->pp_d2h, pl->ev_run[set], 0));
  CCONV_CUDA(cudaMemcpyAsync(hOut, pl->pp_out[set], no, cudaMemcpyDeviceToHost, pl->pp_d2h));
  CCONV_CUDA(cudaEventRecord(pl->ev_out[set], pl->pp_d2h));
  return CCONV_OK;
}

int cconv_host_wait(cconv_plan* pl, void* cuda_stream) {
  if (!pl || pl->device < 0) return CCONV_EINVAL;
  if (pl->pp_d2h) CCONV_CUDA(cudaStreamSynchronize(pl->pp_d2h));
  int detail = 0;
  return cconv_plan_status(pl, cuda_stream, &detail);
}

int cconv_plan_trace_read(const cconv_plan* pl, unsigned long long* host_out, int max_u64) {
  if (!pl || !host_out || max_u64 <= 0) return CCONV_EINVAL;
  if (!pl->d_trace) return 0;
  const int n = std::min(max_u64, pl->trace_rows * 16);
  CCONV_CUDA(cudaMemcpy(host_out, pl->d_trace, size_t(n) * 8, cudaMemcpyDeviceToHost));
  return n;
}

int cconv_stream_order_probe(void* stream_key, const void* image_lo, const void* image_hi,
                             const void* filter_lo, const void* filter_hi, const void* out_lo,
                             const void* out_hi, int overlap, double sms_by_memory,
                             double sms_by_threads, int sm_count) {
  if (overlap < 0 || overlap > 2 || sm_count <= 0) return CCONV_EINVAL;
  CallSpans c;
  c.image = Span{static_cast<const char*>(image_lo), static_cast<const char*>(image_hi)};
  c.filter = Span{static_cast<const char*>(filter_lo), static_cast<const char*>(filter_hi)};
  c.out = Span{static_cast<const char*>(out_lo), static_cast<const char*>(out_hi)};
  c.sms = sms_by_memory;
  c.sms_by_threads = sms_by_threads;
  const Overlap how = overlap == 0 ? Overlap::kNone : overlap == 1 ? Overlap::kInputsEarly : Overlap::kDeep;
  return note_call_hazards(stream_key, c, how, sm_count);
}

int cconv_plan_status(const cconv_plan* pl, void* cuda_stream, int* detail_out) {
  if (!pl || pl->device < 0 || !pl->d_status) return CCONV_EINVAL;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  int st = 0;
  CCONV_CUDA(cudaMemcpyAsync(&st, pl->d_status, sizeof(int), cudaMemcpyDeviceToHost, stream));
  CCONV_CUDA(cudaStreamSynchronize(stream));
  if (st != 0) {
    CCONV_CUDA(cudaMemsetAsync(pl->d_status, 0, sizeof(int), stream));
    CCONV_CUDA(cudaStreamSynchronize(stream));
  }
  // (accumulating calls and calls that had to wait run on twin plans with status words of their own)
  for (const cconv_plan* twin : {pl->acc_twin, pl->wait_twin}) {
    if (!twin) continue;
    int st2 = 0;
    const int rc2 = cconv_plan_status(twin, cuda_stream, &st2);
    if (rc2 != CCONV_OK && rc2 != CCONV_EDEVICE_TIMEOUT) return rc2;
    st |= st2;
  }
  if (detail_out) *detail_out = st;
  return st != 0 ? CCONV_EDEVICE_TIMEOUT : CCONV_OK;
}

}  // extern "C"
