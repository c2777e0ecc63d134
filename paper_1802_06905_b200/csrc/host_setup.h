// Host-side helpers shared by the entry points: last-error text, the halo kernel's parameter block
// and the Image tensor map.  No device memory is allocated here.
#pragma once
#include <cuda.h>

#include <string>

#include "kernels.h"
#include "planner.h"

namespace cconv {

void set_last_cuda_error(const std::string& msg);  // per host thread
const char* last_cuda_error();

// Everything cconv_halo_kernel needs to know about a shape and its tile (descriptors included).
void build_halo_params(const Dims& d, const HaloTile& t, HaloKernelParams* p);

// TMA descriptor of the Image view `v` as (b, c, x, y) with the tile's halo box.  Returns 0, or -3
// (CCONV_ECUDA) with the last-error text set.  A pure host-side encode.
int encode_image_map(const ImageView& v, const HaloTile& t, const void* image, CUtensorMap* tm);

// The direct-Filter kernel: parameter block, Image map (b, c, x, y) with the tile's halo box, and
// Filter map: [K][R][S][C] viewed as (c, k, tap) with a box of bc channels x 128*kt out-channels x
// tg taps, K-major rows swizzled over bc*2 bytes.
void build_direct_params(const Dims& d, const DirectTile& t, DirectKernelParams* p);
int encode_direct_image_map(const ImageView& v, const DirectTile& t, const void* image, CUtensorMap* tm);
int encode_direct_filter_map(const Dims& d, const DirectTile& t, const void* filter, CUtensorMap* tm);
// Out [K][H][W][B] as a 4-D tensor (b, w, h, k) whose box is one epilogue warp's piece: 32 out-channel
// rows of 128 contiguous bytes, 128-byte swizzle; *merged_wb = 1 when the first coordinate is the
// merged subscript w*B + b and the second is unused.  CCONV_EUNSUPPORTED where a piece is not
// contiguous in Out (bf16, b_b = 32 < B).
int encode_direct_out_map(const Dims& d, const DirectTile& t, bool out_f32, void* out, CUtensorMap* tm,
                          int* merged_wb);

// The same two pieces for the small-C ("stem") kernel: Image viewed as (b, m = y*C + c, x).
void build_stem_params(const Dims& d, const StemTile& t, StemKernelParams* p);
int encode_stem_image_map(const Dims& d, const StemTile& t, const void* image, CUtensorMap* tm);


// ---- ordering between calls that overlap on the GPU -------------------------------------------
// The tensor-core kernels let the next kernel of their stream start before they are complete (that
// hides launch gaps, and lets small calls run side by side on different SMs), and every one of them
// ends only after the kernel in front of it has, so completion still propagates in stream order.
// What stream order also promises -- a call sees the results of the calls before it, and does not
// overwrite what they still read -- is kept by the host: per stream it remembers the address ranges
// of the calls that may still be running, and a new call whose arrays conflict with one of them is
// told to wait for the stream's earlier work before it touches memory.
struct Span {
  const char* lo = nullptr;
  const char* hi = nullptr;
  bool meets(const Span& o) const { return lo < o.hi && o.lo < hi; }
};
struct CallSpans {
  Span image, filter, out;
  // SMs' worth of CTAs the call keeps resident, counted on one resource each: by shared / tensor
  // memory (grid / CTAs per SM: the tensor-core kernels) and by thread slots (pooling blocks).
  // Either sum reaching the SM count proves that the calls behind it are complete; a call adds
  // nothing to a resource it hardly uses, which only keeps older calls on the list for longer.
  double sms = 0, sms_by_threads = 0;
};
CallSpans spans_of(const Dims& d, int out_dtype, const void* Image, const void* Filter, const void* Out);

enum class Overlap {
  kNone,         // the call's kernels neither start early nor release early (ordinary launches)
  kInputsEarly,  // halo / stem calls: inputs may be read while the call in front still runs; Out is
                 // written only after every earlier call is complete; at most this call is still
                 // running when the next one starts
  kDeep,         // direct calls: reads and writes may overlap any number of earlier calls
};
// Registers a call and says whether it must wait for the stream's earlier work before touching
// memory.  Calls known to be complete are forgotten: every CTA of an overlapping call stays
// resident until the call in front of it is complete, so a call can still be running only while
// the CTAs of all calls launched after it (but the newest) fit the `sm_count` SMs together.
bool note_call(void* stream, const CallSpans& c, Overlap how, int sm_count);
// The same, telling the two kinds of conflict apart: kHazardInputs = this call's Image or Filter
// meets the Out of a call that may still be running; kHazardOut = its Out meets one of their arrays.
constexpr int kHazardInputs = 1, kHazardOut = 2;
int note_call_hazards(void* stream, const CallSpans& c, Overlap how, int sm_count);
// An ordinary launch of this library (pooling, the accumulate pass, ...) went into the stream.
void note_ordinary_launch(void* stream);

}  // namespace cconv
