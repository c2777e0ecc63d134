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

// The same two pieces for the small-C ("stem") kernel: Image viewed as (b, m = y*C + c, x).
void build_stem_params(const Dims& d, const StemTile& t, StemKernelParams* p);
int encode_stem_image_map(const Dims& d, const StemTile& t, const void* image, CUtensorMap* tm);

}  // namespace cconv
