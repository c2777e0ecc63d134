// cconv_forward_noalloc: the tensor-core convolution for callers that must not allocate.
//
// Some callers cannot call cudaMalloc when they need a convolution: code that runs while a CUDA
// graph is being captured, a callback on a latency-critical serving path whose memory was carved
// up at start-up, a process whose allocator forbids (or would serialise on) device allocation.
// The planned entry points keep the repacked Filter and a status word in memory they cudaMalloc at
// plan creation; this one keeps both in a fixed array that is part of the library image.
//
// The array lives in this translation unit.  In host code its name is only a stand-in for the
// device object (handing it to a kernel would pass a host address), so its device address is
// looked up once per device with cudaGetSymbolAddress, with that device current, and that pointer
// is what the kernels receive.
#include <cuda.h>
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/cconv.h"
#include "host_setup.h"
#include "kernels.h"
#include "planner.h"

using namespace cconv;

namespace {

constexpr size_t kStatusBytes = 256;  // the status word, padded so the Filter blocks stay aligned
// Every GPU that loads the library holds this array until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kStatusBytes + CCONV_NOALLOC_MAX_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;

struct DeviceSetup {
  bool ready = false;
  unsigned char* scratch = nullptr;  // device address of g_noalloc_scratch on this device
  Machine machine{};
  int prepared_smem = 0;  // largest dynamic shared memory the halo kernels were opted in to
};

std::mutex g_mu;
DeviceSetup g_dev[kMaxDevices];

int fail(cudaError_t e, const char* what) {
  set_last_cuda_error(std::string(what) + ": " + cudaGetErrorString(e));
  return CCONV_ECUDA;
}

// Once per device, with that device current: the scratch array's device address and the device's
// limits.  Neither call allocates.
int setup_device(int dev, DeviceSetup** out) {
  if (dev < 0 || dev >= kMaxDevices) return CCONV_EINVAL;
  DeviceSetup& s = g_dev[dev];
  if (!s.ready) {
    void* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
    if (e != cudaSuccess) return fail(e, "cudaGetSymbolAddress(g_noalloc_scratch)");
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, dev);
    if (e != cudaSuccess) return fail(e, "cudaGetDeviceProperties");
    if (prop.major != 10) return CCONV_EUNSUPPORTED;
    s.scratch = static_cast<unsigned char*>(ptr);
    s.machine.sm_count = prop.multiProcessorCount;
    s.machine.smem_optin_bytes = int(prop.sharedMemPerBlockOptin);
    s.machine.l2_bytes = prop.l2CacheSize;
    s.ready = true;
  }
  *out = &s;
  return CCONV_OK;
}

}  // namespace

extern "C" int cconv_forward_noalloc(const void* Image, const void* Filter, void* Out, int B, int C,
                                     int K, int W, int H, int R, int S, int sw, int sh,
                                     int out_dtype, void* cuda_stream, int* device_status_out) {
  if (!Image || !Filter || !Out) return CCONV_EINVAL;
  const Dims d{B, C, K, W, H, R, S, sw, sh};
  if (!d.positive()) return CCONV_EINVAL;
  if (out_dtype != CCONV_OUT_BF16 && out_dtype != CCONV_OUT_F32) return CCONV_EINVAL;
  if (((reinterpret_cast<uintptr_t>(Image) | reinterpret_cast<uintptr_t>(Filter)) & 15u) ||
      (reinterpret_cast<uintptr_t>(Out) & 31u))
    return CCONV_EINVAL;
  const ImageView view = image_view(d);
  const Dims& dk = view.dk;
  if (!halo_supported(dk, nullptr)) return CCONV_EUNSUPPORTED;

  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(e, "cudaGetDevice");
  std::lock_guard<std::mutex> lk(g_mu);  // one scratch array: host-side calls are serialised too
  DeviceSetup* ds = nullptr;
  int rc = setup_device(dev, &ds);
  if (rc != CCONV_OK) return rc;

  HaloTile tile;
  const int no_force[6] = {0, 0, 0, 0, 0, 0};
  if (!choose_halo_tile(dk, ds->machine, no_force, &tile)) return CCONV_EUNSUPPORTED;
  if (tile.packed_filter_bytes > (long long)CCONV_NOALLOC_MAX_SCRATCH_BYTES) return CCONV_ETOOLARGE;

  HaloKernelParams kp;
  build_halo_params(dk, tile, &kp);
  CUtensorMap tm;
  rc = encode_image_map(view, tile, Image, &tm);
  if (rc != CCONV_OK) return rc;
  if (tile.smem_bytes > ds->prepared_smem) {
    // (raises every instantiation to the device's limit: needed once per device)
    e = halo_kernel_prepare(tile.smem_bytes);
    if (e != cudaSuccess) return fail(e, "cudaFuncSetAttribute(max dynamic shared memory)");
    ds->prepared_smem = ds->machine.smem_optin_bytes;
  }

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  int* status = reinterpret_cast<int*>(ds->scratch);
  unsigned char* packed = ds->scratch + kStatusBytes;
  // The array keeps whatever the last call left.  The packed Filter is rewritten in full (zero
  // padding included) by the packing kernel; the status word only ever has bits OR-ed into it by the
  // kernels and is cleared by whoever reads it (below, or cconv_noalloc_status).
  // Stream order: the packing kernel is an ordinary launch, so everything in front of this call is
  // complete before it reads anything; the convolution lets the kernel behind it start early, so the
  // call is registered like a planned one (a following call that reads this Out will wait).
  note_call(cuda_stream, spans_of(d, out_dtype, Image, Filter, Out), Overlap::kInputsEarly,
            ds->machine.sm_count);
  e = launch_pack_filter(Filter, packed, d, tile.c16, tile.tiles_k, /*overlap_prev=*/false, stream);
  if (e != cudaSuccess) return fail(e, "launch_pack_filter");
  e = launch_halo(tm, packed, Out, out_dtype == CCONV_OUT_F32, kp, tile.grid, tile.smem_bytes, status,
                  stream);
  if (e != cudaSuccess) return fail(e, "launch_halo");
  if (device_status_out) {
    *device_status_out = 0;
    e = cudaMemcpyAsync(device_status_out, status, sizeof(int), cudaMemcpyDeviceToHost, stream);
    if (e != cudaSuccess) return fail(e, "cudaMemcpyAsync(status)");
    e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return fail(e, "cudaStreamSynchronize");
    if (*device_status_out != 0) {
      e = cudaMemsetAsync(status, 0, sizeof(int), stream);
      if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
      if (e != cudaSuccess) return fail(e, "clearing the status word");
      return CCONV_EDEVICE_TIMEOUT;
    }
  }
  return CCONV_OK;
}

extern "C" int cconv_noalloc_status(void* cuda_stream, int* detail_out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(e, "cudaGetDevice");
  std::lock_guard<std::mutex> lk(g_mu);
  DeviceSetup* ds = nullptr;
  const int rc = setup_device(dev, &ds);
  if (rc != CCONV_OK) return rc;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  int* status = reinterpret_cast<int*>(ds->scratch);
  int st = 0;
  e = cudaMemcpyAsync(&st, status, sizeof(int), cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  if (e == cudaSuccess && st != 0) {
    e = cudaMemsetAsync(status, 0, sizeof(int), stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  }
  if (e != cudaSuccess) return fail(e, "reading the status word");
  if (detail_out) *detail_out = st;
  return st != 0 ? CCONV_EDEVICE_TIMEOUT : CCONV_OK;
}
