// pvt_vstep_select_noalloc: the subspace choice for callers that cannot allocate.
//
// Some users of this library have no way to obtain device memory at the moment
// they need a selection: a training loop whose allocator is frozen (every byte
// handed out up front, or an allocator that must not be entered from a callback
// or a real-time thread), a plug-in that runs inside a host application owning
// all device memory, or code that runs where cudaMalloc would synchronise the
// whole device.  pvt_vstep_select needs a caller-provided workspace of about
// 4 bytes per weight group; this variant brings its own, a fixed array that is
// part of the library image, so the caller passes only inputs and outputs.
//
// The price: the array occupies device memory on every GPU that loads the
// library until the process exits, the layer size is capped, and all calls share
// the one array (see the notes at the entry point).
#include <mutex>

#include "pvt_internal.h"

namespace pvt {
namespace {

// Largest layer the built-in scratch serves: 2^21 groups of 8 weights, e.g. a
// 4096 x 4096 matrix.  Layout needs: 256 B header + 18 KiB histograms + 4 B per
// group (keys) + 8 B per tile of 4096 groups + 1 B per group (candidate list of a
// quarter of the groups), each part rounded up to 256 B.
constexpr uint64_t kNoAllocMaxGroups = 1ull << 21;
constexpr size_t kNoAllocScratchBytes =
    256 + 18432 + 4 * kNoAllocMaxGroups + 8 * (kNoAllocMaxGroups / kSelTile) + kNoAllocMaxGroups + 1280;

// File-scope device array.  In host code this name is only a handle for the
// runtime's symbol table, not a device address: the address is looked up with
// cudaGetSymbolAddress below and only that pointer is given to kernels.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mu;
void* g_scratch_ptr[kMaxDevices] = {};  // device address of the array, per device ordinal

// Device address of the scratch array on the current device; looked up once per
// device (with that device current) and cached.
cudaError_t scratch_for_current_device(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mu);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    if (!p || (reinterpret_cast<uintptr_t>(p) & (kWsAlign - 1))) return cudaErrorInvalidSymbol;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

}  // namespace
}  // namespace pvt

using namespace pvt;

extern "C" int pvt_vstep_select_noalloc(const pvt_layer* layer, uint64_t k, uint32_t* idx_out, uint32_t* status_out,
                                        void* cuda_stream) {
  if (!layer) return PVT_EINVAL;
  if (layer->rows <= 0 || layer->cols <= 0) return PVT_EINVAL;
  if (layer->group_dim != kGroupDim) return layer->group_dim > 0 ? PVT_EUNSUPPORTED : PVT_EINVAL;
  if (layer->cols % kGroupDim != 0) return PVT_EINVAL;
  const uint64_t G = (uint64_t)layer->rows * (uint64_t)(layer->cols / kGroupDim);
  if (!(layer->eta >= 0.0f) || !(layer->eta <= 3.0e38f)) return PVT_EINVAL;
  if (k < 1 || k > G) return PVT_EINVAL;
  if (!layer->g || (reinterpret_cast<uintptr_t>(layer->g) & 15u) || !idx_out) return PVT_EINVAL;
  if ((reinterpret_cast<uintptr_t>(idx_out) & 3u) || (reinterpret_cast<uintptr_t>(status_out) & 3u)) return PVT_EINVAL;
  if (G > kNoAllocMaxGroups || select_layout(G).bytes > kNoAllocScratchBytes) return PVT_ETOOLARGE;

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  void* ws = nullptr;
  cudaError_t e = scratch_for_current_device(&ws);
  // the array keeps whatever the previous call left: the status word must start at zero
  // (launch_select clears the selection state and the histograms itself)
  if (e == cudaSuccess) e = cudaMemsetAsync(ws, 0, sizeof(uint32_t), stream);
  if (e == cudaSuccess) e = launch_select(*layer, G, k, idx_out, ws, device_sm_count(), stream);
  if (e == cudaSuccess && status_out)
    e = cudaMemcpyAsync(status_out, ws, sizeof(uint32_t), cudaMemcpyDeviceToDevice, stream);
  if (e != cudaSuccess) {
    record_cuda_error(e);
    return PVT_ECUDA;
  }
  return PVT_OK;
}
