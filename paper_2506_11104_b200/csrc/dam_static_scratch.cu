// dam_build_masks_static: stage 1 for callers that cannot allocate device memory.
//
// Some users of this library run with a frozen device-memory plan: an inference server that handed the
// whole GPU to its own pool at start-up, or a latency-critical loop that must not call cudaMalloc (which
// may synchronise the device and can fail once the pool owns everything).  Such callers have nowhere to
// get the scratch buffer dam_build_masks asks for.  This entry point takes the scratch from a fixed
// array that is part of the library image instead, so the call allocates nothing at all.
//
// The array is file-scope device memory of kStaticScratchBytes; every GPU that loads the library holds
// it until the process exits.  In host code the array's name is only a stand-in for the symbol, not a
// device address, so its address is looked up with cudaGetSymbolAddress, once per device, with that
// device current, and that pointer is what the kernels receive.
#include "dam_internal.cuh"

namespace {

constexpr size_t kStaticScratchBytes = 8u << 20;   // 8 MiB: covers every shape up to 131072 tokens x 32 heads, PCL 4096
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// device pointer of g_static_scratch per device ordinal, filled on first use on that device
void* g_scratch_ptr[kMaxDevices] = {nullptr};

dam_status_t static_scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return DAM_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return DAM_ERR_UNSUPPORTED;
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p) return DAM_ERR_CUDA;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return DAM_OK;
}

}  // namespace

extern "C" dam_status_t dam_build_masks_static(const void* Q, const void* K, const dam_shape_t* shape,
                                               const dam_rule_t* rule, void* mask, size_t mask_capacity,
                                               void* stream) {
  size_t need = 0;
  dam_status_t st = dam_mask_sizes(shape, rule, 1, nullptr, &need, nullptr);
  if (st != DAM_OK) return st;
  if (need > kStaticScratchBytes) return DAM_ERR_BUFFER_TOO_SMALL;   // shape too large for the built-in scratch
  void* scratch = nullptr;
  if ((st = static_scratch_for_current_device(&scratch)) != DAM_OK) return st;
  // dam_build_masks clears every counter it accumulates into, so the previous call's contents do not matter
  return dam_build_masks(Q, K, shape, rule, mask, mask_capacity, scratch, kStaticScratchBytes, nullptr, stream);
}

extern "C" size_t dam_static_scratch_bytes(void) { return kStaticScratchBytes; }
