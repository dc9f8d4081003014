// as_ssm_forward_static: the layer forward for callers that are not allowed to allocate device memory.
//
// Who needs it: code that runs as a guest inside a host program which has handed out all device memory
// up front and forbids (or cannot tolerate) cudaMalloc from guest code - for example a plug-in inside an
// inference server whose memory budget is frozen at start-up, or a control loop where cudaMalloc's implicit
// device-wide synchronisation would break the latency budget.  Such callers can pass input and output
// buffers they were given, but have nowhere to get the scratch buffer as_ssm_forward asks for.
//
// Here the scratch lives in a fixed array inside the library's own device image.  Consequences a user
// should know:
//   * Every GPU context that loads this library holds AS_STATIC_SCRATCH_BYTES of device memory for the
//     array until the process exits, whether or not this entry point is ever called.
//   * Shapes whose forward scratch (as_workspace_bytes, fwd_bytes) exceeds the array are rejected with
//     AS_ERR_LIMIT; nothing is launched.
//   * The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that
//     device current).  That is a synchronous runtime call: make the first call per device during set-up,
//     before any stream capture begins.  Later calls only enqueue work.
//   * All calls on a device share the one array, and it keeps whatever the previous call left in it.  The
//     entry point clears the words that must start at zero itself.  Two calls whose kernels can overlap on
//     the GPU (different streams, no ordering between them) race on the array and corrupt each other.
//   * No cudaMalloc, cudaFree or other allocating routine is called, by this entry point or by anything it
//     launches.
#include "as_internal.cuh"

namespace {

static __device__ __align__(256) unsigned char g_static_scratch[AS_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
// Device address of g_static_scratch per device ordinal, in the device's primary context (the context the CUDA runtime
// API uses; a caller that makes its own driver-API contexts current is not supported by this entry point).  Atomic so
// that host threads may make their first calls concurrently: both would store the same address.
std::atomic<void*> g_scratch_addr[kMaxDevices] = {};

// The name g_static_scratch is, in host code, only a handle for the runtime: it is not a device address and
// must never be passed to a kernel.  The address a kernel can use comes from cudaGetSymbolAddress, queried
// once per device while that device is current.
int scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return AS_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return AS_ERR_LIMIT;
  void* p = g_scratch_addr[dev].load(std::memory_order_acquire);
  if (!p) {
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return AS_ERR_CUDA;
    g_scratch_addr[dev].store(p, std::memory_order_release);
  }
  *out = p;
  return AS_OK;
}

}  // namespace

// The status word of as_ssm_forward_static lives at the head of the static array: as_check_status(NULL, stream)
// reads it through this.
int as::static_scratch_address(void** out) { return scratch_for_current_device(out); }

extern "C" int as_ssm_forward_static(const as_shape_t* shape, const as_params_t* params, const void* x, void* y,
                                     void* stream) {
  size_t need = 0;
  int e = as_workspace_bytes(shape, shape ? shape->seqlen : 1, &need, nullptr);
  if (e) return e;
  if (need > (size_t)AS_STATIC_SCRATCH_BYTES) return AS_ERR_LIMIT;
  void* scratch = nullptr;
  e = scratch_for_current_device(&scratch);
  if (e) return e;
  // as_ssm_forward zeroes the status word at the head of the scratch and overwrites every other region it reads
  return as_ssm_forward(shape, params, x, y, scratch, (size_t)AS_STATIC_SCRATCH_BYTES, stream);
}
