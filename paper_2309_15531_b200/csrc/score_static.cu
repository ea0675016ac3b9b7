// adadim_score_select_static: the scorer for callers that must not allocate device memory.
//
// adadim_score_select needs a caller-provided workspace.  Some callers cannot produce one:
// code running where cudaMalloc is forbidden or unaffordable - inside a region whose memory
// budget is frozen (a serving process that has handed all free memory to its cache), in a
// plugin that is given tensors but no allocator, or on a latency path where an allocation's
// implicit device synchronisation is unacceptable.  For them this file reserves a fixed
// scratch array in the library's own device image and runs the same kernels on it.
//
// The array exists once per GPU that uses the library and stays until the process exits.  With
// the CUDA runtime's lazy module loading it becomes resident on a device when its address is
// first looked up there, i.e. at the first call of this entry point on that device.
#include <mutex>

#include "common.cuh"

namespace adadim {
size_t score_workspace_bytes(int64_t out, int64_t in);
int score_launch(const void* W, int wdtype, int64_t out, int64_t in, int64_t ldw, const float* H, int bits, int group,
                 const adadim_qtensor* q_oc, const adadim_qtensor* q_ic, double* err, int* chosen, int* status_dev,
                 void* workspace, cudaStream_t st);
}  // namespace adadim

namespace {

// File-scope device array.  In host code this name is only a handle for the runtime: it is not
// a device address, so it is never passed to a kernel; the address comes from
// cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_score_scratch[ADADIM_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device (looked up once per device).
int scratch_address(void** out_ptr) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ADADIM_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (g_scratch_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_score_scratch) != cudaSuccess || p == nullptr) return ADADIM_ERR_CUDA;
    g_scratch_ptr[dev] = p;
  }
  *out_ptr = g_scratch_ptr[dev];
  return ADADIM_OK;
}

}  // namespace

extern "C" {

size_t adadim_static_scratch_bytes(void) { return ADADIM_STATIC_SCRATCH_BYTES; }

int adadim_score_select_static(const void* W, int wdtype, int64_t out, int64_t in, int64_t ldw, const float* H,
                               int bits, int group, const adadim_qtensor* q_oc, const adadim_qtensor* q_ic,
                               double* err, int* chosen, int* status_dev, void* cuda_stream) {
  using namespace adadim;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // the same argument rules as adadim_score_select, checked by the same function
  int rc = check_score_args(W, wdtype, out, in, ldw, H, bits, group, q_oc, q_ic, err, chosen);
  if (rc != ADADIM_OK) return rc;
  // the size limit: the layer's scoring workspace must fit the built-in array
  if (score_workspace_bytes(out, in) > ADADIM_STATIC_SCRATCH_BYTES) return ADADIM_ERR_WORKSPACE;
  void* scratch = nullptr;
  rc = scratch_address(&scratch);
  if (rc != ADADIM_OK) return rc;
  // Nothing in the scratch has to start at zero: every region the kernels read (the weight
  // differences and the per-tile partial sums) is fully rewritten by this call before it is
  // read, so whatever an earlier call left behind is never observed.
  return score_launch(W, wdtype, out, in, ldw, H, bits, group, q_oc, q_ic, err, chosen, status_dev, scratch, st);
}

}  // extern "C"
