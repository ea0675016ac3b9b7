// adadim_score_select_static: the scorer for callers that must not allocate device memory.
//
// adadim_score_select needs a caller-provided workspace.  Some callers cannot produce one:
// code running where cudaMalloc is forbidden or unaffordable - inside a region whose memory
// budget is frozen (a serving process that has handed all free memory to its cache), in a
// plugin that is given tensors but no allocator, or on a latency path where an allocation's
// implicit device synchronisation is unacceptable.  For them this file reserves a fixed
// scratch array in the library's own device image and runs the same kernels on it.
//
// The array exists once per GPU that loads the library, from load until the process exits,
// whether or not this entry point is ever called.
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
  // the same argument rules as adadim_score_select
  if (bits != 3 && bits != 4) return ADADIM_ERR_PARAM;
  if (group != 32 && group != 64 && group != 128) return ADADIM_ERR_PARAM;
  if (out <= 0 || in <= 0 || ldw < in) return ADADIM_ERR_SHAPE;
  if (W == nullptr || H == nullptr || err == nullptr || chosen == nullptr) return ADADIM_ERR_NULL;
  if (wdtype != ADADIM_F16 && wdtype != ADADIM_F32) return ADADIM_ERR_DTYPE;
  if (!aligned16(W) || (ldw * (wdtype == ADADIM_F16 ? 2 : 4)) % 16 != 0 || !aligned16(H)) return ADADIM_ERR_ALIGN;
  if (in % 64 != 0 || out % 128 != 0) return ADADIM_ERR_SHAPE;
  if (q_oc == nullptr && q_ic == nullptr) return ADADIM_ERR_NULL;
  const adadim_qtensor* qs[2] = {q_oc, q_ic};
  for (int d = 0; d < 2; ++d) {
    if (qs[d] == nullptr) continue;
    if (qs[d]->codes == nullptr || qs[d]->scales == nullptr || qs[d]->zeros == nullptr) return ADADIM_ERR_NULL;
    if (!aligned16(qs[d]->codes) || !aligned16(qs[d]->scales) || !aligned16(qs[d]->zeros)) return ADADIM_ERR_ALIGN;
    if ((d == 0 ? in : out) % group != 0) return ADADIM_ERR_SHAPE;
  }
  // the size limit: the layer's scoring workspace must fit the built-in array
  if (score_workspace_bytes(out, in) > ADADIM_STATIC_SCRATCH_BYTES) return ADADIM_ERR_WORKSPACE;
  void* scratch = nullptr;
  int rc = scratch_address(&scratch);
  if (rc != ADADIM_OK) return rc;
  if (status_dev != nullptr && cudaMemsetAsync(status_dev, 0, sizeof(int), st) != cudaSuccess) return ADADIM_ERR_CUDA;
  // Nothing in the scratch has to start at zero: every region the kernels read (the weight
  // differences, the two halves of H, the per-tile partial sums) is fully rewritten by this
  // call before it is read, so whatever an earlier call left behind is never observed.
  return score_launch(W, wdtype, out, in, ldw, H, bits, group, q_oc, q_ic, err, chosen, status_dev, scratch, st);
}

}  // extern "C"
