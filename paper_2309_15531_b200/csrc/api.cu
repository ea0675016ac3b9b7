// extern "C" entry points: argument validation on the host, then the kernel launchers.
#include "common.cuh"

namespace adadim {
int rtn_launch(const void* W, int wdtype, int64_t out, int64_t in, int64_t ldw, int bits, int group, int dim,
               const adadim_qtensor& qoc, const adadim_qtensor& qic, cudaStream_t st);
int unpack_launch(const uint32_t* codes, int64_t out, int64_t in, int bits, uint8_t* dst, cudaStream_t st);
int hessian_bf16_launch(const void* X, int64_t n_tokens, int64_t in, int64_t ldx, float* H, int* status_dev,
                        cudaStream_t st);
int hessian_f32_launch(const float* X, int64_t n_tokens, int64_t in, int64_t ldx, float* H, cudaStream_t st);
size_t hessian_f32_tc_workspace_bytes(int64_t n_tokens, int64_t in);
int hessian_f32_tc_launch(const float* X, int64_t n_tokens, int64_t in, int64_t ldx, float* H, int* status_dev,
                          void* workspace, cudaStream_t st);
size_t score_workspace_bytes(int64_t out, int64_t in);
int score_launch(const void* W, int wdtype, int64_t out, int64_t in, int64_t ldw, const float* H, int bits, int group,
                 const adadim_qtensor* q_oc, const adadim_qtensor* q_ic, double* err, int* chosen, int* status_dev,
                 void* workspace, cudaStream_t st);
size_t factor_workspace_bytes(int64_t n);
int factor_launch(const float* H, int64_t n, double percdamp, double* U, int* status_dev, void* workspace,
                  cudaStream_t st, const int* perm);
size_t gptq_workspace_bytes(int64_t rows, int64_t in);
struct GptqLayer {
  const void* W;
  int64_t out, ldw;
  const adadim_qtensor* q_oc;
  const adadim_qtensor* q_ic;
  int dim;
  const int* chosen;
  double* loss;
};
int gptq_launch(const GptqLayer* layers, int n_layers, int wdtype, int64_t in, const float* H, const double* U,
                int bits, int group, double percdamp, int* status_dev, void* workspace, cudaStream_t st, bool reorder,
                int* perm_out);

size_t gemv_workspace_bytes(int64_t out, int64_t in, int group);
int gemv_launch(const adadim_qtensor& q, int64_t out, int64_t in, int bits, int group, const void* x, void* y,
                void* workspace, cudaStream_t st);

namespace {

int check_weight(const void* W, int wdtype, int64_t out, int64_t in, int64_t ldw) {
  if (W == nullptr) return ADADIM_ERR_NULL;
  if (wdtype != ADADIM_F16 && wdtype != ADADIM_F32) return ADADIM_ERR_DTYPE;
  if (out < 0 || in < 0 || ldw < in) return ADADIM_ERR_SHAPE;
  const int64_t esz = wdtype == ADADIM_F16 ? 2 : 4;
  if (!aligned16(W) || (ldw * esz) % 16 != 0) return ADADIM_ERR_ALIGN;
  return ADADIM_OK;
}

// every entry point takes groups 32, 64, 128 and 256; at 256 GPTQ needs whole pairs of its 128-row
// slabs and 128-column blocks (out and in multiples of 256)
int check_quant_params(int bits, int group, bool allow_256) {
  if (bits != 2 && bits != 3 && bits != 4 && bits != 8) return ADADIM_ERR_PARAM;
  if (group != 32 && group != 64 && group != 128 && !(allow_256 && group == 256)) return ADADIM_ERR_PARAM;
  return ADADIM_OK;
}

int check_qtensor(const adadim_qtensor* q) {
  if (q == nullptr || q->codes == nullptr || q->scales == nullptr || q->zeros == nullptr) return ADADIM_ERR_NULL;
  if (!aligned16(q->codes) || !aligned16(q->scales) || !aligned16(q->zeros)) return ADADIM_ERR_ALIGN;
  return ADADIM_OK;
}

}  // namespace

int check_score_args(const void* W, int wdtype, int64_t out, int64_t in, int64_t ldw, const float* H, int bits,
                     int group, const adadim_qtensor* q_oc, const adadim_qtensor* q_ic, const double* err,
                     const int* chosen) {
  int rc = check_quant_params(bits, group, true);
  if (rc != ADADIM_OK) return rc;
  if (out <= 0 || in <= 0) return ADADIM_ERR_SHAPE;
  rc = check_weight(W, wdtype, out, in, ldw);
  if (rc != ADADIM_OK) return rc;
  if (in % 64 != 0 || out % 128 != 0) return ADADIM_ERR_SHAPE;
  if (q_oc == nullptr && q_ic == nullptr) return ADADIM_ERR_NULL;
  if (q_oc != nullptr && in % group != 0) return ADADIM_ERR_SHAPE;
  if (q_ic != nullptr && out % group != 0) return ADADIM_ERR_SHAPE;
  if (q_oc != nullptr && (rc = check_qtensor(q_oc)) != ADADIM_OK) return rc;
  if (q_ic != nullptr && (rc = check_qtensor(q_ic)) != ADADIM_OK) return rc;
  if (H == nullptr || err == nullptr || chosen == nullptr) return ADADIM_ERR_NULL;
  if (!aligned16(H)) return ADADIM_ERR_ALIGN;
  return ADADIM_OK;
}

}  // namespace adadim

using namespace adadim;

extern "C" {

int adadim_version(void) { return 100; }

const char* adadim_strerror(int status) {
  switch (status) {
    case ADADIM_OK: return "ok";
    case ADADIM_ERR_NULL: return "a required pointer is NULL";
    case ADADIM_ERR_SHAPE: return "a size is negative or violates a divisibility rule";
    case ADADIM_ERR_DTYPE: return "unsupported element type";
    case ADADIM_ERR_PARAM: return "bits, group, dim, percdamp or blocksize out of range";
    case ADADIM_ERR_ALIGN: return "pointer or leading dimension not suitably aligned";
    case ADADIM_ERR_WORKSPACE: return "workspace too small";
    case ADADIM_ERR_NOT_PD: return "damped Hessian is not positive definite";
    case ADADIM_ERR_NUMERIC: return "a reconstruction error is NaN";
    case ADADIM_ERR_TIMEOUT: return "an internal device-side wait exceeded its limit";
    case ADADIM_ERR_CUDA: return "a CUDA call failed";
    default: return "unknown status";
  }
}

size_t adadim_workspace_bytes(int kind, int64_t out, int64_t in, int bits, int group) {
  (void)bits;
  if (out < 0 || in < 0) return 0;
  switch (kind) {
    case ADADIM_WS_HESSIAN: return out > 0 ? hessian_f32_tc_workspace_bytes(out, in) : 0;   // out = tokens of an fp32 chunk
    case ADADIM_WS_GPTQ: return gptq_workspace_bytes(2 * out, in);
    case ADADIM_WS_GPTQ_ROWS: return gptq_workspace_bytes(out, in);
    case ADADIM_WS_GEMV: return group > 0 ? gemv_workspace_bytes(out, in, group) : 0;
    case ADADIM_WS_SCORE: return score_workspace_bytes(out, in);
    case ADADIM_WS_FACTOR: return factor_workspace_bytes(in);
    default: return 0;
  }
}

int adadim_hessian_accumulate(const void* X, int xdtype, int64_t n_tokens, int64_t in, int64_t ldx, float* H,
                              int64_t* n_seen, int* status_dev, void* workspace, size_t workspace_bytes,
                              void* cuda_stream) {
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (xdtype != ADADIM_BF16 && xdtype != ADADIM_F32) return ADADIM_ERR_DTYPE;
  if (n_tokens < 0 || in < 0 || ldx < in || in % 8 != 0) return ADADIM_ERR_SHAPE;
  if (n_tokens > 0x7fffffff || in > (1 << 20)) return ADADIM_ERR_SHAPE;
  if (in == 0) return ADADIM_OK;
  if (H == nullptr) return ADADIM_ERR_NULL;
  if (!aligned16(H)) return ADADIM_ERR_ALIGN;
  if (n_tokens == 0) return ADADIM_OK;
  int rc = ADADIM_OK;
  if (X == nullptr) return ADADIM_ERR_NULL;
  const int64_t esz = xdtype == ADADIM_BF16 ? 2 : 4;
  if (!aligned16(X) || (ldx * esz) % 16 != 0) return ADADIM_ERR_ALIGN;
  if (xdtype == ADADIM_BF16) {
    rc = hessian_bf16_launch(X, n_tokens, in, ldx, H, status_dev, st);
  } else if (workspace != nullptr && aligned256(workspace) &&
             workspace_bytes >= hessian_f32_tc_workspace_bytes(n_tokens, in)) {
    rc = hessian_f32_tc_launch(static_cast<const float*>(X), n_tokens, in, ldx, H, status_dev, workspace, st);
  } else {
    rc = hessian_f32_launch(static_cast<const float*>(X), n_tokens, in, ldx, H, st);
  }
  if (rc == ADADIM_OK && n_seen != nullptr) *n_seen += n_tokens;
  return rc;
}

int adadim_quantize_rtn(const void* W, int wdtype, int64_t out, int64_t in, int64_t ldw, int bits, int group, int dim,
                        const adadim_qtensor* q_oc, const adadim_qtensor* q_ic, void* cuda_stream) {
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int rc = check_quant_params(bits, group, true);
  if (rc != ADADIM_OK) return rc;
  if (dim != ADADIM_DIM_OC && dim != ADADIM_DIM_IC && dim != ADADIM_DIM_BOTH) return ADADIM_ERR_PARAM;
  if (out < 0 || in < 0) return ADADIM_ERR_SHAPE;
  if (out == 0 || in == 0) return ADADIM_OK;
  rc = check_weight(W, wdtype, out, in, ldw);
  if (rc != ADADIM_OK) return rc;
  if (in % 32 != 0) return ADADIM_ERR_SHAPE;
  const bool oc = dim != ADADIM_DIM_IC, ic = dim != ADADIM_DIM_OC;
  if (oc && in % group != 0) return ADADIM_ERR_SHAPE;
  if (ic && out % group != 0) return ADADIM_ERR_SHAPE;
  if (oc && (rc = check_qtensor(q_oc)) != ADADIM_OK) return rc;
  if (ic && (rc = check_qtensor(q_ic)) != ADADIM_OK) return rc;
  adadim_qtensor none = {nullptr, nullptr, nullptr};
  return rtn_launch(W, wdtype, out, in, ldw, bits, group, dim, oc ? *q_oc : none, ic ? *q_ic : none, st);
}

int adadim_cholesky_inverse_factor(const float* H, int64_t in, double percdamp, double* U, int* status_dev,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream) {
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (in < 0 || in % 64 != 0) return ADADIM_ERR_SHAPE;
  if (!(percdamp >= 0.0) || !(percdamp < 1e6)) return ADADIM_ERR_PARAM;
  if (in == 0) return ADADIM_OK;
  if (H == nullptr || U == nullptr || workspace == nullptr) return ADADIM_ERR_NULL;
  if (!aligned16(H) || !aligned16(U) || !aligned256(workspace)) return ADADIM_ERR_ALIGN;
  if (workspace_bytes < factor_workspace_bytes(in)) return ADADIM_ERR_WORKSPACE;
  return factor_launch(H, in, percdamp, U, status_dev, workspace, st, nullptr);
}

int adadim_quantize_gptq(const void* W, int wdtype, int64_t out, int64_t in, int64_t ldw, const float* H,
                         const double* U, int bits, int group, int dim, double percdamp, int blocksize,
                         const adadim_qtensor* q_oc, const adadim_qtensor* q_ic, double* gptq_loss, int* status_dev,
                         void* workspace, size_t workspace_bytes, void* cuda_stream) {
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int rc = check_quant_params(bits, group, true);
  if (rc != ADADIM_OK) return rc;
  if (dim != ADADIM_DIM_OC && dim != ADADIM_DIM_IC && dim != ADADIM_DIM_BOTH) return ADADIM_ERR_PARAM;
  if (blocksize != 128) return ADADIM_ERR_PARAM;
  if (!(percdamp >= 0.0) || !(percdamp < 1e6)) return ADADIM_ERR_PARAM;
  if (out < 0 || in < 0) return ADADIM_ERR_SHAPE;
  if (out == 0 || in == 0) return ADADIM_OK;
  rc = check_weight(W, wdtype, out, in, ldw);
  if (rc != ADADIM_OK) return rc;
  if (in % 128 != 0 || out % 128 != 0) return ADADIM_ERR_SHAPE;
  if (group == 256 && (in % 256 != 0 || out % 256 != 0)) return ADADIM_ERR_SHAPE;
  if (H == nullptr || workspace == nullptr) return ADADIM_ERR_NULL;
  if (!aligned16(H) || (U != nullptr && !aligned16(U)) || !aligned256(workspace)) return ADADIM_ERR_ALIGN;
  const bool oc = dim != ADADIM_DIM_IC, ic = dim != ADADIM_DIM_OC;
  if (oc && (rc = check_qtensor(q_oc)) != ADADIM_OK) return rc;
  if (ic && (rc = check_qtensor(q_ic)) != ADADIM_OK) return rc;
  if (workspace_bytes < gptq_workspace_bytes(2 * out, in)) return ADADIM_ERR_WORKSPACE;
  const GptqLayer layer = {W, out, ldw, q_oc, q_ic, dim, nullptr, gptq_loss};
  return gptq_launch(&layer, 1, wdtype, in, H, U, bits, group, percdamp, status_dev, workspace, st, false, nullptr);
}

int adadim_quantize_gptq_batched(const adadim_gptq_layer* layers, int n_layers, int wdtype, int64_t in, const float* H,
                                 const double* U, int bits, int group, double percdamp, int blocksize, int* status_dev,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream) {
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int rc = check_quant_params(bits, group, true);
  if (rc != ADADIM_OK) return rc;
  if (blocksize != 128) return ADADIM_ERR_PARAM;
  if (!(percdamp >= 0.0) || !(percdamp < 1e6)) return ADADIM_ERR_PARAM;
  if (n_layers < 0 || n_layers > ADADIM_MAX_BATCHED_LAYERS || in < 0) return ADADIM_ERR_SHAPE;
  if (n_layers == 0 || in == 0) return ADADIM_OK;
  if (layers == nullptr || H == nullptr || workspace == nullptr) return ADADIM_ERR_NULL;
  if (in % 128 != 0 || (group == 256 && in % 256 != 0)) return ADADIM_ERR_SHAPE;
  if (!aligned16(H) || (U != nullptr && !aligned16(U)) || !aligned256(workspace)) return ADADIM_ERR_ALIGN;
  GptqLayer ls[ADADIM_MAX_BATCHED_LAYERS];
  int64_t rows = 0;
  int copies = 0;
  for (int l = 0; l < n_layers; ++l) {
    const adadim_gptq_layer& y = layers[l];
    if (y.out <= 0 || y.out % 128 != 0 || (group == 256 && y.out % 256 != 0)) return ADADIM_ERR_SHAPE;
    rc = check_weight(y.W, wdtype, y.out, in, y.ldw);
    if (rc != ADADIM_OK) return rc;
    if (y.dim != ADADIM_DIM_OC && y.dim != ADADIM_DIM_IC && y.dim != ADADIM_DIM_BOTH && y.dim != ADADIM_DIM_CHOSEN)
      return ADADIM_ERR_PARAM;
    if (y.dim == ADADIM_DIM_CHOSEN && y.chosen == nullptr) return ADADIM_ERR_NULL;
    const bool oc = y.dim != ADADIM_DIM_IC, ic = y.dim != ADADIM_DIM_OC;
    if (oc && (rc = check_qtensor(y.q_oc)) != ADADIM_OK) return rc;
    if (ic && (rc = check_qtensor(y.q_ic)) != ADADIM_OK) return rc;
    const int nd = y.dim == ADADIM_DIM_BOTH ? 2 : 1;
    copies += nd;
    rows += nd * y.out;
    ls[l] = {y.W, y.out, y.ldw, y.q_oc, y.q_ic, y.dim, y.chosen, y.gptq_loss};
  }
  if (copies > ADADIM_MAX_BATCHED_LAYERS) return ADADIM_ERR_SHAPE;
  if (workspace_bytes < gptq_workspace_bytes(rows, in)) return ADADIM_ERR_WORKSPACE;
  return gptq_launch(ls, n_layers, wdtype, in, H, U, bits, group, percdamp, status_dev, workspace, st, false, nullptr);
}

int adadim_quantize_gptq_reordered(const void* W, int wdtype, int64_t out, int64_t in, int64_t ldw, const float* H,
                                   int bits, int group, int dim, double percdamp, int blocksize,
                                   const adadim_qtensor* q_oc, const adadim_qtensor* q_ic, double* gptq_loss,
                                   int32_t* perm_out, int* status_dev, void* workspace, size_t workspace_bytes,
                                   void* cuda_stream) {
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int rc = check_quant_params(bits, group, true);
  if (rc != ADADIM_OK) return rc;
  if (dim != ADADIM_DIM_OC && dim != ADADIM_DIM_IC && dim != ADADIM_DIM_BOTH) return ADADIM_ERR_PARAM;
  if (blocksize != 128) return ADADIM_ERR_PARAM;
  if (!(percdamp >= 0.0) || !(percdamp < 1e6)) return ADADIM_ERR_PARAM;
  if (out < 0 || in < 0) return ADADIM_ERR_SHAPE;
  if (out == 0 || in == 0) return ADADIM_OK;
  rc = check_weight(W, wdtype, out, in, ldw);
  if (rc != ADADIM_OK) return rc;
  if (in % 128 != 0 || out % 128 != 0) return ADADIM_ERR_SHAPE;
  if (group == 256 && (in % 256 != 0 || out % 256 != 0)) return ADADIM_ERR_SHAPE;
  if (H == nullptr || workspace == nullptr) return ADADIM_ERR_NULL;
  if (!aligned16(H) || !aligned256(workspace)) return ADADIM_ERR_ALIGN;
  const bool oc = dim != ADADIM_DIM_IC, ic = dim != ADADIM_DIM_OC;
  if (oc && (rc = check_qtensor(q_oc)) != ADADIM_OK) return rc;
  if (ic && (rc = check_qtensor(q_ic)) != ADADIM_OK) return rc;
  if (workspace_bytes < gptq_workspace_bytes(2 * out, in)) return ADADIM_ERR_WORKSPACE;
  const GptqLayer layer = {W, out, ldw, q_oc, q_ic, dim, nullptr, gptq_loss};
  return gptq_launch(&layer, 1, wdtype, in, H, nullptr, bits, group, percdamp, status_dev, workspace, st, true,
                     perm_out);
}

int adadim_score_select(const void* W, int wdtype, int64_t out, int64_t in, int64_t ldw, const float* H, int bits,
                        int group, const adadim_qtensor* q_oc, const adadim_qtensor* q_ic, double* err, int* chosen,
                        int* status_dev, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int rc = check_score_args(W, wdtype, out, in, ldw, H, bits, group, q_oc, q_ic, err, chosen);
  if (rc != ADADIM_OK) return rc;
  if (workspace == nullptr) return ADADIM_ERR_NULL;
  if (!aligned256(workspace)) return ADADIM_ERR_ALIGN;
  if (workspace_bytes < score_workspace_bytes(out, in)) return ADADIM_ERR_WORKSPACE;
  return score_launch(W, wdtype, out, in, ldw, H, bits, group, q_oc, q_ic, err, chosen, status_dev, workspace, st);
}

int adadim_dequant_gemv(const adadim_qtensor* q, int dim, int64_t out, int64_t in, int bits, int group, const void* x,
                        void* y, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (bits != 3 && bits != 4) return ADADIM_ERR_PARAM;
  if (dim != ADADIM_DIM_IC) return ADADIM_ERR_PARAM;
  if (group < 16 || group % 16 != 0) return ADADIM_ERR_PARAM;
  if (out < 0 || in < 0) return ADADIM_ERR_SHAPE;
  if (out == 0 || in == 0) return ADADIM_OK;
  if (out % group != 0 || in % 128 != 0) return ADADIM_ERR_SHAPE;
  int rc = check_qtensor(q);
  if (rc != ADADIM_OK) return rc;
  if (x == nullptr || y == nullptr || workspace == nullptr) return ADADIM_ERR_NULL;
  if (!aligned16(x) || !aligned256(workspace) || (reinterpret_cast<uintptr_t>(y) & 1u) != 0) return ADADIM_ERR_ALIGN;
  if (workspace_bytes < gemv_workspace_bytes(out, in, group)) return ADADIM_ERR_WORKSPACE;
  return gemv_launch(*q, out, in, bits, group, x, y, workspace, static_cast<cudaStream_t>(cuda_stream));
}

int adadim_unpack_codes(const uint32_t* codes, int64_t out, int64_t in, int bits, uint8_t* dst, void* cuda_stream) {
  if (bits != 2 && bits != 3 && bits != 4 && bits != 8) return ADADIM_ERR_PARAM;
  if (out < 0 || in < 0 || in % 32 != 0) return ADADIM_ERR_SHAPE;
  if (out == 0 || in == 0) return ADADIM_OK;
  if (codes == nullptr || dst == nullptr) return ADADIM_ERR_NULL;
  if (!aligned16(dst)) return ADADIM_ERR_ALIGN;
  return unpack_launch(codes, out, in, bits, dst, static_cast<cudaStream_t>(cuda_stream));
}

}  // extern "C"
