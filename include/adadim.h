/*
 * adadim.h - C ABI of the AdaDim layer-quantization library for NVIDIA B200 (sm_100a).
 *
 * The library quantizes one linear layer's weight W[out,in] to b-bit group-wise asymmetric
 * integers under both grouping dimensions of the paper "Rethinking Channel Dimensions to
 * Isolate Outliers for Low-bit Weight Quantization of LLMs" (arxiv 2309.15531): groups of g
 * consecutive weights inside an output channel (a row of W, "per-OC", Section 2.1) and
 * inside an input channel (a column of W, "per-IC", Section 3.2), scores both by the
 * layer-output reconstruction error of Section 3.3, Eq. 1, and selects one.
 *
 * Conventions that hold for every entry point
 *   - All matrices are row-major.  W[o,i] is at W + o*ldw + i; X[t,i] (token t) at X + t*ldx + i.
 *   - Unless an argument is marked "host", every pointer is a DEVICE pointer owned by the
 *     caller.  The library allocates no device memory and keeps no state between calls
 *     (the one exception, a built-in scratch array, is described at
 *     adadim_score_select_static); inputs are never modified.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*, NULL = default
 *     stream).  No entry point synchronizes; results are valid once the stream has run.
 *     adadim_cholesky_inverse_factor and the GPTQ entry points overlap parts of their work
 *     on streams of their own (two; four in the factor), which they create on entry and release
 *     before returning;
 *     that work starts after everything already enqueued on `cuda_stream` and is joined back
 *     into it, so to the caller these calls are ordered on `cuda_stream` like the others.
 *   - The return value is an adadim_status.  Argument errors are found on the host before
 *     anything is launched.  Conditions only the device can see (a non-positive Cholesky
 *     pivot, a NaN error, a wait that ran out) are written to the caller's `status_dev` word;
 *     kernels never trap.  The word is STICKY: the caller sets it to ADADIM_OK (0) once, may
 *     pass the same word to any sequence of calls, and reads it when convenient; a call only
 *     ever changes it from ADADIM_OK to the first condition it meets and never clears it, so
 *     an early call's error survives the later calls.
 *   - Non-finite weights or activations give unspecified codes (no error is raised).
 */
#ifndef ADADIM_H_
#define ADADIM_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define ADADIM_API __attribute__((visibility("default")))
#else
#define ADADIM_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  ADADIM_OK = 0,
  ADADIM_ERR_NULL = 1,       /* a required pointer is NULL                                  */
  ADADIM_ERR_SHAPE = 2,      /* a size is negative or violates a divisibility rule          */
  ADADIM_ERR_DTYPE = 3,      /* unknown element type for this argument                      */
  ADADIM_ERR_PARAM = 4,      /* bits / group / dim / percdamp / blocksize out of range      */
  ADADIM_ERR_ALIGN = 5,      /* pointer or leading dimension not 16-byte aligned            */
  ADADIM_ERR_WORKSPACE = 6,  /* workspace smaller than adadim_workspace_bytes() says        */
  ADADIM_ERR_NOT_PD = 7,     /* (device) damped Hessian is not positive definite            */
  ADADIM_ERR_NUMERIC = 8,    /* (device) a reconstruction error is NaN                      */
  ADADIM_ERR_TIMEOUT = 9,    /* (device) an internal wait exceeded its limit                */
  ADADIM_ERR_CUDA = 10       /* a CUDA runtime / driver call failed                         */
} adadim_status;

typedef enum { ADADIM_F32 = 0, ADADIM_F16 = 1, ADADIM_BF16 = 2 } adadim_dtype;
/* ADADIM_DIM_CHOSEN (batched GPTQ only): the dimension is read from a device word at run time. */
typedef enum { ADADIM_DIM_OC = 0, ADADIM_DIM_IC = 1, ADADIM_DIM_BOTH = 2, ADADIM_DIM_CHOSEN = 3 } adadim_dim;
/* ADADIM_WS_GPTQ: one layer [out][in] in up to both dimensions.  ADADIM_WS_GPTQ_ROWS: `out` is the
 * total number of working rows of a batched call (sum over its layers of out, twice for a layer
 * quantized in both dimensions). */
typedef enum { ADADIM_WS_HESSIAN = 0, ADADIM_WS_GPTQ = 1, ADADIM_WS_SCORE = 2,
               ADADIM_WS_FACTOR = 3, ADADIM_WS_GPTQ_ROWS = 4, ADADIM_WS_GEMV = 5 } adadim_ws_kind;

/*
 * One quantized tensor (device pointers, caller-owned).
 *   codes  [out][in*bits/32] uint32.  Code k of row o occupies bits [k*bits, (k+1)*bits) of
 *          that row's little-endian stream of 32-bit words; the layout is the same for both
 *          grouping dimensions.  (The paper fixes no packed format; its storage accounting,
 *          Appendix C, counts bits only.)
 *   scales fp16 bit patterns.  per-OC: [out][in/g];  per-IC: [out/g][in]   (Section 3.2).
 *   zeros  fp16 bit patterns holding the integer zero point 0..2^bits-1, same shape.
 * Dequantized weight: q = scale * (code - zero).
 */
typedef struct {
  uint32_t* codes;
  uint16_t* scales;
  uint16_t* zeros;
} adadim_qtensor;

/*
 * Calibration Hessian  H += 2 * X^T X  over one chunk of tokens (Section 4.4: the inverse
 * Hessian GPTQ uses is "formed by activations"; Section 2.2).
 *   X        [n_tokens][in], xdtype ADADIM_BF16 or ADADIM_F32, both on the tcgen05 tensor cores: an
 *            fp32 chunk is split exactly into three bf16 pieces in the workspace (without a
 *            workspace of that size a plain multiply-add kernel is used instead).
 *            ldx in elements; X and ldx*sizeof(elem) must be 16-byte aligned.
 *   H        [in][in] fp32, in/out, symmetric on entry: the caller zeroes it before the first
 *            chunk and passes it back unchanged for the next ones.  Both triangles are valid
 *            on return.  in must be a multiple of 8.
 *   n_seen   host pointer, in/out, may be NULL: incremented by n_tokens.
 *   status_dev  device int, may be NULL.
 *   workspace   bf16 X: unused, may be NULL.  fp32 X: adadim_workspace_bytes(ADADIM_WS_HESSIAN,
 *               n_tokens, in, 0, 0) bytes (the chunk's token count in the `out` argument),
 *               256-byte aligned, for the tensor-core path.
 */
ADADIM_API int adadim_hessian_accumulate(const void* X, int xdtype, int64_t n_tokens, int64_t in, int64_t ldx,
                              float* H, int64_t* n_seen, int* status_dev,
                              void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Round-to-nearest group quantizer (Section 4.1: uniform asymmetric, group size g; Appendix A.2:
 * min-max), in one pass over W for one or both grouping dimensions (Section 3.3: the weights are
 * quantized independently per-IC and per-OC).  Per group G, in IEEE binary32:
 *     lo = min(0, min_G w)   hi = max(0, max_G w)
 *     s  = fp16_rn((hi - lo) / maxq);   if s == 0 or s is not finite: s = 1, z = 0, codes 0
 *     z  = clamp(rint(-lo / s), 0, maxq)
 *     c  = clamp(rint(w / s) + z, 0, maxq)          maxq = 2^bits - 1, rint = ties to even
 *   W      [out][in], wdtype ADADIM_F16 or ADADIM_F32; ldw in elements, 16-byte aligned rows.
 *   bits   2, 3, 4 or 8 (INT3 is the paper's headline, INT4 its Appendix; 2 and 8 bound the range);
 *          group 32, 64, 128 or 256 (the paper's sweep, Section 4.4, uses 64, 128, 256).
 *   dim    ADADIM_DIM_OC (q_oc written), ADADIM_DIM_IC (q_ic written) or ADADIM_DIM_BOTH.
 *   Shape rules: in % 32 == 0; per-OC needs in % group == 0; per-IC needs out % group == 0.
 *   out == 0 or in == 0 is accepted and does nothing.
 */
ADADIM_API int adadim_quantize_rtn(const void* W, int wdtype, int64_t out, int64_t in, int64_t ldw,
                        int bits, int group, int dim,
                        const adadim_qtensor* q_oc, const adadim_qtensor* q_ic, void* cuda_stream);

/*
 * Damped Cholesky-inverse factor used by GPTQ (Section 2.2; the damping is the published
 * algorithm's): columns with H[i,i] == 0 get H[i,i] = 1 ("dead" columns), then
 *     Hd = H + lambda*I,  lambda = percdamp * mean(diag H),   U upper triangular, Hd^-1 = U^T U.
 *   H  [in][in] fp32 (not modified);  U [in][in] fp64 out, strictly-lower part set to 0.
 *      (U is binary64 because GPTQ's rounding decisions thousands of columns later depend on
 *      it: see adadim_quantize_gptq.)
 *   in must be a multiple of 64.
 *   workspace  adadim_workspace_bytes(ADADIM_WS_FACTOR, 0, in, 0, 0) bytes, 256-byte aligned.
 *   status_dev ADADIM_ERR_NOT_PD if a pivot is not positive.
 */
ADADIM_API int adadim_cholesky_inverse_factor(const float* H, int64_t in, double percdamp, double* U,
                                   int* status_dev, void* workspace, size_t workspace_bytes,
                                   void* cuda_stream);

/*
 * GPTQ (Section 2.2; Section 3.3: the per-IC variant changes only the quantization step):
 * columns are quantized in order; after column i the rounding error e = (w_i - q_i) / U[i,i]
 * is propagated to the not-yet-quantized columns, W[:, j] -= e * U[i, j] (j > i), lazily
 * batched in blocks of `blocksize` columns.  Group parameters come from the CURRENT
 * (already compensated) weights with the formula of adadim_quantize_rtn: per-OC at each
 * group's first column, from that group's columns; per-IC at every column, from its g-row
 * groups.  Weights of dead columns are treated as 0.
 * Precision: the working weights, U and every error and update are binary64; the weight as it
 * stands when its column is reached is rounded once to binary32 and quantized with the binary32
 * formula above.  (A binary32 working copy drifts by a few 1e-6 of a quantization step over
 * thousands of columns, which is enough to flip individual roundings, and every flip changes
 * all later columns of its row or group.)
 *   H          [in][in] fp32, required: its diagonal marks the dead columns, and when U == NULL
 *              the factor is computed from it into workspace.
 *   U          optional precomputed adadim_cholesky_inverse_factor of the same H, or NULL.
 *   blocksize  128.  group 32, 64, 128 or 256.  in % 128 == 0, out % 128 == 0; at group 256 a per-OC
 *              group spans two column blocks and a per-IC group two 128-row slabs (two CTAs of a
 *              cluster exchange the column's minimum and maximum), so in % 256 == 0 and out % 256 == 0.
 *   gptq_loss  optional device double[2] (OC, IC): 1/2 * sum of e^2 (only the element of a
 *              dimension that was run is written).
 *   workspace  adadim_workspace_bytes(ADADIM_WS_GPTQ, out, in, bits, group), 256-byte aligned.
 */
ADADIM_API int adadim_quantize_gptq(const void* W, int wdtype, int64_t out, int64_t in, int64_t ldw,
                         const float* H, const double* U, int bits, int group, int dim,
                         double percdamp, int blocksize,
                         const adadim_qtensor* q_oc, const adadim_qtensor* q_ic,
                         double* gptq_loss, int* status_dev,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * GPTQ for several layers that share their input (Section 3.3 and Appendix B give the per-layer
 * flow: the dimension is chosen with RTN, then GPTQ runs in it; in a transformer block q, k, v
 * (and gate, up) read the same activations, hence the same H and U).  The layers' working rows are
 * stacked, so one chain of 128-column steps serves all of them: the sequential depth of the
 * method is paid once instead of once per layer, and the device is filled by 3-4 times the rows.
 * Every layer is quantized exactly as adadim_quantize_gptq would quantize it alone.
 *   layers     host array of n_layers descriptors (read during the call only).  Per layer:
 *                W, out, ldw      the weight [out][in], element type wdtype (shared), out % 128 == 0
 *                q_oc, q_ic       outputs; both are required for ADADIM_DIM_BOTH and
 *                                 ADADIM_DIM_CHOSEN, the one named by dim otherwise
 *                dim              ADADIM_DIM_OC, _IC, _BOTH, or ADADIM_DIM_CHOSEN: the dimension is read
 *                                 on the device from *chosen when the kernels run (for example the
 *                                 word adadim_score_select wrote for this layer's RTN results), so
 *                                 the paper's flow needs no host round trip between its two halves;
 *                                 only the chosen tensor is written
 *                chosen           device int (adadim_dim), used with ADADIM_DIM_CHOSEN
 *                gptq_loss        optional device double[2]: element [dim] receives 1/2 sum e^2
 *   A layer in both dimensions counts as two working copies; at most ADADIM_MAX_BATCHED_LAYERS
 *   copies per call.  workspace: adadim_workspace_bytes(ADADIM_WS_GPTQ_ROWS, rows, in, ..) with
 *   rows the total of the copies' out.  Other arguments as adadim_quantize_gptq.
 */
#define ADADIM_MAX_BATCHED_LAYERS 16
typedef struct {
  const void* W;
  int64_t out;
  int64_t ldw;
  const adadim_qtensor* q_oc;
  const adadim_qtensor* q_ic;
  int dim;
  const int* chosen;
  double* gptq_loss;
} adadim_gptq_layer;
ADADIM_API int adadim_quantize_gptq_batched(const adadim_gptq_layer* layers, int n_layers, int wdtype, int64_t in,
                         const float* H, const double* U, int bits, int group,
                         double percdamp, int blocksize, int* status_dev,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * GPTQ with activation reordering (Section 2.2; Appendix A.1): the input channels are quantized
 * in the order of descending diag(H) (a zero diagonal counts as 1; equal values keep their
 * original order), so the channels that see the largest activations are rounded first and are
 * not used afterwards to absorb the error of the others.  The method is adadim_quantize_gptq
 * applied to the reordered problem; every output is stored at the channel's ORIGINAL position,
 * so the tensors have the same layout as without reordering:
 *   per-IC  group parameters are taken from the current weights of the column being quantized,
 *           as before; scales/zeros [out/g][in] stay contiguous (the point of Appendix A.1).
 *   per-OC  "static groups" (Section 2.2): the parameters of every group of g consecutive
 *           original columns are fixed from the original weights before anything is reordered
 *           or updated (they equal adadim_quantize_rtn's per-OC parameters); a column is coded
 *           with the parameters of the group it originally belongs to.
 *   perm_out   optional device int32[in]: the order used (perm_out[i] = original index of the
 *              i-th channel quantized).
 *   The factor is always computed here (a factor of the unpermuted H does not apply).
 *   Other arguments, shapes, workspace size (ADADIM_WS_GPTQ) and errors as adadim_quantize_gptq.
 */
ADADIM_API int adadim_quantize_gptq_reordered(const void* W, int wdtype, int64_t out, int64_t in, int64_t ldw,
                         const float* H, int bits, int group, int dim,
                         double percdamp, int blocksize,
                         const adadim_qtensor* q_oc, const adadim_qtensor* q_ic,
                         double* gptq_loss, int32_t* perm_out, int* status_dev,
                         void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Reconstruction error of both quantized tensors and the selection (Section 3.3, Eq. 1;
 * Appendix B):  E_dim = || X (W - Q_dim)^T ||_F^2 = 1/2 trace((W - Q_dim) H (W - Q_dim)^T)
 * with the undamped H = 2 X^T X;  chosen = IC iff E_ic < E_oc (ties and NaN give OC, the
 * dimension evaluated first).
 *   err     device double[2] = {E_oc, E_ic};  chosen  device int (adadim_dim).
 *   Either q_oc or q_ic may be NULL: its error is reported as +infinity.
 *   in % 64 == 0, out % 128 == 0.
 *   workspace  adadim_workspace_bytes(ADADIM_WS_SCORE, out, in, bits, group), 256-byte aligned.
 */
ADADIM_API int adadim_score_select(const void* W, int wdtype, int64_t out, int64_t in, int64_t ldw,
                        const float* H, int bits, int group,
                        const adadim_qtensor* q_oc, const adadim_qtensor* q_ic,
                        double* err, int* chosen, int* status_dev,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * adadim_score_select without a workspace argument, for callers that cannot allocate device
 * memory (the paper has no counterpart: this is a convenience of this library).
 *
 * Who needs it: code that may not call cudaMalloc - a component running inside a process
 * whose device memory is already fully committed (an inference server that gave every free
 * byte to its cache), a plugin that receives tensors but no allocator, or a latency-critical
 * path that cannot accept the device-wide synchronisation an allocation may imply.  Such a
 * caller still passes all inputs and outputs; only the scratch comes from the library: a
 * fixed array of ADADIM_STATIC_SCRATCH_BYTES (16 MiB) in the library's device image, present
 * on every GPU that loads the library for as long as the process lives.
 *
 *   Limit      adadim_workspace_bytes(ADADIM_WS_SCORE, out, in, ..) must not exceed
 *              ADADIM_STATIC_SCRATCH_BYTES (for example out = in = 1024 fits, out = in = 2048
 *              does not); larger layers are refused with ADADIM_ERR_WORKSPACE and nothing is
 *              launched.
 *   First call The first call on each device looks up the array's device address.  With the
 *              CUDA runtime's lazy loading this lookup is also the moment the 16 MiB become
 *              resident on that device, so make the first call early - before the process
 *              commits the device's remaining memory, and outside any stream capture.  If the
 *              memory cannot be had, that call returns ADADIM_ERR_CUDA.
 *   Sharing    All calls on a device use the same array.  It keeps the previous call's
 *              contents, which no call reads (each call rewrites what it uses).  Two calls
 *              whose kernels can overlap on the GPU - different streams, or different host
 *              threads using different streams - race on it and give wrong results: keep
 *              calls on one device ordered on a single stream, or otherwise serialized.
 *   No cudaMalloc, cudaFree or other allocating call is made.  Arguments (validated by the
 *   same code), results, status codes and numerical behaviour are those of adadim_score_select.
 */
#define ADADIM_STATIC_SCRATCH_BYTES (16u << 20)
ADADIM_API int adadim_score_select_static(const void* W, int wdtype, int64_t out, int64_t in, int64_t ldw,
                                          const float* H, int bits, int group,
                                          const adadim_qtensor* q_oc, const adadim_qtensor* q_ic,
                                          double* err, int* chosen, int* status_dev, void* cuda_stream);
ADADIM_API size_t adadim_static_scratch_bytes(void);

/*
 * y = Q x with the quantized weights of a per-IC quantized layer (Section 4.5 and Appendix D:
 * one matrix-vector product of a decoder layer, fp16 vector in, fp16 vector out), consuming the
 * tensors this library emits as they are:  Q[o,i] = scale[o/g, i] * (code[o,i] - zero[o/g, i]).
 *   q       codes [out][in*bits/32], scales and zeros [out/group][in]   (dim must be ADADIM_DIM_IC)
 *   bits    3 or 4;  group any multiple of 16 that divides out (Appendix D measures 128 ... 2048)
 *   x       fp16 [in], 16-byte aligned;  y  fp16 [out].  in % 128 == 0.
 *   Within every 128-column block the sums are formed exactly in integers against a 21-bit
 *   fixed-point image of scale * x; blocks are added in binary32 in column order; the result is
 *   rounded to fp16 once at the end.
 *   workspace  adadim_workspace_bytes(ADADIM_WS_GEMV, out, in, bits, group), 256-byte aligned.
 */
ADADIM_API int adadim_dequant_gemv(const adadim_qtensor* q, int dim, int64_t out, int64_t in, int bits, int group,
                        const void* x, void* y, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Helpers. */
ADADIM_API size_t adadim_workspace_bytes(int kind, int64_t out, int64_t in, int bits, int group);
/* Unpack the bitstream format above: dst [out][in] uint8 (device). */
ADADIM_API int adadim_unpack_codes(const uint32_t* codes, int64_t out, int64_t in, int bits, uint8_t* dst,
                        void* cuda_stream);
ADADIM_API const char* adadim_strerror(int status);
ADADIM_API int adadim_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ADADIM_H_ */
