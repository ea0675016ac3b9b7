"""ctypes binding of libadadim.so.

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  Functions take torch CUDA tensors (used purely as device buffers),
pass their data pointers and the current stream, and raise AdadimError on a
non-zero status.  There is no CPU fallback: if the library cannot be loaded,
every call fails with an ImportError naming the missing file.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

OK = 0
F32, F16, BF16 = 0, 1, 2
DIM_OC, DIM_IC, DIM_BOTH, DIM_CHOSEN = 0, 1, 2, 3
WS_HESSIAN, WS_GPTQ, WS_SCORE, WS_FACTOR, WS_GPTQ_ROWS, WS_GEMV = 0, 1, 2, 3, 4, 5
DIM_NAMES = {DIM_OC: "oc", DIM_IC: "ic"}

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libadadim.so")
_lib = None


class AdadimError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({strerror(status)})")


class QTensorC(C.Structure):
    _fields_ = [("codes", C.c_void_p), ("scales", C.c_void_p), ("zeros", C.c_void_p)]


class GptqLayerC(C.Structure):
    _fields_ = [("W", C.c_void_p), ("out", C.c_int64), ("ldw", C.c_int64), ("q_oc", C.POINTER(QTensorC)),
                ("q_ic", C.POINTER(QTensorC)), ("dim", C.c_int), ("chosen", C.c_void_p), ("gptq_loss", C.c_void_p)]


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2309_15531_b200.build` "
                              "(there is no CPU fallback)")
        L = C.CDLL(_LIB_PATH)
        i64, vp, sz = C.c_int64, C.c_void_p, C.c_size_t
        qp = C.POINTER(QTensorC)
        L.adadim_version.restype = C.c_int
        L.adadim_strerror.restype = C.c_char_p
        L.adadim_strerror.argtypes = [C.c_int]
        L.adadim_workspace_bytes.restype = sz
        L.adadim_workspace_bytes.argtypes = [C.c_int, i64, i64, C.c_int, C.c_int]
        L.adadim_hessian_accumulate.restype = C.c_int
        L.adadim_hessian_accumulate.argtypes = [vp, C.c_int, i64, i64, i64, vp, C.POINTER(i64), vp, vp, sz, vp]
        L.adadim_quantize_rtn.restype = C.c_int
        L.adadim_quantize_rtn.argtypes = [vp, C.c_int, i64, i64, i64, C.c_int, C.c_int, C.c_int, qp, qp, vp]
        L.adadim_cholesky_inverse_factor.restype = C.c_int
        L.adadim_cholesky_inverse_factor.argtypes = [vp, i64, C.c_double, vp, vp, vp, sz, vp]
        L.adadim_quantize_gptq.restype = C.c_int
        L.adadim_quantize_gptq.argtypes = [vp, C.c_int, i64, i64, i64, vp, vp, C.c_int, C.c_int, C.c_int, C.c_double,
                                           C.c_int, qp, qp, vp, vp, vp, sz, vp]
        L.adadim_quantize_gptq_batched.restype = C.c_int
        L.adadim_quantize_gptq_batched.argtypes = [C.POINTER(GptqLayerC), C.c_int, C.c_int, i64, vp, vp, C.c_int,
                                                   C.c_int, C.c_double, C.c_int, vp, vp, sz, vp]
        L.adadim_quantize_gptq_reordered.restype = C.c_int
        L.adadim_quantize_gptq_reordered.argtypes = [vp, C.c_int, i64, i64, i64, vp, C.c_int, C.c_int, C.c_int,
                                                     C.c_double, C.c_int, qp, qp, vp, vp, vp, vp, sz, vp]
        L.adadim_score_select.restype = C.c_int
        L.adadim_score_select.argtypes = [vp, C.c_int, i64, i64, i64, vp, C.c_int, C.c_int, qp, qp, vp, vp, vp, vp,
                                          sz, vp]
        L.adadim_score_select_static.restype = C.c_int
        L.adadim_score_select_static.argtypes = [vp, C.c_int, i64, i64, i64, vp, C.c_int, C.c_int, qp, qp, vp, vp,
                                                 vp, vp]
        L.adadim_static_scratch_bytes.restype = sz
        L.adadim_dequant_gemv.restype = C.c_int
        L.adadim_dequant_gemv.argtypes = [qp, C.c_int, i64, i64, C.c_int, C.c_int, vp, vp, vp, sz, vp]
        L.adadim_unpack_codes.restype = C.c_int
        L.adadim_unpack_codes.argtypes = [vp, i64, i64, C.c_int, vp, vp]
        _lib = L
    return _lib


def strerror(status: int) -> str:
    return lib().adadim_strerror(int(status)).decode()


def version() -> int:
    return lib().adadim_version()


def workspace_bytes(kind: int, out: int, inp: int, bits: int = 0, group: int = 0) -> int:
    return int(lib().adadim_workspace_bytes(kind, out, inp, bits, group))


_DT = {torch.float32: F32, torch.float16: F16, torch.bfloat16: BF16}


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(rc: int, where: str):
    if rc != OK:
        raise AdadimError(rc, where)


class QTensor:
    """Device buffers of one quantized tensor (see include/adadim.h for the layout)."""

    def __init__(self, out: int, inp: int, bits: int, group: int, dim: int, device="cuda"):
        self.out, self.inp, self.bits, self.group, self.dim = out, inp, bits, group, dim
        self.codes = torch.zeros(out, inp * bits // 32, dtype=torch.int32, device=device)
        shape = (out, inp // group) if dim == DIM_OC else (out // group, inp)
        self.scales = torch.zeros(shape, dtype=torch.float16, device=device)
        self.zeros = torch.zeros(shape, dtype=torch.float16, device=device)

    def c(self) -> QTensorC:
        return QTensorC(self.codes.data_ptr(), self.scales.data_ptr(), self.zeros.data_ptr())

    def unpacked(self) -> torch.Tensor:
        dst = torch.empty(self.out, self.inp, dtype=torch.uint8, device=self.codes.device)
        _check(lib().adadim_unpack_codes(self.codes.data_ptr(), self.out, self.inp, self.bits, dst.data_ptr(),
                                         _stream()), "adadim_unpack_codes")
        return dst


def _ws(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)


def hessian_accumulate(X: torch.Tensor, H: torch.Tensor, status: Optional[torch.Tensor] = None,
                       workspace: Optional[torch.Tensor] = None, tensor_cores: bool = True) -> None:
    """H += 2 X^T X for X[n_tokens, in] (bf16 or fp32), H[in, in] fp32.  fp32 X runs on the tensor cores
    through a workspace (allocated here if none is given); tensor_cores=False selects the plain kernel."""
    assert X.is_cuda and H.is_cuda and X.stride(1) == 1 and H.is_contiguous()
    ws_ptr, ws_len = None, 0
    if X.dtype == torch.float32 and tensor_cores and X.shape[0] > 0:
        if workspace is None:
            workspace = _ws(workspace_bytes(WS_HESSIAN, X.shape[0], X.shape[1]), X.device)
        ws_ptr, ws_len = workspace.data_ptr(), workspace.numel()
    rc = lib().adadim_hessian_accumulate(X.data_ptr(), _DT[X.dtype], X.shape[0], X.shape[1], X.stride(0),
                                         H.data_ptr(), None, status.data_ptr() if status is not None else None,
                                         ws_ptr, ws_len, _stream())
    _check(rc, "adadim_hessian_accumulate")


def quantize_rtn(W: torch.Tensor, bits: int, group: int, dim: int = DIM_BOTH,
                 q_oc: Optional[QTensor] = None, q_ic: Optional[QTensor] = None):
    assert W.is_cuda and W.stride(1) == 1
    out, inp = W.shape
    if dim != DIM_IC and q_oc is None:
        q_oc = QTensor(out, inp, bits, group, DIM_OC, W.device)
    if dim != DIM_OC and q_ic is None:
        q_ic = QTensor(out, inp, bits, group, DIM_IC, W.device)
    coc = q_oc.c() if q_oc is not None else None
    cic = q_ic.c() if q_ic is not None else None
    rc = lib().adadim_quantize_rtn(W.data_ptr(), _DT[W.dtype], out, inp, W.stride(0), bits, group, dim,
                                   C.byref(coc) if coc is not None else None,
                                   C.byref(cic) if cic is not None else None, _stream())
    _check(rc, "adadim_quantize_rtn")
    return q_oc, q_ic


def cholesky_inverse_factor(H: torch.Tensor, percdamp: float = 0.01, status: Optional[torch.Tensor] = None,
                            workspace: Optional[torch.Tensor] = None, U: Optional[torch.Tensor] = None) -> torch.Tensor:
    n = H.shape[0]
    if U is None:
        U = torch.empty(n, n, dtype=torch.float64, device=H.device)
    if workspace is None:
        workspace = _ws(workspace_bytes(WS_FACTOR, 0, n), H.device)
    rc = lib().adadim_cholesky_inverse_factor(H.data_ptr(), n, percdamp, U.data_ptr(),
                                              status.data_ptr() if status is not None else None,
                                              workspace.data_ptr(), workspace.numel(), _stream())
    _check(rc, "adadim_cholesky_inverse_factor")
    return U


def quantize_gptq(W: torch.Tensor, H: torch.Tensor, bits: int, group: int, dim: int = DIM_BOTH,
                  percdamp: float = 0.01, U: Optional[torch.Tensor] = None,
                  q_oc: Optional[QTensor] = None, q_ic: Optional[QTensor] = None,
                  loss: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None,
                  workspace: Optional[torch.Tensor] = None):
    assert W.is_cuda and W.stride(1) == 1 and H.is_contiguous()
    out, inp = W.shape
    if dim != DIM_IC and q_oc is None:
        q_oc = QTensor(out, inp, bits, group, DIM_OC, W.device)
    if dim != DIM_OC and q_ic is None:
        q_ic = QTensor(out, inp, bits, group, DIM_IC, W.device)
    if workspace is None:
        workspace = _ws(workspace_bytes(WS_GPTQ, out, inp, bits, group), W.device)
    coc = q_oc.c() if q_oc is not None else None
    cic = q_ic.c() if q_ic is not None else None
    rc = lib().adadim_quantize_gptq(W.data_ptr(), _DT[W.dtype], out, inp, W.stride(0), H.data_ptr(),
                                    U.data_ptr() if U is not None else None, bits, group, dim, percdamp, 128,
                                    C.byref(coc) if coc is not None else None,
                                    C.byref(cic) if cic is not None else None,
                                    loss.data_ptr() if loss is not None else None,
                                    status.data_ptr() if status is not None else None,
                                    workspace.data_ptr(), workspace.numel(), _stream())
    _check(rc, "adadim_quantize_gptq")
    return q_oc, q_ic


def quantize_gptq_batched(Ws, H: torch.Tensor, bits: int, group: int, dims, percdamp: float = 0.01,
                          U: Optional[torch.Tensor] = None, chosen=None, qs=None, losses=None,
                          status: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None):
    """GPTQ for layers that share H (and U): one call, one chain of column steps for all of them.
    Ws: list of weights [out_l, in] of one dtype; dims: one of DIM_OC / DIM_IC / DIM_BOTH / DIM_CHOSEN per
    layer; chosen: per layer a device int32[1] (required for DIM_CHOSEN, e.g. score_select's output);
    qs: optional list of (q_oc, q_ic) to write into.  Returns the list of (q_oc, q_ic); with DIM_CHOSEN
    both are allocated and the one named by the device word is written."""
    n = len(Ws)
    inp = Ws[0].shape[1]
    assert all(w.is_cuda and w.stride(1) == 1 and w.shape[1] == inp and w.dtype == Ws[0].dtype for w in Ws)
    out_qs, keep, arr = [], [], (GptqLayerC * n)()
    rows = 0
    for l, W in enumerate(Ws):
        out, dim = W.shape[0], dims[l]
        q_oc, q_ic = qs[l] if qs is not None else (None, None)
        if dim != DIM_IC and q_oc is None:
            q_oc = QTensor(out, inp, bits, group, DIM_OC, W.device)
        if dim != DIM_OC and q_ic is None:
            q_ic = QTensor(out, inp, bits, group, DIM_IC, W.device)
        coc = q_oc.c() if q_oc is not None else None
        cic = q_ic.c() if q_ic is not None else None
        keep.append((coc, cic))
        arr[l].W, arr[l].out, arr[l].ldw, arr[l].dim = W.data_ptr(), out, W.stride(0), dim
        arr[l].q_oc = C.pointer(coc) if coc is not None else None
        arr[l].q_ic = C.pointer(cic) if cic is not None else None
        arr[l].chosen = chosen[l].data_ptr() if chosen is not None and chosen[l] is not None else None
        arr[l].gptq_loss = losses[l].data_ptr() if losses is not None and losses[l] is not None else None
        out_qs.append((q_oc, q_ic))
        rows += out * (2 if dim == DIM_BOTH else 1)
    if workspace is None:
        workspace = _ws(workspace_bytes(WS_GPTQ_ROWS, rows, inp, bits, group), Ws[0].device)
    rc = lib().adadim_quantize_gptq_batched(arr, n, _DT[Ws[0].dtype], inp, H.data_ptr(),
                                            U.data_ptr() if U is not None else None, bits, group, percdamp, 128,
                                            status.data_ptr() if status is not None else None,
                                            workspace.data_ptr(), workspace.numel(), _stream())
    _check(rc, "adadim_quantize_gptq_batched")
    return out_qs


def quantize_gptq_reordered(W: torch.Tensor, H: torch.Tensor, bits: int, group: int, dim: int = DIM_BOTH,
                            percdamp: float = 0.01,
                            q_oc: Optional[QTensor] = None, q_ic: Optional[QTensor] = None,
                            loss: Optional[torch.Tensor] = None, perm: Optional[torch.Tensor] = None,
                            status: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None):
    """GPTQ with activation reordering (per-IC: dynamic groups; per-OC: static groups).
    `perm`, if given, is an int32[in] device tensor that receives the column order."""
    assert W.is_cuda and W.stride(1) == 1 and H.is_contiguous()
    out, inp = W.shape
    if dim != DIM_IC and q_oc is None:
        q_oc = QTensor(out, inp, bits, group, DIM_OC, W.device)
    if dim != DIM_OC and q_ic is None:
        q_ic = QTensor(out, inp, bits, group, DIM_IC, W.device)
    if workspace is None:
        workspace = _ws(workspace_bytes(WS_GPTQ, out, inp, bits, group), W.device)
    coc = q_oc.c() if q_oc is not None else None
    cic = q_ic.c() if q_ic is not None else None
    rc = lib().adadim_quantize_gptq_reordered(W.data_ptr(), _DT[W.dtype], out, inp, W.stride(0), H.data_ptr(),
                                              bits, group, dim, percdamp, 128,
                                              C.byref(coc) if coc is not None else None,
                                              C.byref(cic) if cic is not None else None,
                                              loss.data_ptr() if loss is not None else None,
                                              perm.data_ptr() if perm is not None else None,
                                              status.data_ptr() if status is not None else None,
                                              workspace.data_ptr(), workspace.numel(), _stream())
    _check(rc, "adadim_quantize_gptq_reordered")
    return q_oc, q_ic


def score_select(W: torch.Tensor, H: torch.Tensor, bits: int, group: int,
                 q_oc: Optional[QTensor], q_ic: Optional[QTensor],
                 err: Optional[torch.Tensor] = None, chosen: Optional[torch.Tensor] = None,
                 status: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None):
    """Returns (err float64[2] = (E_oc, E_ic), chosen int32[1]) as device tensors."""
    assert W.is_cuda and W.stride(1) == 1 and H.is_contiguous()
    out, inp = W.shape
    if err is None:
        err = torch.empty(2, dtype=torch.float64, device=W.device)
    if chosen is None:
        chosen = torch.empty(1, dtype=torch.int32, device=W.device)
    if workspace is None:
        workspace = _ws(workspace_bytes(WS_SCORE, out, inp, bits, group), W.device)
    coc = q_oc.c() if q_oc is not None else None
    cic = q_ic.c() if q_ic is not None else None
    rc = lib().adadim_score_select(W.data_ptr(), _DT[W.dtype], out, inp, W.stride(0), H.data_ptr(), bits, group,
                                   C.byref(coc) if coc is not None else None,
                                   C.byref(cic) if cic is not None else None,
                                   err.data_ptr(), chosen.data_ptr(),
                                   status.data_ptr() if status is not None else None,
                                   workspace.data_ptr(), workspace.numel(), _stream())
    _check(rc, "adadim_score_select")
    return err, chosen


def dequant_gemv(codes: torch.Tensor, scales: torch.Tensor, zeros: torch.Tensor, bits: int, group: int,
                 x: torch.Tensor, y: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """y = Q x for a per-IC quantized layer: codes int32 [out, in*bits/32], scales / zeros fp16
    [out/group, in], x fp16 [in]; returns y fp16 [out]."""
    out, inp = codes.shape[0], scales.shape[1]
    assert x.dtype == torch.float16 and x.is_contiguous() and codes.is_contiguous()
    if y is None:
        y = torch.empty(out, dtype=torch.float16, device=x.device)
    if workspace is None:
        workspace = _ws(workspace_bytes(WS_GEMV, out, inp, bits, group), x.device)
    qc = QTensorC(codes.data_ptr(), scales.data_ptr(), zeros.data_ptr())
    rc = lib().adadim_dequant_gemv(C.byref(qc), DIM_IC, out, inp, bits, group, x.data_ptr(), y.data_ptr(),
                                   workspace.data_ptr(), workspace.numel(), _stream())
    _check(rc, "adadim_dequant_gemv")
    return y


def static_scratch_bytes() -> int:
    return int(lib().adadim_static_scratch_bytes())


def score_select_static(W: torch.Tensor, H: torch.Tensor, bits: int, group: int,
                        q_oc: Optional[QTensor], q_ic: Optional[QTensor],
                        err: torch.Tensor, chosen: torch.Tensor, status: Optional[torch.Tensor] = None) -> None:
    """score_select on the library's built-in scratch array, for callers that cannot allocate
    device memory.  The caller passes every buffer, outputs included (err float64[2], chosen
    int32[1]); this wrapper creates no tensor.  Layers whose scoring workspace exceeds
    static_scratch_bytes() raise AdadimError(status 6).  Calls on one device must not overlap
    on the GPU: they share the array."""
    out, inp = W.shape
    coc = q_oc.c() if q_oc is not None else None
    cic = q_ic.c() if q_ic is not None else None
    rc = lib().adadim_score_select_static(W.data_ptr(), _DT[W.dtype], out, inp, W.stride(0), H.data_ptr(), bits, group,
                                          C.byref(coc) if coc is not None else None,
                                          C.byref(cic) if cic is not None else None,
                                          err.data_ptr(), chosen.data_ptr(),
                                          status.data_ptr() if status is not None else None, _stream())
    _check(rc, "adadim_score_select_static")
