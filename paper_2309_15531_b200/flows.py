"""The paper's per-layer flows (Section 3.3, Appendix B) as sequences of library calls.

Orchestration only: every computation happens in the C-ABI entry points.  All tensors stay
on the device; the chosen dimension is read back once per layer because it decides which
kernel runs next.
"""
from __future__ import annotations

from typing import Optional

import torch

from . import binding as B


def rtn_ada(W: torch.Tensor, H: torch.Tensor, bits: int, group: int, status: Optional[torch.Tensor] = None):
    """Quantize W in both dimensions with RTN, score both against H, keep the lower error.
    Returns (chosen dim, err float64[2] on device, (q_oc, q_ic))."""
    q_oc, q_ic = B.quantize_rtn(W, bits, group, B.DIM_BOTH)
    err, chosen = B.score_select(W, H, bits, group, q_oc, q_ic, status=status)
    return int(chosen.item()), err, (q_oc, q_ic)


def gptq_ada(W: torch.Tensor, H: torch.Tensor, bits: int, group: int, percdamp: float = 0.01,
             U: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None):
    """The paper's GPTQ flow: choose the dimension with RTN, then run GPTQ in it.
    Returns (chosen dim, RTN errors, quantized tensor of the chosen dimension)."""
    dim, err, _ = rtn_ada(W, H, bits, group, status)
    q_oc, q_ic = B.quantize_gptq(W, H, bits, group, dim, percdamp, U=U, status=status)
    return dim, err, (q_oc if dim == B.DIM_OC else q_ic)


def gptq_ada_reordered(W: torch.Tensor, H: torch.Tensor, bits: int, group: int, percdamp: float = 0.01,
                       status: Optional[torch.Tensor] = None):
    """The paper's final GPTQ design (Section 4.1, Appendix A.1): choose the dimension with RTN,
    then GPTQ in it with activation reordering (static groups when per-OC was chosen).
    Returns (chosen dim, RTN errors, quantized tensor of the chosen dimension)."""
    dim, err, _ = rtn_ada(W, H, bits, group, status)
    q_oc, q_ic = B.quantize_gptq_reordered(W, H, bits, group, dim, percdamp, status=status)
    return dim, err, (q_oc if dim == B.DIM_OC else q_ic)


def gptq_both(W: torch.Tensor, H: torch.Tensor, bits: int, group: int, percdamp: float = 0.01,
              U: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None):
    """GPTQ in both dimensions, scored with the undamped H, lower error kept.
    Returns (chosen dim, err float64[2] on device, (q_oc, q_ic))."""
    q_oc, q_ic = B.quantize_gptq(W, H, bits, group, B.DIM_BOTH, percdamp, U=U, status=status)
    err, chosen = B.score_select(W, H, bits, group, q_oc, q_ic, status=status)
    return int(chosen.item()), err, (q_oc, q_ic)


_SIDE_STREAMS = {}


def _side_stream(device) -> torch.cuda.Stream:
    """One extra stream per device, kept for the life of the process."""
    key = torch.device(device).index if torch.device(device).index is not None else torch.cuda.current_device()
    if key not in _SIDE_STREAMS:
        _SIDE_STREAMS[key] = torch.cuda.Stream(device=key)
    return _SIDE_STREAMS[key]


def block_gptq_ada(layers, bits: int, group: int, percdamp: float = 0.01, status: Optional[torch.Tensor] = None,
                   max_stacked_rows: int = 148 * 128):
    """The paper's flow (RTN in both dimensions -> score -> select -> GPTQ in the chosen dimension)
    for the layers of a transformer block, without a host round trip between the two halves.

    layers: list of (name, W, X) with X the calibration activations of that layer's input; layers that
    are given the SAME X tensor share one Hessian and one factor, and their GPTQ runs stacked in one
    batched call (at most max_stacked_rows working rows per call: one 128-row slab per SM).  The
    Hessian and the factor of an input are computed on a second stream while RTN and scoring of that
    input's layers wait only for the Hessian.
    Returns {name: (chosen device int32[1], RTN errors device float64[2], (q_oc, q_ic))}: of the two
    GPTQ tensors only the one named by `chosen` holds the result.
    """
    main = torch.cuda.current_stream()
    side = _side_stream(layers[0][1].device)
    groups = {}
    for name, W, X in layers:
        groups.setdefault(id(X), (X, []))[1].append((name, W))
    result = {}
    for X, members in groups.values():
        inp = X.shape[1]
        H = torch.zeros(inp, inp, device=X.device)
        # buffers the second stream will use come from this stream's pool: they are handed over and
        # taken back by events, so the caching allocator can reuse them call after call
        U = torch.empty(inp, inp, dtype=torch.float64, device=X.device)
        ws_f = torch.empty(B.workspace_bytes(B.WS_FACTOR, 0, inp), dtype=torch.uint8, device=X.device)
        B.hessian_accumulate(X, H, status)
        h_ready = torch.cuda.Event()
        h_ready.record(main)
        with torch.cuda.stream(side):                   # the factor needs H only; scoring below runs beside it
            side.wait_event(h_ready)
            B.cholesky_inverse_factor(H, percdamp, status, ws_f, U)
            u_ready = torch.cuda.Event()
            u_ready.record(side)
        chosen, errs = {}, {}
        for name, W in members:
            q_oc, q_ic = B.quantize_rtn(W, bits, group, B.DIM_BOTH)
            errs[name], chosen[name] = B.score_select(W, H, bits, group, q_oc, q_ic, status=status)
        main.wait_event(u_ready)
        batch, rows = [], 0
        def flush():
            nonlocal batch, rows
            if not batch:
                return
            qs = B.quantize_gptq_batched([W for _, W in batch], H, bits, group, [B.DIM_CHOSEN] * len(batch), percdamp,
                                         U=U, chosen=[chosen[n] for n, _ in batch], status=status)
            for (n, _), q in zip(batch, qs):
                result[n] = (chosen[n], errs[n], q)
            batch, rows = [], 0
        for name, W in members:
            if batch and (rows + W.shape[0] > max_stacked_rows or len(batch) == 16):
                flush()
            batch.append((name, W))
            rows += W.shape[0]
        flush()
    return result
