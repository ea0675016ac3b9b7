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
