"""The larger workload shapes through the C ABI, against the oracle on sampled slabs.

The Hessian is an INPUT of these tests (GPTQ and the scorer take it as given): it is formed
with torch in fp64 from the seeded activations, rounded to fp32 once, and handed to both the
library and the oracle.  The library's own Hessian kernel is tested in test_gpu_hessian.py.
The oracle's Cholesky-inverse factor is a LAPACK inverse + factorization of the full matrix;
its GPTQ recurrence runs on one or two 128-row slabs (rows are independent under per-OC
grouping, 128-row slabs under per-IC grouping).

What is compared.  GPTQ takes thousands of rounding decisions in sequence, each on a weight
that carries the compensation of all earlier ones, and with group parameters recomputed from
those weights.  Any two evaluations that round the intermediate weights differently (fp64 vs
fp32, or two fp32 orders of summation) agree at first and then drift apart: a weight that
lands on the other side of a rounding boundary changes the error that is fed forward.  On
these long layers with strong outlier channels a plain numpy fp32 evaluation of the oracle's
own recurrence differs from its fp64 evaluation at 4.6 % of per-IC codes (in = 8192, 4-bit),
nearly all of it in the later columns (the library: 4.0 % there, 13 % on the 11008-column
skewed layer, 0.04 % on the 4096-column one).  The tests therefore check (1) the codes of the
first 1024 columns, where the two evaluations have not yet separated, at the 0.1 % / one-level
bar, (2) the reconstruction error of the whole slab against the oracle's within 1e-3, i.e.
that the two results are equally good, and (3) that the overall difference stays far from
that of unrelated codes.  Which of two equally good greedy paths is taken is not unique.
The library's own consistency over a whole layer (its reported loss against
1/2 trace(D Hd D^T) of its own result) is checked in test_gpu_gptq.py.
"""
import numpy as np
import pytest
import torch

from oracle import adadim_oracle as O
from paper_2309_15531_b200 import binding as B
from paper_2309_15531_b200 import flows as F
from paper_2309_15531_b200 import inputs as I
from tests.helpers import code_mismatch, q_to_np, status_tensor, to_np

pytestmark = pytest.mark.gpu


def _hessian_input(X):
    Xd = X.double()
    H = (2.0 * (Xd.T @ Xd)).float()
    return H.contiguous()


def _check_slab(W, H, bits, group, rows, U_ref, dead, q_oc, q_ic, tag):
    Wn = to_np(W[rows]).astype(np.float32)
    Hn = to_np(H)
    H64 = Hn.astype(np.float64)
    for name, q in (("oc", q_oc), ("ic", q_ic)):
        if q is None:
            continue
        ref = O.quantize_gptq(Wn, Hn, bits, group, name, 0.01, U=U_ref, dead=dead)
        codes, s, z = q_to_np(q)
        frac, lvl = code_mismatch(codes[rows], ref["codes"])
        frac0, lvl0 = code_mismatch(codes[rows, :1024], ref["codes"][:, :1024])
        Q = O.dequantize(codes, s, z, group, name)[rows]
        e_gpu = O.recon_error_trace(Wn, Q, H64)
        e_ref = O.recon_error_trace(Wn, ref["Q"], H64)
        print(f"{tag} gptq {name} b{bits} g{group}: codes differ {100 * frac0:.4f}% in the first 1024 columns "
              f"(max {lvl0} levels), {100 * frac:.4f}% overall (max {lvl} levels), "
              f"E gpu {e_gpu:.6e} oracle {e_ref:.6e}")
        assert frac0 <= 1e-3 and lvl0 <= 1
        assert frac <= 0.3                        # drift of rounding order (random codes would differ at ~85 %)
        assert e_gpu == pytest.approx(e_ref, rel=1e-3)


def test_down_proj_gptq_4bit_g128_and_3bit_g64():
    """LLaMA-7B down_proj shape, skewed activations (the Hessian has a strong rank-one part)."""
    wl = I.workload_downproj(n_tokens=8192)
    wspec, xspec = wl["layers"]["down_proj"]
    W = I.make_weight(wspec, "cuda")
    H = _hessian_input(I.make_calib(xspec, "cuda"))
    st = status_tensor()
    U = B.cholesky_inverse_factor(H, 0.01, status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    Hd, dead = O.damped_hessian(to_np(H).astype(np.float64), 0.01)
    U_ref = O.cholesky_inverse_factor(Hd)
    scale = np.diag(U_ref)[:, None]
    e = float(np.max(np.abs(to_np(U).astype(np.float64) - U_ref) / scale))
    print(f"factor n={wspec.inp}: max |U - Uref| / U_ii = {e:.3e}")
    assert e < 1e-6
    rows = slice(2048, 2176)
    for bits, group in wl["variants"]:
        q_oc, q_ic = B.quantize_gptq(W, H, bits, group, B.DIM_BOTH, 0.01, U=U, status=st)
        err, chosen = B.score_select(W, H, bits, group, q_oc, q_ic, status=st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        _check_slab(W, H, bits, group, rows, U_ref, dead, q_oc, q_ic, "down_proj")
        e = err.cpu().numpy()
        assert np.isfinite(e).all() and int(chosen.item()) == (B.DIM_IC if e[1] < e[0] else B.DIM_OC)


def test_mlp70b_gate_gptq_4bit():
    """LLaMA-2-70B gate_proj shape (28672 x 8192), RTN and GPTQ 4-bit g128 in both dimensions."""
    wl = I.workload_mlp70b(n_tokens=8192)
    wspec, xspec = wl["layers"]["gate_proj"]
    W = I.make_weight(wspec, "cuda")
    H = _hessian_input(I.make_calib(xspec, "cuda"))
    st = status_tensor()
    dim, err, (q_oc, q_ic) = F.gptq_both(W, H, 4, 128, status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    Hd, dead = O.damped_hessian(to_np(H).astype(np.float64), 0.01)
    U_ref = O.cholesky_inverse_factor(Hd)
    _check_slab(W, H, 4, 128, slice(12800, 12928), U_ref, dead, q_oc, q_ic, "70b_gate")
    e = err.cpu().numpy()
    assert dim == (B.DIM_IC if e[1] < e[0] else B.DIM_OC)


def test_decoder_block_flow():
    """The paper's flow per layer (RTN in both dimensions -> score -> select -> GPTQ in the
    chosen dimension) on three layers of the LLaMA-7B-shaped block; the layers with the same
    input share one Hessian and one factor."""
    wl = I.workload_block(n_tokens=4096)
    st = status_tensor()
    Hs, Us = {}, {}
    for name in ("q_proj", "gate_proj", "down_proj"):
        wspec, xspec = wl["layers"][name]
        if xspec not in Hs:
            Hs[xspec] = _hessian_input(I.make_calib(xspec, "cuda"))
            Us[xspec] = B.cholesky_inverse_factor(Hs[xspec], 0.01, status=st)
        H, U = Hs[xspec], Us[xspec]
        W = I.make_weight(wspec, "cuda")
        dim, err, q = F.gptq_ada(W, H, 3, 128, U=U, status=st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        # the selection against the oracle's RTN errors
        Wn = to_np(W).astype(np.float32)
        H64 = to_np(H).astype(np.float64)
        ref = {d: O.recon_error_trace(Wn, O.quantize_rtn(Wn, 3, 128, d)["Q"], H64) for d in ("oc", "ic")}
        e = err.cpu().numpy()
        print(f"block {name}: E_rtn gpu {e}, oracle {ref}, chosen {B.DIM_NAMES[dim]}")
        assert e[0] == pytest.approx(ref["oc"], rel=1e-3) and e[1] == pytest.approx(ref["ic"], rel=1e-3)
        if abs(ref["oc"] - ref["ic"]) > 1e-4 * max(ref["oc"], ref["ic"]):
            assert B.DIM_NAMES[dim] == O.select_dim(ref["oc"], ref["ic"])
        # GPTQ in the chosen dimension improves on RTN in that dimension
        codes, s, z = q_to_np(q)
        Q = O.dequantize(codes, s, z, 128, B.DIM_NAMES[dim])
        assert O.recon_error_trace(Wn, Q, H64) < ref[B.DIM_NAMES[dim]]
