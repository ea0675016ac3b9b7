"""Shared helpers of the GPU parity tests: tensor <-> numpy plumbing and comparison metrics."""
import numpy as np
import torch

from oracle import adadim_oracle as O
from paper_2309_15531_b200 import binding as B


def to_np(t):
    if t.dtype == torch.bfloat16:
        return t.detach().float().cpu().numpy()
    return t.detach().cpu().numpy()


def q_to_np(q):
    """(codes uint8 [out,in], scales fp16, zeros fp16) of a binding.QTensor; also checks that the
    library's own unpacker and the oracle's reading of the packed format agree."""
    packed = q.codes.cpu().numpy().view(np.uint32)
    codes = O.unpack_codes(packed, q.inp, q.bits)
    lib_codes = q.unpacked().cpu().numpy()
    assert np.array_equal(codes, lib_codes), "packed-format unpackers disagree"
    return codes, q.scales.cpu().numpy(), q.zeros.cpu().numpy()


def assert_rtn_equal(q, ref, what=""):
    codes, scales, zeros = q_to_np(q)
    ds = int((scales.view(np.uint16) != ref["scales"].view(np.uint16)).sum())
    dz = int((zeros.view(np.uint16) != ref["zeros"].view(np.uint16)).sum())
    dc = int((codes != ref["codes"]).sum())
    assert ds == 0 and dz == 0 and dc == 0, f"{what}: {dc} codes, {ds} scales, {dz} zeros differ"


def code_mismatch(codes, ref_codes):
    """(fraction of differing positions, largest difference in levels)."""
    diff = np.abs(codes.astype(np.int16) - ref_codes.astype(np.int16))
    return float((diff != 0).mean()), int(diff.max()) if diff.size else 0


def status_tensor():
    return torch.zeros(1, dtype=torch.int32, device="cuda")


def gptq_trajectory_check(Wn, codes, s, z, U, dead, bits, group, dim, margin=1e-3):
    """Is a GPTQ result a valid run of the method, judged from the result alone?

    GPTQ is a greedy recurrence: when two evaluations differ in one rounding, everything after
    it legitimately differs, so agreement with one reference run is not the only thing that can
    be checked.  What every correct run satisfies, whatever path it took: with D = W - Q and U
    the Cholesky-inverse factor, the propagated errors are Err = D U^-1 (because W - Q = Err U),
    the weight of column i as it stood when it was quantized is cur_i = q_i + Err_i U_ii, and
      (1) every code is the nearest level of (float32) cur_i under the stored (scale, zero),
      (2) every stored (scale, zero) is the quantizer's formula applied to the weights it was
          taken from: per-IC the g rows of cur_i; per-OC the group's columns as they stood at
          the group's first column, cur_j + sum_{i in group, i < j} Err_i U_ij.
    Everything is recomputed here in binary64 from W, the result and the oracle's U; positions
    whose weight lies within `margin` of a quantization step from a rounding boundary (and
    groups whose range lies that close to an fp16 rounding boundary of the scale) cannot be
    decided by a binary64 recomputation of a binary64 run and are counted as undecided.
    Returns dict(bad_codes, bad_params, undecided_codes, undecided_params, n_codes, n_params).
    """
    import scipy.linalg as sl
    W = np.array(Wn, dtype=np.float64)
    W[:, dead] = 0.0
    out, inp = W.shape
    Q = O.dequantize(codes, s, z, group, dim).astype(np.float64)
    D = W - Q
    # Err U = D  <=>  U^T Err^T = D^T
    Err = sl.solve_triangular(U, D.T, trans="T", lower=False).T
    du = np.diag(U)
    cur = Q + Err * du[None, :]
    maxq = float(2 ** bits - 1)
    sf = s.astype(np.float64)
    zf = z.astype(np.float64)
    if dim == "oc":
        # weights at the time the group's parameters were taken
        start = np.empty_like(cur)
        for g0 in range(0, inp, group):
            Ug = np.triu(U[g0:g0 + group, g0:g0 + group], 1)
            start[:, g0:g0 + group] = cur[:, g0:g0 + group] + Err[:, g0:g0 + group] @ Ug
        G = start.astype(np.float32).reshape(out, inp // group, group)
        lo, hi = G.min(axis=2), G.max(axis=2)
        se, ze = np.repeat(sf, group, axis=1), np.repeat(zf, group, axis=1)
    else:
        G = cur.astype(np.float32).reshape(out // group, group, inp)
        lo, hi = G.min(axis=1), G.max(axis=1)
        se, ze = np.repeat(sf, group, axis=0), np.repeat(zf, group, axis=0)
    s_exp, z_exp, bad = O.group_params(lo, hi, bits)
    # (2) parameters
    lo64 = np.minimum(lo.astype(np.float64), 0.0)
    hi64 = np.maximum(hi.astype(np.float64), 0.0)
    raw = (hi64 - lo64) / maxq                         # the scale before fp16 rounding
    ulp16 = np.maximum(np.spacing(raw.astype(np.float16)).astype(np.float64), 2.0 ** -24)
    frac16 = np.abs((raw / ulp16) % 1.0 - 0.5)         # distance from an fp16 rounding boundary, in ulps
    zq = (-lo64) / np.where(sf == 0, 1.0, sf)
    fracz = np.abs(zq % 1.0 - 0.5)
    und_p = (frac16 < margin) | (fracz < margin)
    okp = (s_exp.astype(np.float16).view(np.uint16) == s.view(np.uint16)) & \
          (z_exp.astype(np.float16).view(np.uint16) == z.view(np.uint16))
    bad_params = int((~okp & ~und_p).sum())
    # (1) codes: nearest level of cur under the stored parameters
    t = cur.astype(np.float32).astype(np.float64) / se
    c_exp = np.clip(np.rint(t) + ze, 0, maxq)
    und_c = np.abs(t % 1.0 - 0.5) < margin
    okc = c_exp == codes.astype(np.float64)
    bad_codes = int((~okc & ~und_c).sum())
    return {"bad_codes": bad_codes, "bad_params": bad_params,
            "undecided_codes": int((~okc & und_c).sum()), "undecided_params": int((~okp & und_p).sum()),
            "n_codes": int(codes.size), "n_params": int(s.size)}
