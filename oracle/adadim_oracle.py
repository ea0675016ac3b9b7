"""CPU oracle for the AdaDim quantization path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, readable numpy statement of what the path computes, written
from the paper (arxiv 2309.15531) and, for GPTQ's internals, from the
published algorithm the paper builds on.  It exists so that the CUDA library
can be compared with something that is obviously right.  Nothing in the
product may import this module; only the tests, the smoke check and the
benchmark's CPU-baseline leg do.  It shares no code with the CUDA path.

Precision: the group quantizer is evaluated in IEEE binary32 exactly as
stated below (it is a bit-exact contract); everything else is binary64.

Notation (paper, Section 3): W[out, in] is a linear layer's weight, X[N, in]
the calibration activations (one row per token), b the bit width,
maxq = 2^b - 1, g the group size.  "oc" = groups of g consecutive weights
inside one output channel (a row of W); "ic" = groups of g consecutive
weights inside one input channel (a column of W) (Section 3.2, Figure 1).

Pins (tests/test_oracle_*.py): brute-force nearest-level search on tiny
matrices, the transpose identity ic(W) == oc(W^T)^T, idempotence, the
half-step error bound, on-grid reproduction; Hessian against per-entry
sums and Freivalds probes; trace form against the explicit layer-output
form of Eq. 1; GPTQ against H = I (reduces to RTN), the identities
W - Q = Err U and |Err|^2 = trace(D Hd D^T), an independent
eliminate-one-coordinate (OBS) formulation, and grid-nearest codes; the
dequantized matrix-vector product against an element-by-element loop, the
identity per-IC(W) x == (per-OC(W^T))^T x and the quantization error bound.
Every function here has at least one such pin.
"""
from __future__ import annotations

import numpy as np

F32 = np.float32


# ---------------------------------------------------------------------------
# Group quantizer: uniform asymmetric min-max, b bits (Section 4.1,
# "uniform asymmetric", group size 128; Appendix A.2 "the min-max quantizer").
# The paper prints no formula; the reading used here:
#   lo = min(0, min_G w), hi = max(0, max_G w)        (zero is representable)
#   s  = fp16( (hi - lo) / maxq )                      (stored scale)
#   z  = clamp( rint(-lo / s), 0, maxq )               (integer zero point)
#   c  = clamp( rint(w / s) + z, 0, maxq )             (code)
#   q  = s * (c - z)                                   (dequantized value)
# all in binary32 with round-to-nearest-even and true division; a group
# whose stored scale is zero or not finite gets s = 1, z = 0, codes 0.
# ---------------------------------------------------------------------------

def group_params(lo, hi, bits):
    """(s, z) as float32 arrays from per-group minima / maxima (any shape)."""
    maxq = F32(2 ** bits - 1)
    lo = np.minimum(np.asarray(lo, dtype=F32), F32(0))
    hi = np.maximum(np.asarray(hi, dtype=F32), F32(0))
    with np.errstate(over="ignore", invalid="ignore", divide="ignore"):
        s32 = ((hi - lo) / maxq).astype(F32)
        s = s32.astype(np.float16).astype(F32)            # round to fp16, back to fp32
        bad = (s == 0) | ~np.isfinite(s)
        s = np.where(bad, F32(1), s).astype(F32)
        z = np.rint(((-lo) / s).astype(F32)).astype(F32)
        z = (np.clip(z, F32(0), maxq) + F32(0)).astype(F32)      # an integer 0..maxq: never -0.0
        z = np.where(bad, F32(0), z).astype(F32)
    return s, z, bad


def encode(w, s, z, bits, bad=None):
    """Codes (uint8) of float32 weights w under broadcastable (s, z)."""
    maxq = F32(2 ** bits - 1)
    w = np.asarray(w, dtype=F32)
    with np.errstate(over="ignore", invalid="ignore"):
        c = np.rint((w / s).astype(F32)).astype(F32) + z
        c = np.clip(c.astype(F32), F32(0), maxq)
    if bad is not None:
        c = np.where(bad, F32(0), c)
    return c.astype(np.uint8)


def dequant(c, s, z):
    """q = s * (c - z) in float32 (exact: s has 11 significant bits, c - z at most 4)."""
    return (np.asarray(s, dtype=F32) * (c.astype(F32) - np.asarray(z, dtype=F32))).astype(F32)


def _expand(p, group, dim):
    """Broadcast per-group parameters back to weight shape."""
    return np.repeat(p, group, axis=1 if dim == "oc" else 0)


def quantize_rtn(W, bits, group, dim):
    """Round-to-nearest group quantization of W[out, in] along `dim`.

    oc: parameters have shape [out, in/g]; ic: [out/g, in]  (Section 3.2).
    Returns dict(codes uint8 [out,in], scales float16, zeros float16, Q float32).
    """
    W = np.asarray(W).astype(F32)
    out, inp = W.shape
    if dim == "oc":
        assert inp % group == 0
        G = W.reshape(out, inp // group, group)
        lo, hi = G.min(axis=2), G.max(axis=2)
    elif dim == "ic":
        assert out % group == 0
        G = W.reshape(out // group, group, inp)
        lo, hi = G.min(axis=1), G.max(axis=1)
    else:
        raise ValueError(dim)
    s, z, bad = group_params(lo, hi, bits)
    se, ze, be = _expand(s, group, dim), _expand(z, group, dim), _expand(bad, group, dim)
    c = encode(W, se, ze, bits, be)
    return {"codes": c, "scales": s.astype(np.float16), "zeros": z.astype(np.float16),
            "Q": dequant(c, se, ze)}


def dequantize(codes, scales, zeros, group, dim):
    """Q float32 [out,in] from unpacked codes and fp16 parameters."""
    s = _expand(scales.astype(F32), group, dim)
    z = _expand(zeros.astype(F32), group, dim)
    return dequant(codes, s, z)


# ---------------------------------------------------------------------------
# Packed code format (the paper defines none; its storage accounting, Table 8
# and Appendix C, only counts bits).  Code k of row o occupies bits
# [k*b, (k+1)*b) of that row's little-endian stream of 32-bit words, for both
# grouping dimensions.
# ---------------------------------------------------------------------------

def pack_codes(codes, bits):
    out, inp = codes.shape
    assert (inp * bits) % 32 == 0
    words = np.zeros((out, inp * bits // 32), dtype=np.uint64)
    for k in range(inp):
        bit = k * bits
        wi, sh = bit // 32, bit % 32
        v = codes[:, k].astype(np.uint64) << np.uint64(sh)
        words[:, wi] |= v & np.uint64(0xFFFFFFFF)
        if sh + bits > 32:
            words[:, wi + 1] |= v >> np.uint64(32)
    return words.astype(np.uint32)


def unpack_codes(words, inp, bits):
    out = words.shape[0]
    w64 = words.astype(np.uint64)
    codes = np.zeros((out, inp), dtype=np.uint8)
    mask = np.uint64(2 ** bits - 1)
    for k in range(inp):
        bit = k * bits
        wi, sh = bit // 32, bit % 32
        v = w64[:, wi] >> np.uint64(sh)
        if sh + bits > 32:
            v |= w64[:, wi + 1] << np.uint64(32 - sh)
        codes[:, k] = (v & mask).astype(np.uint8)
    return codes


def average_bits(bits, group, metadata_bits=16):
    """Average storage bits per weight with `metadata_bits` per group
    (the accounting of Table 8 / Appendix C)."""
    return bits + metadata_bits / group


# ---------------------------------------------------------------------------
# Calibration Hessian (Section 4.4: the inverse Hessian is "formed by
# activations"): H = 2 * sum_t x_t^T x_t.
# ---------------------------------------------------------------------------

def hessian(X):
    X = np.asarray(X, dtype=np.float64)
    return 2.0 * (X.T @ X)


# ---------------------------------------------------------------------------
# Reconstruction error and selection (Section 3.3, Eq. 1; Appendix B).
# E(dim) = || X (W - Q_dim)^T ||_F^2, the squared form of Eq. 1's distance
# between the full-precision and quantized layer outputs.  With H = 2 X^T X
# this equals 1/2 trace((W - Q) H (W - Q)^T).  Appendix B's mean of squares
# is E / (N * out); all three are monotone in each other.
# ---------------------------------------------------------------------------

def recon_error_explicit(W, Q, X):
    D = np.asarray(W, dtype=np.float64) - np.asarray(Q, dtype=np.float64)
    Y = np.asarray(X, dtype=np.float64) @ D.T
    return float(np.sum(Y * Y))


def recon_error_trace(W, Q, H):
    D = np.asarray(W, dtype=np.float64) - np.asarray(Q, dtype=np.float64)
    return 0.5 * float(np.sum((D @ np.asarray(H, dtype=np.float64)) * D))


def select_dim(err_oc, err_ic):
    """Argmin of Eq. 1 over {oc, ic}.  oc is evaluated first and replaced only by a
    strictly smaller error (Appendix B's loop order and comparison), so ties give oc."""
    return "ic" if err_ic < err_oc else "oc"


# ---------------------------------------------------------------------------
# GPTQ (Section 2.2: per-column quantization with Hessian-based compensation
# of the rounding error; Section 3.3: the per-IC variant changes only the
# quantization step).  Steps of the published algorithm:
#   dead columns (H_ii = 0): H_ii <- 1, W[:, i] <- 0
#   Hd = H + lambda I, lambda = percdamp * mean(diag H)
#   U = upper-triangular factor with Hd^{-1} = U^T U
#   for each column i, in order:
#       group parameters from the CURRENT weights
#           oc: at i % g == 0, from columns i .. i+g-1 of every row
#           ic: from the g-row groups of column i
#       c = code(W[:, i]);  q = s (c - z)
#       e = (W[:, i] - q) / U_ii
#       W[:, i:] -= e (outer) U[i, i:]
# ---------------------------------------------------------------------------

def damped_hessian(H, percdamp=0.01):
    Hd = np.array(H, dtype=np.float64, copy=True)
    dead = np.diag(Hd) == 0
    idx = np.flatnonzero(dead)
    Hd[idx, idx] = 1.0
    lam = percdamp * float(np.mean(np.diag(Hd)))
    Hd[np.diag_indices_from(Hd)] += lam
    return Hd, dead


def cholesky_inverse_factor(Hd):
    """Upper-triangular U, positive diagonal, with inv(Hd) = U^T U."""
    Hinv = np.linalg.inv(Hd)
    Hinv = 0.5 * (Hinv + Hinv.T)
    return np.linalg.cholesky(Hinv).T.copy()


def quantize_gptq(W, H, bits, group, dim, percdamp=0.01, U=None, dead=None):
    """GPTQ on W[out, in] with group statistics along `dim`.

    For dim == "ic" the rows of W must be whole groups (out % g == 0); passing
    a slab of g-row groups of a larger matrix gives the same result as the
    corresponding rows of the full run (rows interact only inside a group).
    Returns dict(codes, scales, zeros, Q float32, Err float64 [out,in], loss).
    """
    Wc = np.array(np.asarray(W).astype(F32), dtype=np.float64)
    out, inp = Wc.shape
    if U is None:
        Hd, dead = damped_hessian(H, percdamp)
        U = cholesky_inverse_factor(Hd)
    if dead is not None:
        Wc[:, dead] = 0.0
    codes = np.zeros((out, inp), dtype=np.uint8)
    Q = np.zeros((out, inp), dtype=F32)
    Err = np.zeros((out, inp), dtype=np.float64)
    if dim == "oc":
        assert inp % group == 0
        S = np.zeros((out, inp // group), dtype=F32)
        Z = np.zeros((out, inp // group), dtype=F32)
    else:
        assert out % group == 0
        S = np.zeros((out // group, inp), dtype=F32)
        Z = np.zeros((out // group, inp), dtype=F32)
    s = z = bad = None
    for i in range(inp):
        w32 = Wc[:, i].astype(F32)
        if dim == "oc":
            if i % group == 0:
                blk = Wc[:, i:i + group].astype(F32)
                s, z, bad = group_params(blk.min(axis=1), blk.max(axis=1), bits)
                S[:, i // group], Z[:, i // group] = s, z
            se, ze, be = s, z, bad
        else:
            col = w32.reshape(out // group, group)
            s, z, bad = group_params(col.min(axis=1), col.max(axis=1), bits)
            S[:, i], Z[:, i] = s, z
            se, ze, be = np.repeat(s, group), np.repeat(z, group), np.repeat(bad, group)
        c = encode(w32, se, ze, bits, be)
        q = dequant(c, se, ze)
        codes[:, i], Q[:, i] = c, q
        e = (Wc[:, i] - q.astype(np.float64)) / U[i, i]
        Err[:, i] = e
        Wc[:, i:] -= np.outer(e, U[i, i:])
    return {"codes": codes, "scales": S.astype(np.float16), "zeros": Z.astype(np.float16),
            "Q": Q, "Err": Err, "loss": 0.5 * float(np.sum(Err * Err))}


def activation_order(H):
    """Column order of activation reordering (Section 2.2; Appendix A.1): input channels by
    descending activation magnitude, i.e. descending diag(H) after the dead-column fix, equal
    values keeping their original order."""
    d = np.diag(np.asarray(H, dtype=np.float64)).copy()
    d[d == 0.0] = 1.0
    return np.argsort(-d, kind="stable")


def quantize_gptq_reordered(W, H, bits, group, dim, percdamp=0.01, static_groups=False):
    """GPTQ with activation reordering (Section 2.2, Appendix A.1).

    The columns of W (and rows/columns of H) are taken in the order of activation_order(H):
    the method is the plain one applied to W[:, perm] and H[perm][:, perm]; codes, the
    dequantized weights and the per-column errors are returned at the columns' original
    positions.

    dim == "ic": group statistics are dynamic as before (the g rows of the column being
    quantized, from the current weights); a column's scale and zero are stored at its original
    position, so the parameter layout [out/g, in] is unchanged.
    dim == "oc": only with static_groups=True (the hardware-efficient variant of Section 2.2):
    the parameters of every group of g consecutive original columns are fixed before anything
    is reordered or updated, from the original weights, and a column uses the parameters of
    the group it originally belongs to.
    Returns the same dict as quantize_gptq plus "perm".
    """
    Wf = np.asarray(W).astype(F32)
    out, inp = Wf.shape
    Hd, dead = damped_hessian(H, percdamp)
    perm = activation_order(H)
    Hp = Hd[np.ix_(perm, perm)]
    U = cholesky_inverse_factor(Hp)
    Wc = np.array(Wf[:, perm], dtype=np.float64)
    Wc[:, dead[perm]] = 0.0
    codes = np.zeros((out, inp), dtype=np.uint8)
    Q = np.zeros((out, inp), dtype=F32)
    Err = np.zeros((out, inp), dtype=np.float64)
    if dim == "oc":
        if not static_groups:
            raise ValueError("per-OC reordering is defined here only with static groups")
        assert inp % group == 0
        G0 = Wf.reshape(out, inp // group, group)
        S, Z, B = group_params(G0.min(axis=2), G0.max(axis=2), bits)
    else:
        assert out % group == 0
        S = np.zeros((out // group, inp), dtype=F32)
        Z = np.zeros((out // group, inp), dtype=F32)
    for i in range(inp):
        c0 = int(perm[i])                       # original position of the column quantized now
        w32 = Wc[:, i].astype(F32)
        if dim == "oc":
            se, ze, be = S[:, c0 // group], Z[:, c0 // group], B[:, c0 // group]
        else:
            col = w32.reshape(out // group, group)
            s, z, bad = group_params(col.min(axis=1), col.max(axis=1), bits)
            S[:, c0], Z[:, c0] = s, z
            se, ze, be = np.repeat(s, group), np.repeat(z, group), np.repeat(bad, group)
        c = encode(w32, se, ze, bits, be)
        q = dequant(c, se, ze)
        codes[:, c0], Q[:, c0] = c, q
        e = (Wc[:, i] - q.astype(np.float64)) / U[i, i]
        Err[:, c0] = e
        Wc[:, i:] -= np.outer(e, U[i, i:])
    return {"codes": codes, "scales": S.astype(np.float16), "zeros": Z.astype(np.float16),
            "Q": Q, "Err": Err, "loss": 0.5 * float(np.sum(Err * Err)), "perm": perm}


# ---------------------------------------------------------------------------
# Flows (Section 3.3, Appendix B).
# ---------------------------------------------------------------------------

def rtn_ada(W, H, bits, group):
    """Quantize twice (oc, ic) with RTN, score both, keep the lower error."""
    r = {d: quantize_rtn(W, bits, group, d) for d in ("oc", "ic")}
    W32 = np.asarray(W).astype(F32)
    err = {d: recon_error_trace(W32, r[d]["Q"], H) for d in ("oc", "ic")}
    best = select_dim(err["oc"], err["ic"])
    return best, err, r


def gptq_ada(W, H, bits, group, percdamp=0.01):
    """The paper's flow: choose the dimension with RTN, then run GPTQ in it."""
    best, err, _ = rtn_ada(W, H, bits, group)
    return best, err, quantize_gptq(W, H, bits, group, best, percdamp)


def gptq_ada_reordered(W, H, bits, group, percdamp=0.01):
    """The paper's final GPTQ design (Section 4.1; Appendix A.1): the dimension is chosen with RTN,
    then GPTQ runs in it with activation reordering: static groups if per-OC was chosen, plain
    reordering if per-IC was."""
    best, err, _ = rtn_ada(W, H, bits, group)
    return best, err, quantize_gptq_reordered(W, H, bits, group, best, percdamp, static_groups=(best == "oc"))


def gptq_both(W, H, bits, group, percdamp=0.01):
    """GPTQ in both dimensions, scored with the undamped H, lower error kept."""
    Hd, dead = damped_hessian(H, percdamp)
    U = cholesky_inverse_factor(Hd)
    r = {d: quantize_gptq(W, H, bits, group, d, percdamp, U=U, dead=dead) for d in ("oc", "ic")}
    W32 = np.asarray(W).astype(F32)
    err = {d: recon_error_trace(W32, r[d]["Q"], H) for d in ("oc", "ic")}
    return select_dim(err["oc"], err["ic"]), err, r


# ---------------------------------------------------------------------------
# Inference with the quantized weights (Section 4.5, Appendix D: the latency
# of a matrix-vector product with per-IC quantized weights, fp16 input and
# output).  What such a kernel computes has a plain definition: y = Q x with
# Q[o, i] = scale * (code - zero), the group parameters indexed as the
# grouping dimension says.  Any group size that divides the grouped extent
# is allowed here (Appendix D goes up to 2048).
# ---------------------------------------------------------------------------

def dequant_matvec(codes, scales, zeros, group, dim, x):
    """y[o] = sum_i scale * (code[o, i] - zero) * x[i] in binary64 (x, scales, zeros as given)."""
    Q = dequantize(codes, scales, zeros, group, dim).astype(np.float64)
    return Q @ np.asarray(x, dtype=np.float64)
