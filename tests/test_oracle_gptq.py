"""Pins for the oracle's Hessian, scorer, Cholesky-inverse factor and GPTQ (CPU only)."""
import math

import numpy as np
import pytest

from oracle import adadim_oracle as O

RNG = np.random.default_rng(4321)


def _layer(out, inp, n_tok, outliers=(3, 17), scale=40.0):
    W = (RNG.standard_normal((out, inp)) * 0.02).astype(np.float32)
    X = RNG.standard_normal((n_tok, inp)).astype(np.float32)
    for c in outliers:
        X[:, c] *= scale
    return W, X


# ----------------------------------------------------------------------------- Hessian

def test_hessian_entries_by_exact_summation():
    X = RNG.standard_normal((37, 9)).astype(np.float32)
    H = O.hessian(X)
    for i in range(9):
        for j in range(9):
            ref = 2.0 * math.fsum(float(X[t, i]) * float(X[t, j]) for t in range(37))
            assert H[i, j] == pytest.approx(ref, rel=1e-13, abs=1e-13)
    assert np.array_equal(H, H.T)


def test_hessian_freivalds_and_chunk_additivity():
    X = RNG.standard_normal((500, 64)).astype(np.float32)
    H = O.hessian(X)
    v = RNG.standard_normal(64)
    assert np.allclose(H @ v, 2.0 * (X.T.astype(np.float64) @ (X.astype(np.float64) @ v)), rtol=1e-12)
    assert np.allclose(H, O.hessian(X[:123]) + O.hessian(X[123:]), rtol=1e-12, atol=1e-12)


# ----------------------------------------------------------------------------- scorer

def test_trace_form_equals_layer_output_form():
    """1/2 trace((W-Q) H (W-Q)^T) == ||X W^T - X Q^T||_F^2   (Eq. 1, squared)."""
    W, X = _layer(64, 128, 300)
    H = O.hessian(X)
    for dim in ("oc", "ic"):
        Q = O.quantize_rtn(W, 3, 32, dim)["Q"]
        e_tr = O.recon_error_trace(W, Q, H)
        e_ex = O.recon_error_explicit(W, Q, X)
        Y0 = X.astype(np.float64) @ W.astype(np.float64).T          # layer(x) with W
        Y1 = X.astype(np.float64) @ Q.astype(np.float64).T          # layer(x) with Q
        e_fwd = float(np.sum((Y0 - Y1) ** 2))
        assert e_tr == pytest.approx(e_fwd, rel=1e-10)
        assert e_ex == pytest.approx(e_fwd, rel=1e-10)


def test_selection_rule():
    assert O.select_dim(1.0, 0.5) == "ic"
    assert O.select_dim(0.5, 1.0) == "oc"
    assert O.select_dim(1.0, 1.0) == "oc"            # ties keep the first-evaluated dim
    W, X = _layer(128, 128, 400, outliers=(5, 77), scale=60.0)
    H = O.hessian(X)
    best, err, _ = O.rtn_ada(W, H, 3, 128)
    best2, err2, _ = O.rtn_ada(W, 7.5 * H, 3, 128)   # argmin invariant under H -> aH
    assert best == best2
    assert err2["oc"] == pytest.approx(7.5 * err["oc"], rel=1e-12)


def test_grouping_dimension_that_isolates_the_sensitive_weights_wins():
    """Mechanism of Section 3.2: a group shares one step size, so the better dimension is the
    one whose groups do not mix weights of very different magnitude where the activations
    are large.  Small-magnitude input channels that carry activation outliers get their own
    (fine) step under per-IC grouping; a few large-magnitude rows, with no activation
    outliers, inflate only their own steps under per-OC grouping."""
    W, X = _layer(256, 256, 512, outliers=(10, 100, 200), scale=60.0)
    W[:, [10, 100, 200]] *= 0.1
    best, err, _ = O.rtn_ada(W, O.hessian(X), 3, 128)
    assert best == "ic" and err["ic"] < 0.25 * err["oc"]
    W, X = _layer(256, 256, 512, outliers=(), scale=1.0)
    W[[7, 130], :] *= 10.0
    best, err, _ = O.rtn_ada(W, O.hessian(X), 3, 128)
    assert best == "oc" and err["oc"] < 0.5 * err["ic"]


# ----------------------------------------------------------------------------- factor

def test_cholesky_inverse_factor_definition_and_reverse_identity():
    _, X = _layer(8, 48, 200)
    Hd, dead = O.damped_hessian(O.hessian(X), 0.01)
    assert not dead.any()
    U = O.cholesky_inverse_factor(Hd)
    assert np.allclose(np.tril(U, -1), 0) and np.all(np.diag(U) > 0)
    assert np.allclose(U.T @ U @ Hd, np.eye(48), atol=1e-9)
    assert np.allclose(U @ Hd @ U.T, np.eye(48), atol=1e-9)
    # independent route: factor the index-reversed matrix, invert the triangle, reverse back
    P = np.eye(48)[::-1]
    L = np.linalg.cholesky(P @ Hd @ P)
    U2 = P @ np.linalg.inv(L) @ P
    assert np.allclose(U, U2, rtol=1e-9, atol=1e-12)


def test_damping_and_dead_columns():
    H = np.diag([4.0, 0.0, 2.0, 6.0])
    Hd, dead = O.damped_hessian(H, 0.01)
    assert list(dead) == [False, True, False, False]
    lam = 0.01 * (4 + 1 + 2 + 6) / 4
    assert np.allclose(np.diag(Hd), [4 + lam, 1 + lam, 2 + lam, 6 + lam])
    W = (RNG.standard_normal((4, 4)) * 0.1).astype(np.float32)
    r = O.quantize_gptq(W, H, 3, 4, "oc")
    assert np.all(r["Q"][:, 1] == 0)                 # dead column is quantized as zero


# ----------------------------------------------------------------------------- GPTQ

@pytest.mark.parametrize("dim", ["oc", "ic"])
@pytest.mark.parametrize("bits,group", [(3, 32), (4, 64)])
def test_identity_hessian_reduces_to_rtn(dim, bits, group):
    W = (RNG.standard_normal((128, 192)) * 0.02).astype(np.float32)
    r = O.quantize_gptq(W, 3.0 * np.eye(192), bits, group, dim)
    t = O.quantize_rtn(W, bits, group, dim)
    for k in ("codes", "scales", "zeros", "Q"):
        assert np.array_equal(r[k], t[k]), k


@pytest.mark.parametrize("dim", ["oc", "ic"])
def test_error_factor_identities(dim):
    """W - Q = Err U  and  ||Err||^2 = trace(D Hd D^T): consequences of U Hd U^T = I."""
    W, X = _layer(64, 96, 300)
    H = O.hessian(X)
    Hd, _ = O.damped_hessian(H, 0.01)
    U = O.cholesky_inverse_factor(Hd)
    r = O.quantize_gptq(W, H, 3, 32, dim)
    D = W.astype(np.float64) - r["Q"].astype(np.float64)
    assert np.allclose(D, r["Err"] @ U, atol=1e-12)
    assert float(np.sum(r["Err"] ** 2)) == pytest.approx(float(np.sum((D @ Hd) * D)), rel=1e-9)
    assert r["loss"] == pytest.approx(0.5 * float(np.sum((D @ Hd) * D)), rel=1e-9)


def _gptq_by_coordinate_elimination(W, Hd, bits, group, dim):
    """Independent statement of the same greedy procedure: keep the inverse Hessian of the
    not-yet-quantized coordinates explicitly, and after fixing coordinate i remove it by a
    rank-one downdate (the optimal-brain-surgeon update), in plain loops."""
    Wc = W.astype(np.float64).copy()
    out, inp = Wc.shape
    Hinv = np.linalg.inv(Hd)
    codes = np.zeros((out, inp), np.uint8)
    params = None
    for i in range(inp):
        w32 = Wc[:, i].astype(np.float32)
        if dim == "oc":
            if i % group == 0:
                blk = Wc[:, i:i + group].astype(np.float32)
                params = O.group_params(blk.min(1), blk.max(1), bits)
            s, z, bad = params
        else:
            col = w32.reshape(out // group, group)
            s, z, bad = (np.repeat(a, group) for a in O.group_params(col.min(1), col.max(1), bits))
        c = O.encode(w32, s, z, bits, bad)
        codes[:, i] = c
        q = O.dequant(c, s, z).astype(np.float64)
        d = Hinv[i, i]
        for o in range(out):
            Wc[o, i:] -= (Wc[o, i] - q[o]) / d * Hinv[i, i:]
        Hinv = Hinv - np.outer(Hinv[:, i], Hinv[i, :]) / d
    return codes


@pytest.mark.parametrize("dim", ["oc", "ic"])
def test_matches_coordinate_elimination_form(dim):
    W, X = _layer(32, 48, 200, outliers=(3,), scale=20.0)
    H = O.hessian(X)
    Hd, _ = O.damped_hessian(H, 0.01)
    r = O.quantize_gptq(W, H, 3, 16, dim)
    ref = _gptq_by_coordinate_elimination(W, Hd, 3, 16, dim)
    assert np.array_equal(r["codes"], ref)


@pytest.mark.parametrize("dim", ["oc", "ic"])
def test_codes_are_nearest_level_of_current_weight(dim):
    W, X = _layer(32, 64, 200)
    H = O.hessian(X)
    Hd, _ = O.damped_hessian(H, 0.01)
    U = O.cholesky_inverse_factor(Hd)
    g = 16
    r = O.quantize_gptq(W, H, 3, g, dim)
    cur = r["Q"].astype(np.float64) + r["Err"] * np.diag(U)[None, :]     # weight when quantized
    S, Z = r["scales"].astype(np.float64), r["zeros"].astype(np.float64)
    for o in range(32):
        for i in range(64):
            s, z = (S[o, i // g], Z[o, i // g]) if dim == "oc" else (S[o // g, i], Z[o // g, i])
            best = min(range(8), key=lambda c: abs(cur[o, i] - s * (c - z)))
            assert r["codes"][o, i] == best


def test_rows_and_slabs_are_independent():
    W, X = _layer(64, 64, 200)
    H = O.hessian(X)
    full_oc = O.quantize_gptq(W, H, 3, 32, "oc")
    part_oc = O.quantize_gptq(W[10:20], H, 3, 32, "oc")
    assert np.array_equal(full_oc["codes"][10:20], part_oc["codes"])
    full_ic = O.quantize_gptq(W, H, 3, 32, "ic")
    part_ic = O.quantize_gptq(W[32:64], H, 3, 32, "ic")
    assert np.array_equal(full_ic["codes"][32:64], part_ic["codes"])
    assert np.array_equal(full_ic["scales"][1:2], part_ic["scales"])


def test_gptq_lowers_the_layer_output_error():
    W, X = _layer(128, 128, 600, outliers=(7, 90), scale=30.0)
    H = O.hessian(X)
    for dim in ("oc", "ic"):
        e_rtn = O.recon_error_trace(W, O.quantize_rtn(W, 3, 128, dim)["Q"], H)
        e_gptq = O.recon_error_trace(W, O.quantize_gptq(W, H, 3, 128, dim)["Q"], H)
        assert e_gptq < e_rtn


def test_flows():
    W, X = _layer(128, 128, 400, outliers=(5, 77), scale=60.0)
    H = O.hessian(X)
    best, err, r = O.gptq_ada(W, H, 3, 128)
    assert best == O.rtn_ada(W, H, 3, 128)[0]
    assert np.array_equal(r["codes"], O.quantize_gptq(W, H, 3, 128, best)["codes"])
    b2, e2, r2 = O.gptq_both(W, H, 3, 128)
    assert b2 == O.select_dim(e2["oc"], e2["ic"])
    assert np.array_equal(r2["ic"]["codes"], O.quantize_gptq(W, H, 3, 128, "ic")["codes"])


# ----------------------------------------------------------------------------- activation reordering

def test_activation_order_is_descending_and_stable():
    H = np.diag([3.0, 9.0, 0.0, 9.0, 0.5, 1.0])
    # the dead column counts as 1 (its diagonal is set to 1 before anything else), ties keep their order
    assert list(O.activation_order(H)) == [1, 3, 0, 2, 5, 4]
    _, X = _layer(8, 64, 300, outliers=(3, 17), scale=40.0)
    perm = O.activation_order(O.hessian(X))
    assert set(perm[:2]) == {3, 17}                   # the salient channels are quantized first
    assert sorted(perm) == list(range(64))


@pytest.mark.parametrize("dim", ["oc", "ic"])
def test_uncorrelated_channels_reduce_to_rtn_in_any_order(dim):
    """With a diagonal Hessian nothing propagates (U is diagonal), so every column is rounded as it
    stands whatever the order: the result must be RTN's, at the original positions."""
    W = (RNG.standard_normal((64, 96)) * 0.02).astype(np.float32)
    H = np.diag(RNG.uniform(0.5, 50.0, 96))
    r = O.quantize_gptq_reordered(W, H, 3, 32, dim, static_groups=(dim == "oc"))
    assert not np.array_equal(r["perm"], np.arange(96))
    t = O.quantize_rtn(W, 3, 32, dim)
    for k in ("codes", "scales", "zeros", "Q"):
        assert np.array_equal(r[k], t[k]), k


def test_reordered_ic_is_the_plain_method_on_the_permuted_problem():
    W, X = _layer(64, 96, 300, outliers=(5, 40), scale=25.0)
    H = O.hessian(X)
    r = O.quantize_gptq_reordered(W, H, 3, 32, "ic")
    perm = r["perm"]
    p = O.quantize_gptq(np.ascontiguousarray(W[:, perm]), H[np.ix_(perm, perm)], 3, 32, "ic")
    assert np.array_equal(r["codes"][:, perm], p["codes"])
    assert np.array_equal(r["scales"][:, perm].view(np.uint16), p["scales"].view(np.uint16))
    assert np.array_equal(r["zeros"][:, perm].view(np.uint16), p["zeros"].view(np.uint16))
    assert np.array_equal(r["Q"][:, perm], p["Q"])
    assert r["loss"] == pytest.approx(p["loss"], rel=1e-12)
    # and reordering changes the outcome (otherwise the test above proves nothing)
    assert not np.array_equal(r["codes"], O.quantize_gptq(W, H, 3, 32, "ic")["codes"])


def _elimination_in_order(W, Hd, bits, group, dim, order, static=None):
    """Greedy coordinate elimination in the ORIGINAL index space: coordinates are fixed in the
    given order, the inverse Hessian of the coordinates still free is kept explicitly (rows and
    columns of fixed ones become zero through the downdate), no array is ever permuted."""
    Wc = W.astype(np.float64).copy()
    out, inp = Wc.shape
    Hinv = np.linalg.inv(Hd)
    codes = np.zeros((out, inp), np.uint8)
    for c0 in order:
        w32 = Wc[:, c0].astype(np.float32)
        if dim == "oc":
            s, z, bad = (a[:, c0 // group] for a in static)
        else:
            col = w32.reshape(out // group, group)
            s, z, bad = (np.repeat(a, group) for a in O.group_params(col.min(1), col.max(1), bits))
        c = O.encode(w32, s, z, bits, bad)
        codes[:, c0] = c
        q = O.dequant(c, s, z).astype(np.float64)
        d = Hinv[c0, c0]
        Wc -= np.outer((Wc[:, c0] - q) / d, Hinv[c0, :])
        Hinv = Hinv - np.outer(Hinv[:, c0], Hinv[c0, :]) / d
    return codes


@pytest.mark.parametrize("dim", ["oc", "ic"])
def test_reordered_matches_elimination_in_original_coordinates(dim):
    W, X = _layer(32, 48, 200, outliers=(3, 30), scale=20.0)
    H = O.hessian(X)
    Hd, _ = O.damped_hessian(H, 0.01)
    order = O.activation_order(H)
    static = None
    if dim == "oc":
        G0 = W.reshape(32, 3, 16)
        static = O.group_params(G0.min(2), G0.max(2), 3)
    r = O.quantize_gptq_reordered(W, H, 3, 16, dim, static_groups=(dim == "oc"))
    assert np.array_equal(r["codes"], _elimination_in_order(W, Hd, 3, 16, dim, order, static))


@pytest.mark.parametrize("dim", ["oc", "ic"])
def test_reordered_loss_identity_and_static_parameters(dim):
    W, X = _layer(64, 96, 300, outliers=(5, 40), scale=25.0)
    H = O.hessian(X)
    Hd, _ = O.damped_hessian(H, 0.01)
    r = O.quantize_gptq_reordered(W, H, 3, 32, dim, static_groups=(dim == "oc"))
    D = W.astype(np.float64) - r["Q"].astype(np.float64)
    assert r["loss"] == pytest.approx(0.5 * float(np.sum((D @ Hd) * D)), rel=1e-9)
    assert np.array_equal(O.dequantize(r["codes"], r["scales"], r["zeros"], 32, dim), r["Q"])
    if dim == "oc":                                   # static groups: the parameters are RTN's
        t = O.quantize_rtn(W, 3, 32, "oc")
        assert np.array_equal(r["scales"].view(np.uint16), t["scales"].view(np.uint16))
        assert np.array_equal(r["zeros"].view(np.uint16), t["zeros"].view(np.uint16))
    with pytest.raises(ValueError):
        O.quantize_gptq_reordered(W, H, 3, 32, "oc", static_groups=False)


def test_reordered_flow_uses_the_rtn_choice():
    W, X = _layer(128, 128, 400, outliers=(5, 77), scale=60.0)
    H = O.hessian(X)
    best, err, r = O.gptq_ada_reordered(W, H, 3, 128)
    assert best == O.rtn_ada(W, H, 3, 128)[0]
    ref = O.quantize_gptq_reordered(W, H, 3, 128, best, static_groups=(best == "oc"))
    assert np.array_equal(r["codes"], ref["codes"])
