"""Pins of the oracle's dequantized matrix-vector product (CPU only; Section 4.5, Appendix D)."""
import numpy as np

from oracle import adadim_oracle as O


def _case(out, inp, bits, group, dim, seed):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((out, inp)) * 0.02).astype(np.float32)
    r = O.quantize_rtn(W, bits, group, dim)
    x = rng.standard_normal(inp).astype(np.float16)
    return W, r, x


def test_matches_an_element_by_element_loop_in_both_dimensions():
    for dim, out, inp, g in (("ic", 8, 6, 4), ("oc", 6, 8, 4), ("ic", 16, 5, 16)):
        W, r, x = _case(out, inp, 3, g, dim, 7)
        y = O.dequant_matvec(r["codes"], r["scales"], r["zeros"], g, dim, x)
        for o in range(out):
            acc = 0.0
            for i in range(inp):
                k = (o, i // g) if dim == "oc" else (o // g, i)
                acc += float(r["scales"][k]) * (float(r["codes"][o, i]) - float(r["zeros"][k])) * float(x[i])
            assert abs(acc - y[o]) <= 1e-12 * max(1.0, abs(acc))


def test_per_ic_of_w_is_per_oc_of_w_transposed():
    """Groups along the rows of W are groups along the columns of W^T: with x = e_j the product
    returns column j of Q, which must equal row j of the per-OC dequantization of W^T."""
    W, r, _ = _case(64, 32, 4, 32, "ic", 11)
    rt = O.quantize_rtn(W.T.copy(), 4, 32, "oc")
    for j in (0, 5, 31):
        e = np.zeros(32, dtype=np.float16); e[j] = 1
        col = O.dequant_matvec(r["codes"], r["scales"], r["zeros"], 32, "ic", e)
        assert np.array_equal(col, rt["Q"][j].astype(np.float64))


def test_unit_scales_reduce_to_the_integer_product_and_error_bound_holds():
    rng = np.random.default_rng(3)
    codes = rng.integers(0, 16, size=(32, 48)).astype(np.uint8)
    ones = np.ones((1, 48), dtype=np.float16)
    x = rng.integers(-4, 5, size=48).astype(np.float16)
    y = O.dequant_matvec(codes, ones, 0 * ones, 32, "ic", x)
    assert np.array_equal(y, codes.astype(np.int64) @ x.astype(np.int64))
    # |W x - Q x| <= sum_i (s_i / 2) |x_i| for weights inside their group's range
    W, r, x = _case(128, 96, 3, 128, "ic", 5)
    y = O.dequant_matvec(r["codes"], r["scales"], r["zeros"], 128, "ic", x)
    bound = (0.5 * r["scales"].astype(np.float64)[0] * np.abs(x.astype(np.float64))).sum() * (1 + 1e-3)
    assert np.all(np.abs(W.astype(np.float64) @ x.astype(np.float64) - y) <= bound)
    # a large group (Appendix D uses up to 2048) is accepted
    W, r, x = _case(2048, 8, 4, 2048, "ic", 9)
    assert O.dequant_matvec(r["codes"], r["scales"], r["zeros"], 2048, "ic", x).shape == (2048,)
