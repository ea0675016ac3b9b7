"""CUDA reconstruction-error scorer and selection vs the oracle (through the C ABI).
Bar: errors within 1e-3 relative; the chosen dimension matches unless the two errors are
within 1e-4 relative of each other."""
import numpy as np
import pytest
import torch

from oracle import adadim_oracle as O
from paper_2309_15531_b200 import binding as B
from paper_2309_15531_b200 import inputs as I
from tests.helpers import q_to_np, status_tensor, to_np

pytestmark = pytest.mark.gpu


def _score_case(W, X, bits, group):
    Wn = to_np(W).astype(np.float32)
    Href = O.hessian(to_np(X))
    H = torch.as_tensor(Href.astype(np.float32), device="cuda")
    q_oc, q_ic = B.quantize_rtn(W, bits, group)
    st = status_tensor()
    err, chosen = B.score_select(W, H, bits, group, q_oc, q_ic, status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    e = err.cpu().numpy()
    Hn = to_np(H).astype(np.float64)
    ref = {}
    for name, q in (("oc", q_oc), ("ic", q_ic)):
        codes, s, z = q_to_np(q)
        Q = O.dequantize(codes, s, z, group, name)
        ref[name] = O.recon_error_trace(Wn, Q, Hn)
    print(f"score: gpu {e}, oracle {ref}")
    assert e[0] == pytest.approx(ref["oc"], rel=1e-3)
    assert e[1] == pytest.approx(ref["ic"], rel=1e-3)
    if abs(ref["oc"] - ref["ic"]) > 1e-4 * max(ref["oc"], ref["ic"]):
        assert B.DIM_NAMES[int(chosen.item())] == O.select_dim(ref["oc"], ref["ic"])
    return e, q_oc, q_ic, H


def test_small_fp32_layer():
    wl = I.workload_small()
    wspec, xspec = wl["layers"]["linear"]
    _score_case(I.make_weight(wspec, "cuda"), I.make_calib(xspec, "cuda"), 3, 128)


@pytest.mark.parametrize("out,inp,bits,group", [(1024, 768, 3, 128), (384, 320, 4, 64), (128, 64, 3, 32), (256, 256, 2, 64),
                                                (384, 128, 8, 128)])
def test_fp16_shapes(out, inp, bits, group):
    W = I.make_weight(I.WeightSpec(out, inp, "f16", 0.02, 0.001, seed=61), "cuda")
    X = I.make_calib(I.CalibSpec(2048, inp, "bf16", "normal", 4, 50.0, 100.0, seed=62), "cuda")
    e, q_oc, q_ic, H = _score_case(W, X, bits, group)
    # one dimension at a time gives the same number and +inf for the absent one
    e1, c1 = B.score_select(W, H, bits, group, q_oc, None)
    e2, c2 = B.score_select(W, H, bits, group, None, q_ic)
    torch.cuda.synchronize()
    assert e1[0].item() == e[0] and np.isinf(e1[1].item()) and int(c1.item()) == B.DIM_OC
    assert e2[1].item() == e[1] and np.isinf(e2[0].item()) and int(c2.item()) == B.DIM_IC


def test_sensitive_column_case_selects_ic_and_large_row_case_selects_oc():
    W = I.make_weight(I.WeightSpec(256, 256, "f32", 0.02, 0.0, seed=63), "cuda")
    xs = I.CalibSpec(512, 256, "f32", "normal", 3, 60.0, 60.0, seed=64)
    X = I.make_calib(xs, "cuda")
    ids, _ = I.outlier_channels(xs)
    W1 = W.clone(); W1[:, ids.cuda()] *= 0.1
    H = torch.zeros(256, 256, device="cuda"); B.hessian_accumulate(X, H)
    q_oc, q_ic = B.quantize_rtn(W1, 3, 128)
    _, chosen = B.score_select(W1, H, 3, 128, q_oc, q_ic)
    assert int(chosen.item()) == B.DIM_IC
    X2 = I.make_calib(I.CalibSpec(512, 256, "f32", "normal", 0, seed=65), "cuda")
    W2 = W.clone(); W2[[7, 130], :] *= 10.0
    H2 = torch.zeros(256, 256, device="cuda"); B.hessian_accumulate(X2, H2)
    q_oc, q_ic = B.quantize_rtn(W2, 3, 128)
    _, chosen = B.score_select(W2, H2, 3, 128, q_oc, q_ic)
    assert int(chosen.item()) == B.DIM_OC


def test_tie_gives_oc_and_nan_is_reported():
    W = torch.zeros(128, 128, dtype=torch.float16, device="cuda")
    H = torch.eye(128, device="cuda")
    q_oc, q_ic = B.quantize_rtn(W, 3, 128)
    st = status_tensor()
    err, chosen = B.score_select(W, H, 3, 128, q_oc, q_ic, status=st)
    assert err[0].item() == 0.0 and err[1].item() == 0.0 and int(chosen.item()) == B.DIM_OC
    H[3, 3] = float("nan")
    W[:, 3] = 0.013
    q_oc, q_ic = B.quantize_rtn(W, 3, 128)
    err, chosen = B.score_select(W, H, 3, 128, q_oc, q_ic, status=st)
    assert int(st.item()) == 8 and int(chosen.item()) == B.DIM_OC


def test_status_word_is_sticky_across_calls():
    """A device-side condition reported by one call survives later successful calls that are
    given the same status word: the caller may check once after a whole sequence."""
    W = torch.zeros(128, 128, dtype=torch.float16, device="cuda")
    W[:, 3] = 0.013
    Hbad = torch.eye(128, device="cuda")
    Hbad[3, 3] = float("nan")
    Hgood = torch.eye(128, device="cuda")
    q_oc, q_ic = B.quantize_rtn(W, 3, 128)
    st = status_tensor()
    B.score_select(W, Hbad, 3, 128, q_oc, q_ic, status=st)            # reports ADADIM_ERR_NUMERIC
    err, _ = B.score_select(W, Hgood, 3, 128, q_oc, q_ic, status=st)  # a clean call afterwards
    X = I.make_calib(I.CalibSpec(256, 128, "bf16", "normal", 0, seed=59), "cuda")
    B.hessian_accumulate(X, torch.zeros(128, 128, device="cuda"), st)
    B.quantize_gptq(W, Hgood, 3, 128, B.DIM_BOTH, status=st)
    torch.cuda.synchronize()
    assert np.isfinite(err.cpu().numpy()).all()
    assert int(st.item()) == 8
    st.zero_()                                                        # the caller clears it
    B.score_select(W, Hgood, 3, 128, q_oc, q_ic, status=st)
    assert int(st.item()) == 0


def test_workspace_too_small_is_refused():
    W = torch.zeros(128, 128, dtype=torch.float16, device="cuda")
    H = torch.eye(128, device="cuda")
    q_oc, q_ic = B.quantize_rtn(W, 3, 128)
    with pytest.raises(B.AdadimError) as e:
        B.score_select(W, H, 3, 128, q_oc, q_ic, workspace=torch.empty(1024, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 6
