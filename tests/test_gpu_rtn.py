"""CUDA RTN quantizer vs the oracle: codes, scales and zeros are bit-exact (called through the C ABI)."""
import numpy as np
import pytest
import torch

from oracle import adadim_oracle as O
from paper_2309_15531_b200 import binding as B
from paper_2309_15531_b200 import inputs as I
from tests.helpers import assert_rtn_equal, to_np

pytestmark = pytest.mark.gpu


def _check_both(W, bits, group):
    Wn = to_np(W).astype(np.float32)
    q_oc, q_ic = B.quantize_rtn(W, bits, group, B.DIM_BOTH)
    torch.cuda.synchronize()
    assert_rtn_equal(q_oc, O.quantize_rtn(Wn, bits, group, "oc"), f"oc b{bits} g{group}")
    assert_rtn_equal(q_ic, O.quantize_rtn(Wn, bits, group, "ic"), f"ic b{bits} g{group}")
    # single-dimension launches give the same tensors
    s_oc, _ = B.quantize_rtn(W, bits, group, B.DIM_OC)
    _, s_ic = B.quantize_rtn(W, bits, group, B.DIM_IC)
    torch.cuda.synchronize()
    assert torch.equal(s_oc.codes, q_oc.codes) and torch.equal(s_oc.scales, q_oc.scales)
    assert torch.equal(s_ic.codes, q_ic.codes) and torch.equal(s_ic.zeros, q_ic.zeros)


@pytest.mark.parametrize("bits", [3, 4])
@pytest.mark.parametrize("group", [32, 64, 128])
def test_small_fp32_layer(bits, group):
    wl = I.workload_small()
    W = I.make_weight(wl["layers"]["linear"][0], "cuda")
    _check_both(W, bits, group)


@pytest.mark.parametrize("bits", [2, 8])
@pytest.mark.parametrize("group,dtype", [(32, "f16"), (128, "f16"), (64, "f32"), (256, "f16"), (256, "f32")])
def test_two_and_eight_bit_codes(bits, group, dtype):
    """The ends of the precision range (the paper's INT3 / INT4 sit between them): 2-bit codes share a
    32-bit word sixteen at a time, 8-bit codes fill two words per eight weights."""
    W = I.make_weight(I.WeightSpec(512, 384 if group != 256 else 512, dtype, 0.02, 0.01, seed=76), "cuda")
    _check_both(W, bits, group)


@pytest.mark.parametrize("bits,group,out,inp", [(3, 32, 320, 224), (4, 64, 448, 192), (3, 128, 384, 640), (2, 32, 320, 224),
                                                (8, 32, 448, 160)])
def test_ragged_tiles_fp16(bits, group, out, inp):
    W = I.make_weight(I.WeightSpec(out, inp, "f16", 0.02, 0.01, seed=77), "cuda")
    _check_both(W, bits, group)


def test_row_pitch_larger_than_width():
    full = I.make_weight(I.WeightSpec(256, 512, "f16", 0.02, 0.0, seed=78), "cuda")
    W = full[:, :384]
    _check_both(W, 3, 128)


def test_degenerate_and_one_signed_groups():
    W = I.make_weight(I.WeightSpec(256, 256, "f32", 0.02, 0.0, seed=79), "cuda")
    W[0:128, 0:128] = 0.0                 # all-zero groups in both dimensions
    W[128:256, 0:128] = W[128:256, 0:128].abs() + 0.01      # one-signed
    W[0:128, 128:256] = -W[0:128, 128:256].abs() - 0.01
    W[200, 130] = 3.0e6                   # range overflows fp16
    W[5, 250] = 1e-9
    _check_both(W, 3, 128)
    _check_both(W, 4, 64)


def test_ties_round_to_even():
    W = torch.zeros(128, 128, device="cuda")
    W[:, 0], W[:, 1] = -3.0, 4.0
    W[:, 2], W[:, 3], W[:, 4], W[:, 5] = 0.5, 1.5, 2.5, -0.5
    q_oc, _ = B.quantize_rtn(W, 3, 128, B.DIM_OC)
    codes = q_oc.unpacked().cpu().numpy()
    assert list(codes[7, 2:6]) == [3, 5, 5, 3]
    _check_both(W, 3, 128)


def test_full_size_q_proj():
    wl = I.workload_qproj()
    W = I.make_weight(wl["layers"]["q_proj"][0], "cuda")
    _check_both(W, 3, 128)


def test_mlp70b_gate_shape_4bit():
    wl = I.workload_mlp70b()
    W = I.make_weight(wl["layers"]["gate_proj"][0], "cuda")
    Wn = to_np(W).astype(np.float32)
    q_oc, q_ic = B.quantize_rtn(W, 4, 128, B.DIM_BOTH)
    torch.cuda.synchronize()
    assert_rtn_equal(q_oc, O.quantize_rtn(Wn, 4, 128, "oc"), "oc")
    assert_rtn_equal(q_ic, O.quantize_rtn(Wn, 4, 128, "ic"), "ic")


def test_empty_and_bad_arguments():
    W = torch.zeros(0, 128, dtype=torch.float16, device="cuda")
    B.quantize_rtn(W, 3, 128, B.DIM_OC)                      # nothing to do, no error
    W = torch.zeros(128, 128, dtype=torch.float16, device="cuda")
    for bits, group, code in [(5, 128, 4), (3, 48, 4)]:
        with pytest.raises(B.AdadimError) as e:
            B.quantize_rtn(W, bits, group, B.DIM_BOTH)
        assert e.value.status == code
    with pytest.raises(B.AdadimError) as e:                  # in % group != 0
        B.quantize_rtn(torch.zeros(128, 96, dtype=torch.float16, device="cuda"), 3, 64, B.DIM_OC)
    assert e.value.status == 2
    with pytest.raises(B.AdadimError) as e:                  # misaligned rows
        B.quantize_rtn(torch.zeros(128, 132, dtype=torch.float16, device="cuda")[:, 4:], 3, 128, B.DIM_OC)
    assert e.value.status == 5


# ----------------------------------------------------------------------------- g = 256 (Section 4.4 sweep)

@pytest.mark.parametrize("bits", [3, 4])
@pytest.mark.parametrize("dtype", ["f16", "f32"])
def test_group_256(bits, dtype):
    W = I.make_weight(I.WeightSpec(768, 1024, dtype, 0.02, 0.005, seed=83), "cuda")
    W[3, :] *= 15.0
    W[:, 700] *= 25.0
    _check_both(W, bits, 256)


def test_group_256_special_groups_and_partial_tiles():
    W = I.make_weight(I.WeightSpec(512, 768, "f32", 0.02, 0.0, seed=84), "cuda")
    W[0:256, 0:256] = 0.0                                   # all-zero groups in both dimensions
    W[256:512, 0:256] = W[256:512, 0:256].abs() + 0.01      # one-signed
    W[300, 600] = 3.0e6                                     # range overflows fp16
    _check_both(W, 3, 256)
    # per-IC only needs out % 256 == 0: the column tiles may be partial (in % 32 == 0)
    V = I.make_weight(I.WeightSpec(256, 416, "f16", 0.02, 0.0, seed=85), "cuda")
    _, q_ic = B.quantize_rtn(V, 4, 256, B.DIM_IC)
    torch.cuda.synchronize()
    assert_rtn_equal(q_ic, O.quantize_rtn(to_np(V).astype(np.float32), 4, 256, "ic"), "ic b4 g256 partial")


def test_group_256_selection_flow():
    """RTN in both dimensions at g = 256, scored and selected: the setting where the paper reports
    the largest gain of the adaptive choice over plain RTN (Section 4.4)."""
    from paper_2309_15531_b200 import flows
    W = I.make_weight(I.WeightSpec(512, 512, "f16", 0.02, 0.0, seed=86), "cuda")
    X = I.make_calib(I.CalibSpec(2048, 512, "bf16", "normal", 3, 50.0, 100.0, seed=87), "cuda")
    W[:, :8] *= 0.1
    Hn = O.hessian(to_np(X)).astype(np.float32)
    dim, err, _ = flows.rtn_ada(W, torch.as_tensor(Hn, device="cuda"), 3, 256)
    torch.cuda.synchronize()
    best, ref, _ = O.rtn_ada(to_np(W).astype(np.float32), Hn.astype(np.float64), 3, 256)
    assert B.DIM_NAMES[dim] == best
    assert err[0].item() == pytest.approx(ref["oc"], rel=1e-3) and err[1].item() == pytest.approx(ref["ic"], rel=1e-3)


def test_gptq_group_256_needs_whole_pairs_of_slabs_and_blocks():
    """GPTQ at g = 256 works on pairs of its 128-row slabs and 128-column blocks: shapes that are
    multiples of 128 but not of 256 are refused on the host."""
    H = 2.0 * torch.eye(384, device="cuda")
    W = I.make_weight(I.WeightSpec(256, 384, "f16", 0.02, 0.0, seed=88), "cuda")
    with pytest.raises(B.AdadimError) as e:
        B.quantize_gptq(W, H, 3, 256, B.DIM_BOTH)
    assert e.value.status == 2
