"""The dequantizing matrix-vector product on the GPU against the oracle's y = Q x (through the C ABI).
Bar (derived from the kernel's arithmetic): the sums are exact integers against a fixed-point image of
a = scale * x that is within 2^-20 of the group's largest |a| for every column, the two binary32 sums
(codes part, zero-point part) carry 2^-22 of their magnitudes, and the result is rounded to fp16 once:
|y - y_ref| <= 2^-10 |y_ref| + 2^-20 max_i|a_i| sum_i code[o,i] + 2^-21 (sum_i |a_i| code[o,i] + sum_i |a_i| zero_i).
A misplaced column, piece or row shows up at the size of y itself, far outside this."""
import numpy as np
import pytest
import torch

from oracle import adadim_oracle as O
from paper_2309_15531_b200 import binding as B
from paper_2309_15531_b200 import inputs as I
from tests.helpers import q_to_np, to_np

pytestmark = pytest.mark.gpu


def _check(codes_packed, scales, zeros, codes_np, out, inp, bits, group, x):
    y = B.dequant_gemv(codes_packed, scales, zeros, bits, group, x)
    torch.cuda.synchronize()
    s_np, z_np, x_np = scales.cpu().numpy(), zeros.cpu().numpy(), x.cpu().numpy()
    ref = O.dequant_matvec(codes_np, s_np, z_np, group, "ic", x_np)
    a = np.abs(s_np.astype(np.float64) * x_np.astype(np.float64)[None, :])            # [out/g, in]
    ae = np.repeat(a, group, axis=0)
    c = codes_np.astype(np.float64)
    tol = (2.0 ** -10 * np.abs(ref) + 2.0 ** -20 * np.repeat(a.max(axis=1), group) * c.sum(axis=1) +
           2.0 ** -21 * ((ae * c).sum(axis=1) + np.repeat((a * z_np.astype(np.float64)).sum(axis=1), group)))
    err = np.abs(y.double().cpu().numpy() - ref)
    print(f"gemv {out}x{inp} b{bits} g{group}: max err / tol = {float(np.max(err / np.maximum(tol, 1e-30))):.3f}")
    assert np.all(err <= tol)


@pytest.mark.parametrize("bits,group,out,inp", [(4, 128, 256, 512), (3, 128, 256, 512), (3, 32, 96, 128), (4, 64, 192, 384),
                                                (3, 256, 512, 1152), (4, 16, 48, 128)])
def test_gemv_on_library_quantized_layers(bits, group, out, inp):
    """Layers quantized per-IC by this library's own RTN kernel, vector with a few large entries."""
    W = I.make_weight(I.WeightSpec(out, inp, "f16", 0.02, 0.001, seed=91), "cuda")
    g = torch.Generator(device="cuda").manual_seed(92)
    x = torch.randn(inp, device="cuda", generator=g)
    x[::97] *= 60.0
    x = x.half()
    if group in (32, 64, 128, 256):
        _, q = B.quantize_rtn(W, bits, group, B.DIM_IC)
        codes_np, _, _ = q_to_np(q)
        _check(q.codes, q.scales, q.zeros, codes_np, out, inp, bits, group, x)
    else:                                                  # a group size only the oracle quantizes
        r = O.quantize_rtn(to_np(W).astype(np.float32), bits, group, "ic")
        packed = torch.as_tensor(O.pack_codes(r["codes"], bits).view(np.int32), device="cuda")
        _check(packed, torch.as_tensor(r["scales"], device="cuda"), torch.as_tensor(r["zeros"], device="cuda"),
               r["codes"], out, inp, bits, group, x)


@pytest.mark.parametrize("bits,group", [(3, 2048), (4, 512)])
def test_gemv_large_groups_and_split_columns(bits, group):
    """Group sizes of Appendix D beyond what the quantizer kernels take (parameters from the oracle's
    quantizer), on a shape whose columns are split over several CTAs."""
    out, inp = 4096, 3072
    W = I.make_weight(I.WeightSpec(out, inp, "f16", 0.02, 0.001, seed=93), "cpu")
    r = O.quantize_rtn(W.float().numpy(), bits, group, "ic")
    packed = torch.as_tensor(O.pack_codes(r["codes"], bits).view(np.int32), device="cuda")
    x = (torch.randn(inp, generator=torch.Generator().manual_seed(94)) * 0.5).half().cuda()
    _check(packed, torch.as_tensor(r["scales"], device="cuda"), torch.as_tensor(r["zeros"], device="cuda"),
           r["codes"], out, inp, bits, group, x)


def test_gemv_argument_checks():
    q = B.QTensor(128, 128, 3, 128, B.DIM_IC)
    x = torch.zeros(128, dtype=torch.float16, device="cuda")
    with pytest.raises(B.AdadimError) as e:
        B.dequant_gemv(q.codes, q.scales, q.zeros, 5, 128, x)
    assert e.value.status == 4
    with pytest.raises(B.AdadimError) as e:
        B.dequant_gemv(q.codes, q.scales, q.zeros, 3, 96, x)      # 96 does not divide 128 rows
    assert e.value.status == 2
    with pytest.raises(B.AdadimError) as e:
        B.dequant_gemv(q.codes, q.scales, q.zeros, 3, 128, x, workspace=torch.empty(256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 6
    y = B.dequant_gemv(q.codes, q.scales, q.zeros, 3, 128, x)      # all-zero layer and vector
    assert float(y.abs().max().item()) == 0.0
