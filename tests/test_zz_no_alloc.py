"""The allocation-free scorer entry point (adadim_score_select_static) against the regular one.

It serves callers that cannot allocate device memory (a process whose memory is fully
committed, a plugin without an allocator, a path that cannot afford an allocation's
synchronisation): the library's built-in scratch array replaces the workspace argument.  The
two entry points run the same kernels, so their results must agree to the scorer's own
tolerance (1e-3 relative; in practice they are identical), and both must agree with the CPU
oracle's errors.  Calls in a row on different layers (one of them with group size 256, which
both entry points accept through one shared argument check) show that what one call leaves in
the shared array does not leak into the next, and the device's free memory is the same before
and after a call once the array is resident.
This file is collected last so that a failure here cannot hide the other tests' results.
"""
import numpy as np
import pytest
import torch

from oracle import adadim_oracle as O
from paper_2309_15531_b200 import binding as B
from paper_2309_15531_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _layer(out, inp, seed, bits, group):
    W = I.make_weight(I.WeightSpec(out, inp, "f16", 0.02, 0.001, seed=seed), "cuda")
    X = I.make_calib(I.CalibSpec(1024, inp, "bf16", "normal", 3, 50.0, 100.0, seed=seed + 1), "cuda")
    H = torch.zeros(inp, inp, device="cuda")
    B.hessian_accumulate(X, H)
    q_oc, q_ic = B.quantize_rtn(W, bits, group)
    return W, H, q_oc, q_ic


def test_static_scratch_matches_workspace_version_on_two_calls_in_a_row():
    assert B.static_scratch_bytes() == 16 << 20
    cases = [(1024, 1024, 7101, 3, 128), (384, 512, 7201, 4, 64), (512, 768, 7301, 4, 256)]   # the first takes a quarter of the array
    layers = [_layer(*c) for c in cases]
    refs = []
    for (out, inp, _, bits, group), (W, H, q_oc, q_ic) in zip(cases, layers):
        assert B.workspace_bytes(B.WS_SCORE, out, inp) <= B.static_scratch_bytes()
        refs.append(B.score_select(W, H, bits, group, q_oc, q_ic))
    torch.cuda.synchronize()
    err = [torch.zeros(2, dtype=torch.float64, device="cuda") for _ in cases]
    chosen = [torch.full((1,), -1, dtype=torch.int32, device="cuda") for _ in cases]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for k, ((out, inp, _, bits, group), (W, H, q_oc, q_ic)) in enumerate(zip(cases, layers)):
        B.score_select_static(W, H, bits, group, q_oc, q_ic, err[k], chosen[k], status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for k, (out, inp, _, bits, group) in enumerate(cases):
        ref_err, ref_chosen = refs[k]
        W, H, _, _ = layers[k]
        Wn = W.float().cpu().numpy()
        H64 = H.double().cpu().numpy()
        for d, name in enumerate(("oc", "ic")):
            assert err[k][d].item() == pytest.approx(ref_err[d].item(), rel=1e-3)
            e_oracle = O.recon_error_trace(Wn, O.quantize_rtn(Wn, bits, group, name)["Q"], H64)
            assert err[k][d].item() == pytest.approx(e_oracle, rel=1e-3)
        assert int(chosen[k].item()) == int(ref_chosen.item())
    # the array is resident now: a further call changes nothing in the device's free memory
    free_before, _ = torch.cuda.mem_get_info()
    W, H, q_oc, q_ic = layers[0]
    B.score_select_static(W, H, cases[0][3], cases[0][4], q_oc, q_ic, err[0], chosen[0], status)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before


def test_layers_beyond_the_built_in_scratch_are_refused():
    W = torch.zeros(2048, 2048, dtype=torch.float16, device="cuda")
    H = torch.eye(2048, device="cuda")
    q_oc, q_ic = B.quantize_rtn(W, 3, 128)
    err = torch.zeros(2, dtype=torch.float64, device="cuda")
    chosen = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert B.workspace_bytes(B.WS_SCORE, 2048, 2048) > B.static_scratch_bytes()
    with pytest.raises(B.AdadimError) as e:
        B.score_select_static(W, H, 3, 128, q_oc, q_ic, err, chosen)
    assert e.value.status == 6
