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
