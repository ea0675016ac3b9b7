"""CUDA Hessian accumulation vs the oracle (through the C ABI).

Tolerance.  bf16 x bf16 products are exact in fp32; the only error is the fp32 accumulation
over the tokens.  Entries are compared relative to sqrt(H_ii H_jj) (the Cauchy-Schwarz bound on
|H_ij|), with TOL = 1e-4: far below the 1e-3 allowed on reconstruction errors, far above
fp32 accumulation noise at these token counts.
"""
import numpy as np
import pytest
import torch

from oracle import adadim_oracle as O
from paper_2309_15531_b200 import binding as B
from paper_2309_15531_b200 import inputs as I
from tests.helpers import status_tensor, to_np

pytestmark = pytest.mark.gpu
TOL = 1e-4


def _norm_err(H, Href):
    d = np.sqrt(np.diag(Href))
    scale = np.outer(d, d) + 1e-30
    return float(np.max(np.abs(H - Href) / scale))


@pytest.mark.parametrize("tensor_cores", [True, False])
def test_small_fp32_layer(tensor_cores):
    """fp32 activations (configuration 1): on the tensor cores through three exact bf16 pieces, and
    by the plain multiply-add kernel that serves callers without a workspace."""
    wl = I.workload_small()
    X = I.make_calib(wl["layers"]["linear"][1], "cuda")
    H = torch.zeros(512, 512, device="cuda")
    st = status_tensor()
    B.hessian_accumulate(X, H, st, tensor_cores=tensor_cores)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    Href = O.hessian(to_np(X))
    e = _norm_err(to_np(H).astype(np.float64), Href)
    print(f"hessian fp32 X, tensor cores {tensor_cores}: normalised max error {e:.3e}")
    assert e < 1e-5


def test_fp32_tensor_core_path_chunks_and_pitch():
    spec = I.CalibSpec(3000, 384, "f32", "skew", 3, 60.0, 60.0, seed=95)
    X = I.make_calib(spec, "cuda")
    Xv = X[:, :320]                                   # pitch 384, width 320
    H = torch.zeros(320, 320, device="cuda")
    B.hessian_accumulate(Xv[:1700], H)
    B.hessian_accumulate(Xv[1700:], H)
    torch.cuda.synchronize()
    assert _norm_err(to_np(H).astype(np.float64), O.hessian(to_np(Xv))) < 1e-5


@pytest.mark.parametrize("n_tokens,inp", [(1000, 512), (777, 320), (4096, 1024), (130, 64), (64, 8)])
def test_bf16_tensor_core_path(n_tokens, inp):
    spec = I.CalibSpec(n_tokens, inp, "bf16", "normal", max(1, inp // 100), 20.0, 50.0, seed=91)
    X = I.make_calib(spec, "cuda")
    H = torch.zeros(inp, inp, device="cuda")
    st = status_tensor()
    B.hessian_accumulate(X, H, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    Hn = to_np(H).astype(np.float64)
    Href = O.hessian(to_np(X))
    e = _norm_err(Hn, Href)
    print(f"hessian bf16 n={n_tokens} in={inp}: normalised max error {e:.3e}")
    assert e < TOL
    assert np.max(np.abs(Hn - Hn.T)) <= TOL * np.max(np.diag(Href))


def test_chunked_accumulation_and_row_pitch():
    spec = I.CalibSpec(1536, 640, "bf16", "skew", 3, 80.0, 80.0, seed=92)
    X = I.make_calib(spec, "cuda")
    H1 = torch.zeros(512, 512, device="cuda")
    Xv = X[:, :512]                                   # pitch 640, width 512
    B.hessian_accumulate(Xv[:1000], H1)
    B.hessian_accumulate(Xv[1000:], H1)
    torch.cuda.synchronize()
    Href = O.hessian(to_np(Xv))
    assert _norm_err(to_np(H1).astype(np.float64), Href) < TOL
    B.hessian_accumulate(Xv[:0], H1)                  # empty chunk: no change, no error


def test_full_size_sampled_entries_and_probe():
    """262144 tokens x 4096 channels: sampled entries against per-entry fp64 sums, plus a
    Freivalds probe H v == 2 X^T (X v) over all tokens."""
    wl = I.workload_qproj()
    spec = wl["layers"]["q_proj"][1]
    X = I.make_calib(spec, "cuda")
    H = torch.zeros(spec.inp, spec.inp, device="cuda")
    st = status_tensor()
    B.hessian_accumulate(X, H, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    ids, _ = I.outlier_channels(spec)
    rng = np.random.default_rng(5)
    cols = np.unique(np.concatenate([ids.numpy()[:8], rng.integers(0, spec.inp, 40), [0, 255, 256, 4095]]))
    Xs = X[:, torch.as_tensor(cols, device="cuda")].double().cpu().numpy()      # [N, k]
    Hs_ref = 2.0 * (Xs.T @ Xs)
    Hs = H[torch.as_tensor(cols, device="cuda")][:, torch.as_tensor(cols, device="cuda")].double().cpu().numpy()
    d = np.sqrt(np.diag(Hs_ref))
    e = float(np.max(np.abs(Hs - Hs_ref) / np.outer(d, d)))
    print(f"hessian full-size sampled normalised max error {e:.3e}; "
          f"diag rel err max {np.max(np.abs(np.diag(Hs) - np.diag(Hs_ref)) / np.diag(Hs_ref)):.3e}")
    assert e < TOL
    # probe
    v = rng.standard_normal(spec.inp)
    z = np.zeros(spec.inp)
    for t0 in range(0, spec.n_tokens, 16384):
        Xc = X[t0:t0 + 16384].double().cpu().numpy()
        z += Xc.T @ (Xc @ v)
    hv = H.double().cpu().numpy() @ v
    rel = np.linalg.norm(hv - 2.0 * z) / np.linalg.norm(2.0 * z)
    print(f"hessian probe relative error {rel:.3e}")
    assert rel < TOL


def test_bad_arguments():
    X = torch.zeros(64, 100, dtype=torch.bfloat16, device="cuda")       # in % 8 != 0
    with pytest.raises(B.AdadimError) as e:
        B.hessian_accumulate(X, torch.zeros(100, 100, device="cuda"))
    assert e.value.status == 2
    with pytest.raises(KeyError):
        B.hessian_accumulate(torch.zeros(64, 64, dtype=torch.float64, device="cuda"), torch.zeros(64, 64, device="cuda"))
