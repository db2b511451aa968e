"""GPU parity of dgemm_ozaki2 (the real Ozaki-II scheme of Section 3.1) against the staged oracle and the definition."""
import numpy as np
import pytest
import torch

from oracle import direct, staged
from paper_2609_05419_b200 import binding as b

pytestmark = pytest.mark.gpu

from gpu_util import Workspace, empty_dev, to_dev, to_host, ulp_distance  # noqa: E402


def real_inputs(m, n, k, seed, phi=0.5):
    rng = np.random.default_rng(seed)
    A = (rng.random((m, k)) - 0.5) * np.exp(phi * rng.standard_normal((m, k)))
    B = (rng.random((k, n)) - 0.5) * np.exp(phi * rng.standard_normal((k, n)))
    return np.asfortranarray(A), np.asfortranarray(B)


def run(A, B, nmod, kernel=0, ldc=None):
    m, k = A.shape
    n = B.shape[1]
    b.debug_set_gemm_kernel(kernel)
    try:
        with Workspace(b.workspace_bytes(b.OP_DGEMM_OZAKI2, m, n, k, nmod)) as ws:
            C = empty_dev(m, n, torch.float64, ld=ldc, fill=-3.0)
            b.dgemm_ozaki2(to_dev(A), to_dev(B), C, nmod)
            b.device_status()
            lay = b.workspace_layout(b.OP_DGEMM_OZAKI2, m, n, k, nmod)
            raw = ws.buf.cpu().numpy()
            kp, ldp = lay["kp"], lay["ldp"]
            st = dict(eA=raw[lay["off_exp_a"]: lay["off_exp_a"] + 4 * m].view(np.int32).copy(),
                      eB=raw[lay["off_exp_b"]: lay["off_exp_b"] + 4 * n].view(np.int32).copy(),
                      Apl=raw[lay["off_apm"]: lay["off_apm"] + nmod * m * kp].view(np.int8).reshape(nmod, m, kp),
                      Bpl=raw[lay["off_bpm"]: lay["off_bpm"] + nmod * n * kp].view(np.int8).reshape(nmod, n, kp),
                      Cpl=raw[lay["off_cpm"]: lay["off_cpm"] + nmod * n * ldp].view(np.int8).reshape(nmod, n, ldp))
            return to_host(C), st
    finally:
        b.debug_set_gemm_kernel(0)


@pytest.mark.parametrize("kernel", [1, 0], ids=["checkgemm", "tcgen05"])
@pytest.mark.parametrize("shape,nmod,phi", [((200, 150, 300), 15, 0.5), ((129, 257, 128), 12, 1.0), ((33, 19, 50), 20, 2.0), ((64, 300, 1000), 3, 0.5)])
def test_real_scheme_every_stage(shape, nmod, phi, kernel):
    m, n, k = shape
    A, B = real_inputs(m, n, k, seed=91, phi=phi)
    A[2, :] = 0
    C, st = run(A, B, nmod, kernel)
    ref = staged.dgemm_o2_staged(A, B, nmod)
    assert (st["eA"] == ref["eA"]).all() and (st["eB"] == ref["eB"]).all()
    for j in range(nmod):
        assert (st["Apl"][j, :, :k] == ref["Apl"][j]).all(), ("Apl", j)
        assert (st["Bpl"][j, :, :k] == ref["Bpl"][j].T).all(), ("Bpl", j)
        assert (st["Apl"][j, :, k:] == 0).all()
        assert (st["Cpl"][j, :, :m] == ref["Cpl"][j].T).all(), ("Cpl", j)
    assert ulp_distance(C, ref["C"]).max() <= 1 and (C == ref["C"]).mean() > 0.999
    if nmod >= 15:
        Cref, D = direct.dgemm_dd(A, B)
        assert direct.componentwise_error(C, Cref, D) <= 1e-14


def test_real_scheme_1024_padding_panels_and_degenerate_rows():
    m, n, k = 1000, 2304, 640                      # 2304 columns: two panels
    A, B = real_inputs(m, n, k, seed=92)
    A[7, 5] = np.nan
    B[:, 11] *= 2.0 ** 500
    C, _ = run(A, B, 15, ldc=m + 8)
    assert np.isnan(C[7, :]).all() and (C[m:] == -3.0).all()
    ok = np.array([i for i in range(m) if i != 7])
    Cref, D = direct.dgemm_dd(A[ok], B)
    assert direct.componentwise_error(C[ok], Cref, D) <= 1e-14
    with Workspace(4096):
        Z = empty_dev(6, 5, torch.float64, fill=9.0)
        b.dgemm_ozaki2(to_dev(A[:6, :0]), to_dev(B[:0, :5]), Z, 15)      # k = 0: C = 0
        assert (to_host(Z) == 0).all()
        with pytest.raises(b.Gemm2mError, match="NMOD"):
            b.dgemm_ozaki2(to_dev(A[:6, :8]), to_dev(B[:8, :5]), Z, 21)
