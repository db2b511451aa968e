"""Accuracy and speed against the number of moduli at the benchmark size (m = n = k = 8192), for the three exponent
spreads of the workload (phi = 0.5, 1, 2): the error must fall by roughly M^-1/2 per modulus (Section 3.1) down to the
floating-point floor, and 16 moduli must reach double-precision accuracy for phi = 0.5 (Section 4).  The table itself is
printed (one JSON line per spread; `pytest -s` or `-rP` shows it)."""
import json
import math

import numpy as np
import pytest
import torch

from oracle import direct, staged
from paper_2609_05419_b200 import binding as b
from paper_2609_05419_b200 import inputs

pytestmark = pytest.mark.gpu

from gpu_util import Workspace, empty_dev, to_dev  # noqa: E402

NMODS = list(range(8, 23))


@pytest.mark.parametrize("phi", [0.5, 1.0, 2.0])
def test_error_and_time_against_modulus_count(phi):
    m = n = k = 8192
    A, B = inputs.complex_inputs(m, n, k, seed=2, dist="phi", phi=phi)
    pairs = inputs.sample_indices(m, n, 2048, seed=7, tile=128)
    Cs, Ds = direct.zgemm4m_dd_samples(A, B, pairs)
    idx = torch.from_numpy(pairs).cuda()
    dA, dB = to_dev(A), to_dev(B)
    rows = []
    with Workspace(b.workspace_bytes(b.OP_ZGEMM, m, n, k, max(NMODS))):
        C = empty_dev(m, n, torch.complex128)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for nmod in NMODS:
            b.zgemm2m(dA, dB, C, nmod)               # warm
            e0.record()
            for _ in range(3):
                b.zgemm2m(dA, dB, C, nmod)
            e1.record()
            b.device_status()
            ms = e0.elapsed_time(e1) / 3
            got = C[idx[:, 0], idx[:, 1]].cpu().numpy()
            err = direct.componentwise_error(got, Cs, Ds)
            log2M = math.log2(staged.product(staged.greedy_2m_moduli()[:nmod]))
            rows.append(dict(nmod=nmod, log2M=round(log2M, 2), max_err=err, ms=ms, tflops=8.0 * m * n * k / ms / 1e9))
    errs = {r["nmod"]: r["max_err"] for r in rows}
    floor = 4e-16                                    # one rounding of the result relative to |A||B|
    for a, c in zip(NMODS, NMODS[1:]):               # never gets worse by more than noise, and improves while above the floor
        assert errs[c] <= max(1.5 * errs[a], floor), (phi, a, c, errs)
        if errs[c] > 20 * floor:
            assert errs[c] < errs[a] / 3, (phi, a, c, errs)
    need = {0.5: 16, 1.0: 16, 2.0: 18}[phi]
    assert errs[need] <= 1e-14
    assert all(r["max_err"] <= floor * 4 for r in rows if r["nmod"] >= need + 2)
    # the M^-1/2 law between 8 and 12 moduli (far above the floor)
    slope = math.log2(errs[8] / errs[12]) / (rows[4]["log2M"] - rows[0]["log2M"])
    assert 0.35 < slope < 0.65, slope
    # more moduli never make a call faster
    assert rows[-1]["ms"] > rows[0]["ms"]
    print(json.dumps({"phi": phi, "rows": rows}))
