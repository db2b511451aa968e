"""CPU-side checks of the CUDA library's host logic: exported symbols, constants against the oracle's
independent big-integer computation, workspace layout, and argument errors (detected before any launch)."""
import ctypes
import re
import os

import numpy as np
import pytest

from oracle import staged
from paper_2609_05419_b200 import binding as b

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    text = open(os.path.join(ROOT, "include", "gemm2m.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b((?:gemm2m_\w+|zgemm2m|cgemm2m|zherk2m))\s*\(", text))
    assert {"gemm2m_gaussian_int", "zgemm2m", "cgemm2m", "zherk2m", "gemm2m_set_workspace", "gemm2m_workspace_bytes"} <= names
    L = b.lib()
    for name in names:
        assert hasattr(L, name), name


def test_moduli_and_roots_match_oracle():
    mods = staged.greedy_2m_moduli()
    assert b.max_moduli() == len(mods)
    for j, m in enumerate(mods):
        assert b.modulus(j) == (m, staged.sqrt_minus_one(m))
    with pytest.raises(b.Gemm2mError):
        b.modulus(22)


@pytest.mark.parametrize("nmod", [1, 2, 3, 7, 8, 16, 17, 20, 22])
def test_crt_and_scaling_constants_match_oracle(nmod):
    mods = staged.greedy_2m_moduli()[:nmod]
    M = staged.product(mods)
    for k, herk in ((1, False), (300, False), (8192, False), (8192, True), (150000, False)):
        t = b.debug_tables(nmod, k, herk)
        assert (t["Pt"], t["PA"], t["PB"], t["ck"]) == staged.scaling_targets(M, k, herk)
    t = b.debug_tables(nmod, 8192)
    B = 2 ** 40
    assert sum(int(t["Mc"][c]) * B ** c for c in range(4)) == M
    assert (t["nchunks"] - 1) * 40 < ((M - 1) // 2).bit_length() <= t["nchunks"] * 40
    for j, (m, s) in enumerate(zip(mods, [staged.sqrt_minus_one(q) for q in mods])):
        W = M // m
        q = pow(W % m, -1, m)
        Gr = sum(int(t["gr"][j, c]) * B ** c for c in range(4))
        Gi = sum(int(t["gi"][j, c]) * B ** c for c in range(4))
        assert Gr == staged.sym(staged.inv2(m) * q, m) * W          # Eq. (2c) real part folded into the CRT weight
        assert Gi == staged.sym(s * staged.inv2(m) * q, m) * W      # imaginary part
        assert all(abs(t["gr"][j, c]) < B and abs(t["gi"][j, c]) < B for c in range(4))
        for bb in range(8):                                          # byte weights of the residue kernels
            assert int(t["res_w"][j, bb]) == staged.sym(256 ** bb, m)
            assert int(t["res_w"][j, 8 + bb]) == staged.sym(s * 256 ** bb, m)


def test_residue_reduction_constants_are_exact_for_every_reachable_sum():
    """The residue kernels reduce x (a sum of byte-weight products) modulo m with one FP32 FMA and one integer
    multiply-add.  Emulate that FMA in exact integer arithmetic (float operands are dyadic rationals; round to nearest
    even at unit spacing) for EVERY integer x the kernels can reach and require the symmetric residue in the low byte."""
    r = b.debug_residue_reduction(22)
    mods = staged.greedy_2m_moduli()
    for j, m in enumerate(mods):
        y0_bits, xmax = int(r["y0_bits"][j]), int(r["xmax"][j])
        y0 = (y0_bits - 0x4B000000) + 2 ** 23                 # value of the float with that bit pattern (exponent 2^23)
        assert y0 % (256 * m) == 0 and y0 - xmax >= 2 ** 23 and y0 + xmax < 2 ** 24
        s = staged.sqrt_minus_one(m)
        w = [abs(staged.sym(256 ** bb, m)) + abs(staged.sym(s * 256 ** bb, m)) for bb in range(12)]
        assert xmax == 255 * sum(w[:4]) + 128 * sum(w[4:])    # four unsigned bytes, eight balanced digits, both parts
        assert float(r["margin"][j]) > 1.0
        mant, ex = np.frexp(np.float64(r["inv_m"][j]))
        n, e = int(mant * 2 ** 24), 24 - int(ex)               # inv_m = n 2^-e exactly
        assert n * 2.0 ** -e == float(r["inv_m"][j])
        cq = int(r["cq"][j])
        assert cq == float(r["cq"][j]) and cq == 3 * 2 ** 22 - y0 // m
        x = np.arange(-xmax, xmax + 1, dtype=np.int64)
        num = (y0 + x) * n + (cq << e)                          # exact value of the FMA, times 2^e
        fl = num >> e
        rem = num - (fl << e)
        half = 1 << (e - 1)
        t = fl + ((rem > half) | ((rem == half) & (fl & 1 == 1)))   # round to nearest even; 2^23 <= t < 2^24: spacing 1
        assert t.min() >= 2 ** 23 and t.max() < 2 ** 24
        t_bits = 0x4B000000 + (t - 2 ** 23)
        y_bits = y0_bits + x
        low = (y_bits - t_bits * m) & 0xFF
        res = np.where(low >= 128, low - 256, low)
        want = ((x + (m - 1) // 2) % m) - (m - 1) // 2
        assert np.array_equal(res, want), m


def test_folded_crt_weights_reproduce_eq_2c_and_crt():
    # sum_j (c- + c+) Gr_j  and  sum_j (c- - c+) Gi_j  (mod M) must equal CRT of Eq. (2c), for random residues
    rng = np.random.default_rng(0)
    for nmod in (3, 16, 22):
        mods = staged.greedy_2m_moduli()[:nmod]
        roots = [staged.sqrt_minus_one(q) for q in mods]
        M = staged.product(mods)
        t = b.debug_tables(nmod, 64)
        B = 2 ** 40
        for _ in range(20):
            cp = [int(rng.integers(-(m - 1) // 2, (m - 1) // 2 + 1)) for m in mods]
            cm = [int(rng.integers(-(m - 1) // 2, (m - 1) // 2 + 1)) for m in mods]
            post = [staged.post_2m(p, q, m, s) for p, q, m, s in zip(cp, cm, mods, roots)]
            xr = staged.lift(staged.crt([r for r, _ in post], mods), M)
            xi = staged.lift(staged.crt([i for _, i in post], mods), M)
            Sr = sum((q + p) * sum(int(t["gr"][j, c]) * B ** c for c in range(4)) for j, (p, q) in enumerate(zip(cp, cm)))
            Si = sum((q - p) * sum(int(t["gi"][j, c]) * B ** c for c in range(4)) for j, (p, q) in enumerate(zip(cp, cm)))
            assert staged.lift(Sr, M) == xr and staged.lift(Si, M) == xi


def test_workspace_layout_is_ordered_and_sized():
    for op, (m, n, k, nmod) in ((b.OP_ZGEMM, (1000, 900, 700, 16)), (b.OP_CGEMM, (129, 1, 1, 7)),
                                (b.OP_GAUSSIAN_INT, (128, 128, 128, 3)), (b.OP_ZHERK, (500, 500, 333, 16))):
        lay = b.workspace_layout(op, m, n, k, nmod)
        assert lay["kp"] % 128 == 0 and lay["kp"] >= k and lay["ldp"] % 16 == 0 and lay["ldp"] >= m
        herk = op == b.OP_ZHERK
        assert lay["off_exp_a"] < lay["off_apm"] and lay["off_apm"] + 2 * nmod * m * lay["kp"] <= lay["off_bpm"] <= lay["off_cpm"]
        assert lay["off_cpm"] + (1 if herk else 2) * nmod * n * lay["ldp"] <= lay["total_bytes"]
        assert lay["total_bytes"] == b.workspace_bytes(op, m, n, k, nmod)
        for key in ("off_exp_a", "off_exp_b", "off_apm", "off_bpm", "off_cpm"):
            assert lay[key] % 256 == 0
    assert b.workspace_bytes(b.OP_GAUSSIAN_INT, 8, 8, 8, 9) == 0      # int64 result needs M < 2^63
    assert b.workspace_bytes(b.OP_ZGEMM, 8, 8, 8, 23) == 0
    assert b.workspace_bytes(b.OP_ZGEMM, -1, 8, 8, 3) == 0


def test_argument_errors_are_reported_before_any_launch():
    L = b.lib()
    null = ctypes.c_void_p(0)
    one = ctypes.c_void_p(256)      # never dereferenced: argument checks come first
    ARG, NMOD, WS = 1, 2, 3
    assert L.zgemm2m(-1, 4, 4, one, 4, one, 4, one, 4, 16, null) == ARG
    assert L.zgemm2m(4, 4, 4, one, 3, one, 4, one, 4, 16, null) == ARG          # lda < m
    assert L.zgemm2m(4, 4, 4, one, 4, one, 3, one, 4, 16, null) == ARG          # ldb < k
    assert L.zgemm2m(4, 4, 4, one, 4, one, 4, one, 3, 16, null) == ARG          # ldc < m
    assert L.zgemm2m(4, 4, 4, one, 4, one, 4, one, 4, 0, null) == NMOD
    assert L.zgemm2m(4, 4, 4, one, 4, one, 4, one, 4, 23, null) == NMOD
    assert L.zgemm2m(4, 4, 4, null, 4, one, 4, one, 4, 16, null) == ARG         # null A with k > 0
    assert L.zgemm2m(0, 4, 4, null, 1, null, 4, null, 1, 16, null) == 0         # empty: valid no-op
    assert L.cgemm2m(4, 0, 4, null, 4, null, 4, null, 4, 7, null) == 0
    assert L.gemm2m_gaussian_int(4, 4, 4, one, one, 4, one, one, 4, one, one, 4, 9, null) == NMOD
    assert L.gemm2m_gaussian_int(4, 4, 4, one, one, 2, one, one, 4, one, one, 4, 3, null) == ARG
    assert L.zherk2m(4, 4, one, 3, one, 4, 16, null) == ARG
    assert L.zherk2m(0, 4, null, 1, null, 1, 16, null) == 0
    assert L.gemm2m_set_workspace(one, 0) == ARG
    assert L.gemm2m_set_workspace(ctypes.c_void_p(8), 1024) == ARG              # not 256-byte aligned
    assert b.lib().gemm2m_status_string(WS) == b"GEMM2M_ERR_WORKSPACE"
