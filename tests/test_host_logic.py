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
    names = set(re.findall(r"^(?:int|size_t|const char\*)\s+(\w+)\s*\(", text, flags=re.M))      # every declared function
    assert {"gemm2m_gaussian_int", "zgemm2m", "cgemm2m", "zherk2m", "zher2k2m", "dsyrk2m", "dsyr2k2m", "zgemm2m_ex", "cgemm2m_ex",
            "gemm2m_set_workspace", "gemm2m_workspace_bytes", "gemm2m_zscale_exponents_static", "dgemm_ozaki2", "gemm2m_set_scaling"} <= names
    assert len(names) >= 25
    L = b.lib()
    for name in names:
        assert hasattr(L, name), name


def test_moduli_and_roots_match_oracle():
    mods = staged.greedy_2m_moduli()
    assert b.max_2m_moduli() == len(mods)
    for j, m in enumerate(mods):
        assert b.modulus(j) == (m, staged.sqrt_minus_one(m))
    hyb = staged.hybrid_moduli(b.max_moduli())
    assert b.max_moduli() == 26 and hyb[:22] == mods
    for j in range(22, 26):
        assert b.modulus(j) == (hyb[j], 0)                # 3M modulus: no root
    with pytest.raises(b.Gemm2mError):
        b.modulus(26)


@pytest.mark.parametrize("nmod", [1, 2, 3, 7, 8, 16, 17, 20, 22])
def test_crt_and_scaling_constants_match_oracle(nmod):
    mods = staged.greedy_2m_moduli()[:nmod]
    M = staged.product(mods)
    for k, herk in ((1, False), (300, False), (8192, False), (8192, True), (150000, False)):
        t = b.debug_tables(nmod, k, herk)
        assert (t["Pt"], t["PA"], t["PB"], t["ck"]) == staged.scaling_targets(M, k, herk)
    t = b.debug_tables(nmod, 8192)
    B = 2 ** 40
    assert sum(int(t["Mc"][c]) * B ** c for c in range(t["nchunks"])) == M       # the digits the kernel reads
    assert (t["nchunks"] - 1) * 40 < ((M - 1) // 2).bit_length() <= t["nchunks"] * 40
    for j, (m, s) in enumerate(zip(mods, [staged.sqrt_minus_one(q) for q in mods])):
        W = M // m
        q = pow(W % m, -1, m)
        Gr = sum(int(t["gr"][j, c]) * B ** c for c in range(5))
        Gi = sum(int(t["gi"][j, c]) * B ** c for c in range(5))
        assert Gr == staged.sym(staged.inv2(m) * q, m) * W          # Eq. (2c) real part folded into the CRT weight
        assert Gi == staged.sym(s * staged.inv2(m) * q, m) * W      # imaginary part
        assert all(abs(t["gr"][j, c]) < B and abs(t["gi"][j, c]) < B for c in range(5))
        for bb in range(8):                                          # byte weights of the residue kernels
            assert int(t["res_w"][j, bb]) == staged.sym(256 ** bb, m)
            assert int(t["res_w"][j, 8 + bb]) == staged.sym(s * 256 ** bb, m)


def test_residue_reduction_constants_are_exact_for_every_reachable_sum():
    """The residue kernels reduce x (a sum of byte-weight products) modulo m with one FP32 FMA and one integer
    multiply-add.  Emulate that FMA in exact integer arithmetic (float operands are dyadic rationals; round to nearest
    even at unit spacing) for EVERY integer x the kernels can reach and require the symmetric residue in the low byte."""
    r = b.debug_residue_reduction(26)
    mods = staged.hybrid_moduli(26)
    for j, m in enumerate(mods):
        y0_bits, xmax = int(r["y0_bits"][j]), int(r["xmax"][j])
        y0 = (y0_bits - 0x4B000000) + 2 ** 23                 # value of the float with that bit pattern (exponent 2^23)
        assert y0 % (256 * m) == 0 and y0 - xmax >= 2 ** 23 and y0 + xmax < 2 ** 24
        s = staged.sqrt_minus_one(m) if j < 22 else 1          # a 3M modulus takes the plain weights for both parts
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
        want = ((x + m // 2) % m) - m // 2                     # symmetric range; [-m/2, m/2 - 1] for the even modulus
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
            Sr = sum((q + p) * sum(int(t["gr"][j, c]) * B ** c for c in range(5)) for j, (p, q) in enumerate(zip(cp, cm)))
            Si = sum((q - p) * sum(int(t["gi"][j, c]) * B ** c for c in range(5)) for j, (p, q) in enumerate(zip(cp, cm)))
            assert staged.lift(Sr, M) == xr and staged.lift(Si, M) == xi


@pytest.mark.parametrize("nmod", [23, 24, 26])
def test_hybrid_crt_and_scaling_constants_match_oracle(nmod):
    mods = staged.hybrid_moduli(nmod)
    roots = staged.roots_of(mods)
    M = staged.product(mods)
    for k, herk in ((1, False), (300, False), (8192, False), (131000, False)):
        t = b.debug_tables(nmod, k, herk)
        assert (t["Pt"], t["PA"], t["PB"], t["ck"]) == staged.scaling_targets(M, k, herk)
    t = b.debug_tables(nmod, 64)
    B = 2 ** 40
    val = lambda row: sum(int(row[c]) * B ** c for c in range(5))
    assert val(t["Mc"]) == M and all(t["Mc"][c] == 0 for c in range(t["nchunks"], 5))   # only the digits in use: the kernel reads no others
    assert (t["nchunks"] - 1) * 40 < ((M - 1) // 2).bit_length() <= t["nchunks"] * 40
    for j, (m, s) in enumerate(zip(mods, roots)):
        W = M // m
        q = pow(W % m, -1, m)
        if s is not None:
            assert val(t["gr"][j]) == staged.sym(staged.inv2(m) * q, m) * W
            assert val(t["gi"][j]) == staged.sym(s * staged.inv2(m) * q, m) * W
        else:                                                         # Eq. (1) needs no factor besides q_j
            assert val(t["gr"][j]) == staged.sym(q, m) * W == val(t["gi"][j])
        for bb in range(8):
            assert int(t["res_w"][j, bb]) == staged.sym(256 ** bb, m)
            assert int(t["res_w"][j, 8 + bb]) == staged.sym((s or 1) * 256 ** bb, m)
    # the folded sums reproduce post-processing + CRT + lift for random residues of every plane
    rng = np.random.default_rng(nmod)
    for _ in range(20):
        Sr = Si = 0
        res_r, res_i = [], []
        for j, (m, s) in enumerate(zip(mods, roots)):
            draw = lambda: int(rng.integers(-(m // 2), (m - 1) // 2 + 1))
            if s is not None:
                cp, cm = draw(), draw()
                r, i = staged.post_2m(cp, cm, m, s)
                Sr += (cm + cp) * val(t["gr"][j])
                Si += (cm - cp) * val(t["gi"][j])
            else:
                p1, p2, p3 = draw(), draw(), draw()
                r, i = staged.post_3m(p1, p2, p3, m)
                Sr += (p1 - p2) * val(t["gr"][j])
                Si += (p3 - p1 - p2) * val(t["gr"][j])
            res_r.append(r)
            res_i.append(i)
        assert staged.lift(Sr % M, M) == staged.lift(staged.crt(res_r, mods), M)
        assert staged.lift(Si % M, M) == staged.lift(staged.crt(res_i, mods), M)
        assert abs(Sr) < 2 ** 12 * M and abs(Si) < 2 ** 12 * M        # the multiple of M to remove stays below 2^12
    assert 2 ** t["Pt"] / M < 0.494                                   # margin of the quotient estimate in the post kernel


@pytest.mark.parametrize("nmod", [1, 8, 15, 20])
def test_real_scheme_constants_match_oracle(nmod):
    mods = staged.greedy_real_moduli()[:nmod]
    M = staged.product(mods)
    t = b.debug_tables_real(nmod, 8192)
    assert list(t["moduli"]) == mods
    assert (t["Pt"], t["PA"], t["PB"], t["ck"]) == staged.scaling_targets_real(M, 8192)
    B = 2 ** 40
    val = lambda row: sum(int(row[c]) * B ** c for c in range(5))
    assert val(t["Mc"]) == M and all(t["Mc"][c] == 0 for c in range(t["nchunks"], 5))
    assert (t["nchunks"] - 1) * 40 < max(((M - 1) // 2).bit_length(), 1) <= t["nchunks"] * 40
    for j, m in enumerate(mods):
        W = M // m
        assert val(t["g"][j]) == staged.sym(pow(W % m, -1, m) if m > 1 else 0, m) * W
    assert 2 ** t["Pt"] / M < 0.494 or nmod == 1                      # margin of the quotient estimate in the post kernel
    # exactness of the post kernel's digit arithmetic: every digit-column sum, and what is left of it after t M has come off,
    # stays an exact integer in a double for the worst residues (all at -128)
    G = [abs(val(t["g"][j])) for j in range(nmod)]
    t_max = -(-sum(128 * g for g in G) // M) + 1
    for c in range(t["nchunks"]):
        col = sum(128 * abs(int(t["g"][j][c])) for j in range(nmod))
        assert col + t_max * int(t["Mc"][c]) < 2 ** 53, (nmod, c)
    # the residue kernels' reduction, exhaustively, as for the 2M moduli
    assert (t["margin"] > 1.0).all()
    for j, m in enumerate(mods):
        y0_bits, xmax = int(t["y0_bits"][j]), int(t["xmax"][j])
        y0 = (y0_bits - 0x4B000000) + 2 ** 23
        assert y0 % (256 * m) == 0 and y0 - xmax >= 2 ** 23 and y0 + xmax < 2 ** 24
        mant, ex = np.frexp(np.float64(t["inv_m"][j]))
        n, e = int(mant * 2 ** 24), 24 - int(ex)
        cq = int(t["cq"][j])
        assert cq == 3 * 2 ** 22 - y0 // m
        x = np.arange(-xmax, xmax + 1, dtype=np.int64)
        num = (y0 + x) * n + (cq << e)
        fl = num >> e
        rem = num - (fl << e)
        half = 1 << (e - 1)
        tq = fl + ((rem > half) | ((rem == half) & (fl & 1 == 1)))
        low = ((y0_bits + x) - (0x4B000000 + (tq - 2 ** 23)) * m) & 0xFF
        res = np.where(low >= 128, low - 256, low)
        assert np.array_equal(res, ((x + m // 2) % m) - m // 2), m


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
    assert b.workspace_bytes(b.OP_ZGEMM, 8, 8, 8, 27) == 0
    assert b.workspace_bytes(b.OP_ZHERK, 8, 8, 8, 23) == 0            # the hybrid moduli serve the complex GEMMs only
    # hybrid: two planes per 2M modulus, three per 3M modulus
    lay = b.workspace_layout(b.OP_ZGEMM, 100, 60, 200, 25)
    planes = 2 * 22 + 3 * 3
    assert lay["off_apm"] + planes * 100 * lay["kp"] <= lay["off_bpm"] and lay["off_bpm"] + planes * 60 * lay["kp"] <= lay["off_cpm"]
    assert lay["off_cpm"] + planes * 60 * lay["ldp"] <= lay["total_bytes"]
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
    assert L.zgemm2m(4, 4, 4, one, 4, one, 4, one, 4, 27, null) == NMOD
    assert L.zgemm2m(4, 4, 4, null, 4, one, 4, one, 4, 16, null) == ARG         # null A with k > 0
    assert L.zgemm2m(0, 4, 4, null, 1, null, 4, null, 1, 16, null) == 0         # empty: valid no-op
    assert L.cgemm2m(4, 0, 4, null, 4, null, 4, null, 4, 7, null) == 0
    assert L.gemm2m_gaussian_int(4, 4, 4, one, one, 4, one, one, 4, one, one, 4, 9, null) == NMOD
    assert L.gemm2m_gaussian_int(4, 4, 4, one, one, 2, one, one, 4, one, one, 4, 3, null) == ARG
    assert L.zherk2m(4, 4, one, 3, one, 4, 16, null) == ARG
    assert L.zherk2m(0, 4, null, 1, null, 1, 16, null) == 0
    assert L.zherk2m(4, 4, one, 4, one, 4, 23, null) == NMOD                    # rank-k family: 2M moduli only
    assert L.zgemm2m_eisenstein(4, 4, 4, one, 4, one, 4, one, 4, 24, null) == NMOD      # the Eisenstein set has 23 moduli
    assert L.zgemm2m_eisenstein(4, 4, 4, one, 3, one, 4, one, 4, 16, null) == ARG
    assert L.zgemm2m_eisenstein(4, 0, 4, null, 4, null, 4, null, 4, 16, null) == 0
    assert L.zgemm2m_eisenstein_ex(b"X", b"N", 4, 4, 4, null, one, 4, one, 4, null, one, 4, 16, null) == ARG   # bad trans character
    assert L.zgemm2m_eisenstein_ex(b"T", b"N", 4, 4, 8, null, one, 4, one, 8, null, one, 4, 16, null) == ARG   # A stored k x m: lda < k
    assert b.workspace_bytes(b.OP_ZGEMM_EISENSTEIN, 64, 64, 64, 24) == 0 and b.workspace_bytes(b.OP_ZGEMM_EISENSTEIN, 64, 64, 64, 23) > 0
    lay = b.workspace_layout(b.OP_ZGEMM_EISENSTEIN, 100, 90, 70, 23)
    assert lay["off_apm"] + 2 * 23 * 100 * lay["kp"] <= lay["off_bpm"] and lay["off_cpm"] + 2 * 23 * 90 * lay["ldp"] <= lay["total_bytes"]
    assert L.zgemm2m_host(4, 4, 4, one, 3, one, 4, one, 4, 16, null) == ARG                 # host form: same checks
    assert L.zgemm2m_host(4, 4, 4, one, 4, one, 4, null, 4, 16, null) == ARG
    assert L.zgemm2m_host(4, 4, 4, one, 4, one, 4, one, 4, 27, null) == NMOD
    assert L.zgemm2m_host(0, 4, 4, null, 1, null, 4, null, 1, 16, null) == 0
    z, h = b.workspace_bytes(b.OP_ZGEMM, 300, 200, 100, 16), b.workspace_bytes(b.OP_ZGEMM_HOST, 300, 200, 100, 16)
    assert h >= z + 16 * (300 * 100 + 100 * 200 + 300 * 200) and h < z + 16 * (300 * 100 + 100 * 200 + 300 * 200) + 3 * 256
    assert L.gemm2m_set_workspace(one, 0) == ARG
    assert L.gemm2m_set_workspace(ctypes.c_void_p(8), 1024) == ARG              # not 256-byte aligned
    assert b.lib().gemm2m_status_string(WS) == b"GEMM2M_ERR_WORKSPACE"


@pytest.mark.parametrize("nmod", [1, 2, 8, 16, 23])
def test_eisenstein_constants_match_oracle(nmod):
    from oracle import eisenstein as E
    mods = E.greedy_eisenstein_moduli()[:nmod]
    assert b.max_eisenstein_moduli() == len(E.greedy_eisenstein_moduli()) == 23
    assert [b.eisenstein_modulus(j) for j in range(nmod)] == [(m, E.cube_root_of_unity(m)) for m in mods]
    M = staged.product(mods)
    for k in (1, 64, 8192, 10 ** 6):
        t = b.debug_tables_eisenstein(nmod, k)
        assert (t["Pt"], t["PA"], t["PB"], t["ck"]) == E.scaling_targets_e(M, k)
    B = 2 ** 40
    val = lambda row: sum(int(row[c]) * B ** c for c in range(5))
    assert val(t["Mc"]) == M and all(t["Mc"][c] == 0 for c in range(t["nchunks"], 5))
    assert (t["nchunks"] - 1) * 40 < max(((M - 1) // 2).bit_length(), 1) <= t["nchunks"] * 40
    # Folded weights: with planes P+ = 2(a + s b), P- = 2(a + s^2 b) of both operands the products are 4 C+, 4 C-; the kernel
    # forms sum_j gr_j (P-_j + P+_j) and sum_j gi_j (P-_j - P+_j), which must be U = 2 c_a - c_b and V = c_b modulo M.
    rng = np.random.default_rng(nmod)
    for _ in range(20):
        ca, cb = (int(v) for v in rng.integers(-10 ** 9, 10 ** 9, 2))
        U = V = 0
        for j, m in enumerate(mods):
            s = E.cube_root_of_unity(m)
            cp, cm = staged.sym(4 * (ca + s * cb), m), staged.sym(4 * (ca + s * s * cb), m)
            U += val(t["gr"][j]) * (cm + cp)
            V += val(t["gi"][j]) * (cm - cp)
        assert (U - (2 * ca - cb)) % M == 0 and (V - cb) % M == 0
    for j, m in enumerate(mods):
        assert abs(val(t["gr"][j])) <= (m - 1) // 2 * (M // m) and abs(val(t["gi"][j])) <= (m - 1) // 2 * (M // m)
    # the residue kernels' reduction, exhaustively, as for the 2M moduli
    assert (t["margin"] > 1.0).all()
    for j, m in enumerate(mods):
        y0_bits, xmax = int(t["y0_bits"][j]), int(t["xmax"][j])
        y0 = (y0_bits - 0x4B000000) + 2 ** 23
        assert y0 % (256 * m) == 0 and y0 - xmax >= 2 ** 23 and y0 + xmax < 2 ** 24
        mant, ex = np.frexp(np.float64(t["inv_m"][j]))
        n, e = int(mant * 2 ** 24), 24 - int(ex)
        cq = int(t["cq"][j])
        assert cq == 3 * 2 ** 22 - y0 // m
        x = np.arange(-xmax, xmax + 1, dtype=np.int64)
        num = (y0 + x) * n + (cq << e)
        fl = num >> e
        rem = num - (fl << e)
        half = 1 << (e - 1)
        tq = fl + ((rem > half) | ((rem == half) & (fl & 1 == 1)))
        low = ((y0_bits + x) - (0x4B000000 + (tq - 2 ** 23)) * m) & 0xFF
        res = np.where(low >= 128, low - 256, low)
        assert np.array_equal(res, ((x + m // 2) % m) - m // 2), m


def _post_operand_checks(t, mods, M, plane_values, expected, rng_seed):
    """The tensor-core operand of the post-processing, emulated in exact integers: for residues c_p of every plane the kernel
    forms sum_p (c_p + 128) digit_p[k] per byte column k, packs four columns into a chunk, takes off[k] off, and removes a
    multiple of M.  plane_values(rng) -> residues per plane; expected(residues) -> (X_r, X_i) modulo M from the oracle."""
    planes, nb = t["planes"], t["nb"]
    assert t["ks"] == (planes + 31) // 32 and nb % 2 == 0 and 4 * nb <= 24
    Pt = ((M - 1) // 2).bit_length() - 1                              # |X| <= 2^Pt by the scaling rule: the quotient estimate (off by
    assert 2 ** Pt / M + 2 ** -16 < 0.5                               # less than 2^-17) rounds to the right multiple of M
    nbytes = (M.bit_length() + 7) // 8
    assert nb == 2 * ((nbytes + 7) // 8) and M >= 2 ** (32 * nb - 64)        # what the quotient estimate relies on
    weights = [[sum(int(d) << (8 * p) for p, d in enumerate(t["digits"][part, pl])) for pl in range(planes)] for part in range(2)]
    assert all(0 <= w < M for part in range(2) for w in weights[part])
    assert (t["digits"][:, :, 4 * nb:] == 0).all()
    # M in base 2^32, every stored number exact
    mc = [int(v) for v in t["Mc"]]
    assert all(float(v) == t["Mc"][k] for k, v in enumerate(mc)) and sum(mc) == M and all(v == 0 for v in mc[nb:])
    assert all(abs(mc[k]) <= 2 ** 31 * 2 ** (32 * k) and mc[k] % 2 ** (32 * k) == 0 for k in range(nb - 1))
    # offsets: 1.5 2^52 plus the chunk's share of 128 x (sum of the weights), all exact doubles
    for part in range(2):
        off = [int(v) for v in t["off"][part]]
        assert all(float(v) == t["off"][part][k] for k, v in enumerate(off))
        share = [off[k] // 2 ** (32 * k) - 3 * 2 ** 51 for k in range(nb)]
        assert all(off[k] % 2 ** (32 * k) == 0 and 0 <= share[k] < 2 ** 46 for k in range(nb))
        assert sum(share[k] << (32 * k) for k in range(nb)) == 128 * sum(weights[part])
    # worst case of the packed sums: every residue at +127 (c + 128 = 255)
    col_max = max(255 * int(t["digits"][part, :, p].astype(np.int64).sum()) for part in range(2) for p in range(4 * nb))
    assert col_max < 2 ** 22
    assert col_max * 257 < 2 ** 31                                            # a = s0 + 256 s1 is a 32-bit unsigned number
    assert col_max * (1 + 2 ** 8 + 2 ** 16 + 2 ** 24) < 2 ** 47               # the chunk sits far inside the 2^51 of the conversion
    rng = np.random.default_rng(rng_seed)
    for trial in range(24):
        c = plane_values(rng, trial)
        want = expected(c)
        for part in range(2):
            cols = [sum((c[pl] + 128) * int(t["digits"][part, pl, p]) for pl in range(planes)) for p in range(4 * nb)]
            chunk = [sum(cols[4 * k + b] << (8 * b) for b in range(4)) for k in range(nb)]
            W = [chunk[k] - (int(t["off"][part][k]) // 2 ** (32 * k) - 3 * 2 ** 51) for k in range(nb)]
            X1 = sum(W[k] << (32 * k) for k in range(nb))
            assert X1 == sum(c[pl] * weights[part][pl] for pl in range(planes))
            assert (X1 - want[part]) % M == 0
            tq = round(X1 / M) if abs(X1) < 2 ** 1000 else 0
            lead = sum(W[k] << (32 * k) for k in range(max(nb - 3, 0), nb))
            assert abs(lead - X1) * 2 ** 17 <= M and abs(tq) < 2 ** 14      # dropped chunks do not move the quotient
            assert all(abs(W[k] * 2 ** (32 * k) - tq * mc[k]) < 2 ** (47 + 32 * k) for k in range(nb))   # fused multiply-adds exact
            if abs(X1 - tq * M) * 2 <= M and nb > 2:
                _check_three_op_sums([W[k] * 2 ** (32 * k) - tq * mc[k] for k in range(nb)], X1 - tq * M)


def _check_three_op_sums(terms, X, rounded=True):
    """The finish adds its chunks with three-operation error-free additions (s = a + b, z = s - a, e = b - z), which are exact
    when a is a whole multiple of ulp(b).  Emulated here in IEEE doubles (Python floats) in the kernel's order: neighbours
    first, then from the top down; every step must be error-free, so hi plus the error terms is X exactly; the error terms'
    own floating-point sum is off by at most a few 2^-106 of the largest intermediate sum."""
    Wf = [float(v) for v in terms]
    assert all(int(w) == v for w, v in zip(Wf, terms))
    errs, sums = [], [1.0]

    def add(a, b):
        s = a + b
        z = s - a
        e = b - z
        assert int(s) + int(e) == int(a) + int(b), (a, b)
        errs.append(e)
        sums.append(abs(s))
        return s

    ph = [add(Wf[2 * k + 1], Wf[2 * k]) for k in range(len(Wf) // 2)]
    h = ph[-1]
    for k in range(len(ph) - 2, -1, -1):
        h = add(h, ph[k])
    assert int(h) + sum(int(e) for e in errs) == X
    lo = 0.0
    for e in errs:
        lo += e
    slack = abs(int(h) + int(lo) - X)
    assert slack * 2 ** 104 <= int(max(sums))
    if rounded and slack * 2 ** 70 <= abs(X):                      # chunks that cancel to a tiny X aside, the result is X rounded once
        assert h + lo == float(X)


def test_three_operation_sums_hold_for_adversarial_magnitudes():
    # small or zero upper terms beside full-size lower ones: the case the usual |a| >= |b| condition does not cover
    rng = np.random.default_rng(5)
    for nb in (4, 6):
        for trial in range(2000):
            terms = []
            for k in range(nb):
                mag = int(rng.integers(0, 48))
                v = int(rng.integers(-2 ** mag, 2 ** mag + 1)) if rng.random() > 0.2 else 0
                terms.append(v * 2 ** (32 * k))
            _check_three_op_sums(terms, sum(terms), rounded=False)   # (ties between the error terms decide the last bit here)


@pytest.mark.parametrize("nmod", [1, 2, 7, 8, 9, 16, 17, 18, 22, 23, 26])
def test_post_operands_reproduce_eq_2c_eq_1_and_crt(nmod):
    mods = staged.hybrid_moduli(nmod)
    n2 = min(nmod, 22)
    n3 = nmod - n2
    roots = [staged.sqrt_minus_one(q) for q in mods[:n2]]
    M = staged.product(mods)
    t = b.debug_post_operands(nmod)
    assert t["planes"] == 2 * n2 + 3 * n3

    def plane_values(rng, trial):
        lo = lambda m: -(m // 2)
        hi = lambda m: (m - 1) // 2
        pick = (lambda m: hi(m)) if trial == 0 else (lambda m: lo(m)) if trial == 1 else (lambda m: int(rng.integers(lo(m), hi(m) + 1)))
        return [pick(m) for m in mods[:n2]] + [pick(m) for m in mods[:n2]] + [pick(m) for _ in range(3) for m in mods[n2:]]

    def expected(c):
        post = [staged.post_2m(c[j], c[n2 + j], mods[j], roots[j]) for j in range(n2)]
        post += [staged.post_3m(c[2 * n2 + j3], c[2 * n2 + n3 + j3], c[2 * n2 + 2 * n3 + j3], mods[n2 + j3]) for j3 in range(n3)]
        return staged.crt([r for r, _ in post], mods), staged.crt([i for _, i in post], mods)

    _post_operand_checks(t, mods, M, plane_values, expected, nmod)


@pytest.mark.parametrize("nmod", [1, 8, 16, 17, 23])
def test_post_operands_of_the_eisenstein_variant(nmod):
    from oracle import eisenstein as E
    mods = E.greedy_eisenstein_moduli()[:nmod]
    M = staged.product(mods)
    t = b.debug_post_operands(nmod, eisenstein=True)
    assert t["planes"] == 2 * nmod
    state = {}

    def plane_values(rng, trial):
        ca, cb = (int(v) for v in rng.integers(-10 ** 9, 10 ** 9, 2))
        state["want"] = ((2 * ca - cb) % M, cb % M)                  # U = 2 c_a - c_b, V = c_b
        plus = [staged.sym(4 * (ca + E.cube_root_of_unity(m) * cb), m) for m in mods]
        minus = [staged.sym(4 * (ca + E.cube_root_of_unity(m) ** 2 * cb), m) for m in mods]
        return plus + minus

    _post_operand_checks(t, mods, M, plane_values, lambda c: state["want"], 100 + nmod)


@pytest.mark.parametrize("nmod", [1, 7, 16, 17, 22])
def test_post_operands_of_the_rank_k_family(nmod):
    # Section 5: C- = C+^T, so the kernel reads the C+ planes twice; K slots 0 .. nmod-1 hold c+ = C+[i, j], slots H .. H+nmod-1
    # (H = nmod rounded up to 16) hold c- = C+[j, i]; the padding slots carry zero weights.
    mods = staged.greedy_2m_moduli()[:nmod]
    roots = [staged.sqrt_minus_one(q) for q in mods]
    M = staged.product(mods)
    H = 16 * ((nmod + 15) // 16)
    t = b.debug_post_operands(nmod, herk=True)
    assert t["planes"] == 2 * H and t["ks"] == H // 16
    assert (t["digits"][:, nmod:H] == 0).all() and (t["digits"][:, H + nmod:] == 0).all()

    def plane_values(rng, trial):
        pick = (lambda m: (m - 1) // 2) if trial == 0 else (lambda m: -(m // 2)) if trial == 1 else (lambda m: int(rng.integers(-(m // 2), (m - 1) // 2 + 1)))
        pad = [int(rng.integers(-128, 128)) for _ in range(H - nmod)]              # whatever the padding slots hold must not matter
        return [pick(m) for m in mods] + pad + [pick(m) for m in mods] + pad

    def expected(c):
        post = [staged.post_2m(c[j], c[H + j], mods[j], roots[j]) for j in range(nmod)]
        return staged.crt([r for r, _ in post], mods), staged.crt([i for _, i in post], mods)

    _post_operand_checks(t, mods, M, plane_values, expected, 200 + nmod)
