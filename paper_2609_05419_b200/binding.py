"""Thin ctypes binding of the gemm2m C-ABI library (include/gemm2m.h): same entry-point names, argument
marshalling only.  Matrices are torch CUDA tensors viewed column-major (stride 1 along the first dimension);
torch is used for device memory and streams, every step of the computation runs in the library's kernels.

There is no fallback: if libgemm2m.so has not been built (``python -m paper_2609_05419_b200.build``) or cannot
be loaded, every call raises.
"""
from __future__ import annotations

import ctypes
import os

OP_GAUSSIAN_INT, OP_ZGEMM, OP_CGEMM, OP_ZHERK, OP_ZHER2K, OP_DSYRK, OP_DSYR2K, OP_DGEMM_OZAKI2 = 0, 1, 2, 3, 4, 5, 6, 7
OP_ZGEMM_EISENSTEIN = 8
OP_ZGEMM_HOST = 9
OK = 0
ERR_ARG, ERR_NMOD, ERR_WORKSPACE, ERR_CUDA, ERR_ARCH, ERR_DEVICE_TIMEOUT = 1, 2, 3, 4, 5, 6     # gemm2m_status

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgemm2m.so")
_lib = None


class Gemm2mError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        name = lib().gemm2m_status_string(status).decode()
        extra = ""
        if name == "GEMM2M_ERR_CUDA":
            extra = " (" + lib().gemm2m_last_cuda_error().decode() + ")"
        super().__init__(f"{where}: {name}{extra}")


class Layout(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in
                ("off_exp_a", "off_exp_b", "off_apm", "off_bpm", "off_cpm", "kp", "ldp", "total_bytes")]


def lib():
    """The loaded C-ABI library.  Raises if it is missing: there is no CPU or library fallback."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_05419_b200.build` (needs nvcc)")
    L = ctypes.CDLL(LIB_PATH)
    i64, i32, vp, sz = ctypes.c_int64, ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t
    L.gemm2m_status_string.restype = ctypes.c_char_p
    L.gemm2m_status_string.argtypes = [i32]
    L.gemm2m_last_cuda_error.restype = ctypes.c_char_p
    L.gemm2m_max_moduli.restype = i32
    L.gemm2m_max_2m_moduli.restype = i32
    L.gemm2m_modulus.argtypes = [i32, ctypes.POINTER(i32), ctypes.POINTER(i32)]
    L.gemm2m_workspace_bytes.restype = sz
    L.gemm2m_workspace_bytes.argtypes = [i32, i64, i64, i64, i32]
    L.gemm2m_set_workspace.argtypes = [vp, sz]
    L.gemm2m_gaussian_int.argtypes = [i64, i64, i64, vp, vp, i64, vp, vp, i64, vp, vp, i64, i32, vp]
    L.zgemm2m.argtypes = [i64, i64, i64, vp, i64, vp, i64, vp, i64, i32, vp]
    L.cgemm2m.argtypes = [i64, i64, i64, vp, i64, vp, i64, vp, i64, i32, vp]
    L.zgemm2m_host.argtypes = [i64, i64, i64, vp, i64, vp, i64, vp, i64, i32, vp]
    ex = [ctypes.c_char, ctypes.c_char, i64, i64, i64, vp, vp, i64, vp, i64, vp, vp, i64, i32, vp]
    L.zgemm2m_ex.argtypes = ex
    L.cgemm2m_ex.argtypes = ex
    L.zgemm2m_eisenstein.argtypes = [i64, i64, i64, vp, i64, vp, i64, vp, i64, i32, vp]
    L.zgemm2m_eisenstein_ex.argtypes = ex
    L.gemm2m_max_eisenstein_moduli.restype = i32
    L.gemm2m_eisenstein_modulus.argtypes = [i32, ctypes.POINTER(i32), ctypes.POINTER(i32)]
    L.gemm2m_debug_tables_eisenstein.argtypes = [i32, i64] + [vp] * 10
    L.zherk2m.argtypes = [i64, i64, vp, i64, vp, i64, i32, vp]
    L.dsyrk2m.argtypes = [i64, i64, vp, i64, vp, i64, i32, vp]
    L.zher2k2m.argtypes = [i64, i64, vp, i64, vp, i64, vp, i64, i32, vp]
    L.dsyr2k2m.argtypes = [i64, i64, vp, i64, vp, i64, vp, i64, i32, vp]
    L.gemm2m_device_status.argtypes = [vp]
    L.gemm2m_zscale_exponents_static.argtypes = [i64, i64, vp, i64, i32, vp, vp]
    L.gemm2m_set_profiling.argtypes = [i32]
    L.gemm2m_phase_ms.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.POINTER(i32)]
    L.gemm2m_last_launch_count.argtypes = [ctypes.POINTER(i32)]
    L.gemm2m_workspace_layout.argtypes = [i32, i64, i64, i64, i32, ctypes.POINTER(Layout)]
    L.gemm2m_debug_set_gemm_kernel.argtypes = [i32]
    L.gemm2m_debug_wait_selftest.argtypes = [ctypes.c_uint64, vp]
    L.gemm2m_debug_set_panels.argtypes = [i32]
    L.dgemm_ozaki2.argtypes = [i64, i64, i64, vp, i64, vp, i64, vp, i64, i32, vp]
    L.gemm2m_debug_tables_real.argtypes = [i32, i64] + [vp] * 10
    L.gemm2m_set_scaling.argtypes = [i32]
    L.gemm2m_debug_tables.argtypes = [i32, i64, i32, vp, vp, vp, vp, vp, vp]
    L.gemm2m_debug_residue_reduction.argtypes = [i32, vp, vp, vp, vp, vp]
    L.gemm2m_debug_post_operands.argtypes = [i32, i32, vp, vp, vp]
    _lib = L
    return L


def _check(status, where):
    if status != OK:
        raise Gemm2mError(status, where)


def _stream_ptr(stream):
    if stream is None:
        import torch
        return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return ctypes.c_void_p(stream)
    return ctypes.c_void_p(stream.cuda_stream)


def _colmajor(t, name):
    """(pointer, rows, cols, leading dimension) of a 2-D CUDA tensor stored column-major."""
    if t.dim() != 2 or not t.is_cuda:
        raise ValueError(f"{name}: need a 2-D CUDA tensor")
    rows, cols = t.shape
    if rows > 1 and t.stride(0) != 1:
        raise ValueError(f"{name}: need column-major storage (stride 1 along dim 0), e.g. torch.empty(cols, rows).t()")
    ld = t.stride(1) if cols > 1 else max(rows, 1)
    return ctypes.c_void_p(t.data_ptr()), rows, cols, max(ld, 1)


def max_moduli():
    return int(lib().gemm2m_max_moduli())


def max_2m_moduli():
    return int(lib().gemm2m_max_2m_moduli())


def modulus(j):
    m, s = ctypes.c_int(), ctypes.c_int()
    _check(lib().gemm2m_modulus(j, ctypes.byref(m), ctypes.byref(s)), "gemm2m_modulus")
    return m.value, s.value


def workspace_bytes(op, m, n, k, nmod):
    return int(lib().gemm2m_workspace_bytes(op, m, n, k, nmod))


def workspace_layout(op, m, n, k, nmod):
    lay = Layout()
    _check(lib().gemm2m_workspace_layout(op, m, n, k, nmod, ctypes.byref(lay)), "gemm2m_workspace_layout")
    return {name: getattr(lay, name) for name, _ in Layout._fields_}


def set_workspace(tensor):
    """Register a torch uint8 CUDA tensor (kept alive by the caller) as the library's workspace; None unregisters."""
    if tensor is None:
        _check(lib().gemm2m_set_workspace(None, 0), "gemm2m_set_workspace")
    else:
        _check(lib().gemm2m_set_workspace(ctypes.c_void_p(tensor.data_ptr()), tensor.numel() * tensor.element_size()),
               "gemm2m_set_workspace")


def gemm2m_gaussian_int(Ar, Ai, Br, Bi, Cr, Ci, nmod, stream=None):
    pa, m, k, lda = _colmajor(Ar, "Ar")
    pai, _, _, ldai = _colmajor(Ai, "Ai")
    pb, k2, n, ldb = _colmajor(Br, "Br")
    pbi, _, _, ldbi = _colmajor(Bi, "Bi")
    pc, _, _, ldc = _colmajor(Cr, "Cr")
    pci, _, _, ldci = _colmajor(Ci, "Ci")
    if k != k2 or Ai.shape != Ar.shape or Bi.shape != Br.shape or Cr.shape != (m, n) or Ci.shape != (m, n):
        raise ValueError("shape mismatch")
    if (lda, ldb, ldc) != (ldai, ldbi, ldci):
        raise ValueError("real and imaginary planes must share their leading dimension")
    _check(lib().gemm2m_gaussian_int(m, n, k, pa, pai, lda, pb, pbi, ldb, pc, pci, ldc, nmod, _stream_ptr(stream)),
           "gemm2m_gaussian_int")


def _xgemm(fn, name, A, B, C, nmod, stream):
    pa, m, k, lda = _colmajor(A, "A")
    pb, k2, n, ldb = _colmajor(B, "B")
    pc, mc, nc, ldc = _colmajor(C, "C")
    if k != k2 or (mc, nc) != (m, n):
        raise ValueError("shape mismatch")
    _check(fn(m, n, k, pa, lda, pb, ldb, pc, ldc, nmod, _stream_ptr(stream)), name)


def zgemm2m(A, B, C, nmod=16, stream=None):
    _xgemm(lib().zgemm2m, "zgemm2m", A, B, C, nmod, stream)


def _colmajor_host(t, name):
    """(pointer, rows, cols, leading dimension) of a 2-D CPU tensor stored column-major."""
    if t.dim() != 2 or t.is_cuda:
        raise ValueError(f"{name}: need a 2-D CPU tensor")
    rows, cols = t.shape
    if rows > 1 and t.stride(0) != 1:
        raise ValueError(f"{name}: need column-major storage (stride 1 along dim 0), e.g. torch.empty(cols, rows).t()")
    ld = t.stride(1) if cols > 1 else max(rows, 1)
    return ctypes.c_void_p(t.data_ptr()), rows, cols, max(ld, 1)


def zgemm2m_host(A, B, C, nmod=16, stream=None):
    """C = A B with A, B, C complex128 CPU tensors (column-major views; pinned memory lets the copies overlap the kernels).
    Asynchronous on `stream`: C is valid, and A, B may be changed, once the stream has completed."""
    pa, m, k, lda = _colmajor_host(A, "A")
    pb, k2, n, ldb = _colmajor_host(B, "B")
    pc, mc, nc, ldc = _colmajor_host(C, "C")
    if k != k2 or (mc, nc) != (m, n):
        raise ValueError("shape mismatch")
    _check(lib().zgemm2m_host(m, n, k, pa, lda, pb, ldb, pc, ldc, nmod, _stream_ptr(stream)), "zgemm2m_host")


def cgemm2m(A, B, C, nmod=7, stream=None):
    _xgemm(lib().cgemm2m, "cgemm2m", A, B, C, nmod, stream)


def _xgemm_ex(fn, name, ctype, transa, transb, alpha, A, B, beta, C, nmod, stream):
    """C = alpha op(A) op(B) + beta C; A, B as stored (column-major views), trans in 'N', 'T', 'C'."""
    pa, ra, ca, lda = _colmajor(A, "A")
    pb, rb, cb, ldb = _colmajor(B, "B")
    pc, m, n, ldc = _colmajor(C, "C")
    ma, ka = (ra, ca) if transa in "Nn" else (ca, ra)
    kb, nb = (rb, cb) if transb in "Nn" else (cb, rb)
    if ka != kb or (ma, nb) != (m, n):
        raise ValueError("shape mismatch")
    pair = lambda z: None if z is None else (ctype * 2)(complex(z).real, complex(z).imag)
    al, be = pair(alpha), pair(beta)
    ptr = lambda a: None if a is None else ctypes.cast(a, ctypes.c_void_p)
    _check(fn(transa.encode(), transb.encode(), m, n, ka, ptr(al), pa, lda, pb, ldb, ptr(be), pc, ldc, nmod, _stream_ptr(stream)), name)


def zgemm2m_ex(transa, transb, alpha, A, B, beta, C, nmod=16, stream=None):
    _xgemm_ex(lib().zgemm2m_ex, "zgemm2m_ex", ctypes.c_double, transa, transb, alpha, A, B, beta, C, nmod, stream)


def cgemm2m_ex(transa, transb, alpha, A, B, beta, C, nmod=7, stream=None):
    _xgemm_ex(lib().cgemm2m_ex, "cgemm2m_ex", ctypes.c_float, transa, transb, alpha, A, B, beta, C, nmod, stream)


def zgemm2m_eisenstein(A, B, C, nmod=16, stream=None):
    """C = A B through the Eisenstein-integer variant (complex128 CUDA tensors, column-major views)."""
    _xgemm(lib().zgemm2m_eisenstein, "zgemm2m_eisenstein", A, B, C, nmod, stream)


def zgemm2m_eisenstein_ex(transa, transb, alpha, A, B, beta, C, nmod=16, stream=None):
    _xgemm_ex(lib().zgemm2m_eisenstein_ex, "zgemm2m_eisenstein_ex", ctypes.c_double, transa, transb, alpha, A, B, beta, C, nmod, stream)


def max_eisenstein_moduli():
    return int(lib().gemm2m_max_eisenstein_moduli())


def eisenstein_modulus(j):
    m, s = ctypes.c_int(0), ctypes.c_int(0)
    _check(lib().gemm2m_eisenstein_modulus(j, ctypes.byref(m), ctypes.byref(s)), "gemm2m_eisenstein_modulus")
    return m.value, s.value


def debug_tables_eisenstein(nmod, k):
    """Host-side constants of the Eisenstein variant (see gemm2m_debug_tables_eisenstein)."""
    import numpy as np
    scale = np.zeros(4, dtype=np.int32)
    gr = np.zeros((nmod, 5), dtype=np.float64)
    gi = np.zeros((nmod, 5), dtype=np.float64)
    mc = np.zeros(5, dtype=np.float64)
    nch = np.zeros(1, dtype=np.int32)
    y0 = np.zeros(nmod, dtype=np.int32)
    cq = np.zeros(nmod, dtype=np.float32)
    inv = np.zeros(nmod, dtype=np.float32)
    xmax = np.zeros(nmod, dtype=np.int32)
    margin = np.zeros(nmod, dtype=np.float64)
    ptr = lambda a: ctypes.c_void_p(a.ctypes.data)
    _check(lib().gemm2m_debug_tables_eisenstein(nmod, k, ptr(scale), ptr(gr), ptr(gi), ptr(mc), ptr(nch), ptr(y0), ptr(cq), ptr(inv),
                                                ptr(xmax), ptr(margin)), "gemm2m_debug_tables_eisenstein")
    return dict(Pt=int(scale[0]), PA=int(scale[1]), PB=int(scale[2]), ck=int(scale[3]), gr=gr, gi=gi, Mc=mc, nchunks=int(nch[0]),
                y0_bits=y0, cq=cq, inv_m=inv, xmax=xmax, margin=margin)


def dgemm_ozaki2(A, B, C, nmod=15, stream=None):
    """Real C = A B by the real Ozaki-II scheme (float64 CUDA tensors, column-major views)."""
    _xgemm(lib().dgemm_ozaki2, "dgemm_ozaki2", A, B, C, nmod, stream)


def zherk2m(A, C, nmod=16, stream=None):
    pa, n, k, lda = _colmajor(A, "A")
    pc, n1, n2, ldc = _colmajor(C, "C")
    if (n1, n2) != (n, n):
        raise ValueError("shape mismatch")
    _check(lib().zherk2m(n, k, pa, lda, pc, ldc, nmod, _stream_ptr(stream)), "zherk2m")


STATIC_MAX_ROWS = 65536


def zscale_exponents_static(A, e, nmod=16, stream=None):
    """Scale exponents of the rows of A (the ones zgemm2m uses for `nmod` moduli) into the int32 CUDA tensor `e`, for
    callers that may not allocate device memory: the library's built-in scratch replaces the workspace.  At most
    STATIC_MAX_ROWS rows; calls on one GPU must not overlap."""
    pa, m, k, lda = _colmajor(A, "A")
    if m > STATIC_MAX_ROWS:
        raise ValueError(f"zscale_exponents_static: {m} rows exceed the built-in scratch ({STATIC_MAX_ROWS} rows)")
    if e.numel() != m or not e.is_cuda or e.element_size() != 4 or not e.is_contiguous():
        raise ValueError("e: need a contiguous int32 CUDA tensor with one entry per row of A")
    _check(lib().gemm2m_zscale_exponents_static(m, k, pa, lda, nmod, ctypes.c_void_p(e.data_ptr()), _stream_ptr(stream)),
           "gemm2m_zscale_exponents_static")


def _rank(fn, name, A, B, C, nmod, stream):
    pa, n, k, lda = _colmajor(A, "A")
    pc, n1, n2, ldc = _colmajor(C, "C")
    if (n1, n2) != (n, n):
        raise ValueError("shape mismatch")
    if B is None:
        _check(fn(n, k, pa, lda, pc, ldc, nmod, _stream_ptr(stream)), name)
    else:
        pb, nb, kb, ldb = _colmajor(B, "B")
        if (nb, kb) != (n, k):
            raise ValueError("shape mismatch")
        _check(fn(n, k, pa, lda, pb, ldb, pc, ldc, nmod, _stream_ptr(stream)), name)


def zher2k2m(A, B, C, nmod=16, stream=None):
    _rank(lib().zher2k2m, "zher2k2m", A, B, C, nmod, stream)


def dsyrk2m(A, C, nmod=16, stream=None):
    _rank(lib().dsyrk2m, "dsyrk2m", A, None, C, nmod, stream)


def dsyr2k2m(A, B, C, nmod=16, stream=None):
    _rank(lib().dsyr2k2m, "dsyr2k2m", A, B, C, nmod, stream)


def device_status(stream=None):
    _check(lib().gemm2m_device_status(_stream_ptr(stream)), "gemm2m_device_status")


def set_profiling(enabled):
    _check(lib().gemm2m_set_profiling(1 if enabled else 0), "gemm2m_set_profiling")


def phase_ms():
    """Average per-call milliseconds of (scan, residues, GEMMs, post) over the profiled calls, and their number."""
    ms = (ctypes.c_float * 4)()
    calls = ctypes.c_int()
    _check(lib().gemm2m_phase_ms(ms, ctypes.byref(calls)), "gemm2m_phase_ms")
    return [float(x) for x in ms], calls.value


def last_launch_count():
    per = (ctypes.c_int * 4)()
    total = int(lib().gemm2m_last_launch_count(per))
    return total, [int(x) for x in per]


def debug_wait_selftest(budget_ns, stream=None):
    """Enqueue the bounded-wait self-test (see gemm2m_debug_wait_selftest)."""
    _check(lib().gemm2m_debug_wait_selftest(int(budget_ns), _stream_ptr(stream)), "gemm2m_debug_wait_selftest")


def debug_set_gemm_kernel(which):
    _check(lib().gemm2m_debug_set_gemm_kernel(which), "gemm2m_debug_set_gemm_kernel")


def set_scaling(mode):
    """0 = scale factors from the largest part of each row / column (default), 1 = from a bound of its 2-norm."""
    _check(lib().gemm2m_set_scaling(int(mode)), "gemm2m_set_scaling")


def debug_set_overlap(enabled):
    _check(lib().gemm2m_debug_set_overlap(1 if enabled else 0), "gemm2m_debug_set_overlap")


def debug_set_chained_launch(enabled):
    _check(lib().gemm2m_debug_set_chained_launch(1 if enabled else 0), "gemm2m_debug_set_chained_launch")


def debug_set_panels(max_panels):
    _check(lib().gemm2m_debug_set_panels(max_panels), "gemm2m_debug_set_panels")


def debug_tables(nmod, k, herk=False):
    """Host-side constants of the library for `nmod` moduli (see gemm2m_debug_tables)."""
    import numpy as np
    scale = np.zeros(4, dtype=np.int32)
    gr = np.zeros((nmod, 5), dtype=np.float64)
    gi = np.zeros((nmod, 5), dtype=np.float64)
    mc = np.zeros(5, dtype=np.float64)
    nch = np.zeros(1, dtype=np.int32)
    w = np.zeros((nmod, 16), dtype=np.int8)
    ptr = lambda a: ctypes.c_void_p(a.ctypes.data)
    _check(lib().gemm2m_debug_tables(nmod, k, 1 if herk else 0, ptr(scale), ptr(gr), ptr(gi), ptr(mc), ptr(nch), ptr(w)),
           "gemm2m_debug_tables")
    return dict(Pt=int(scale[0]), PA=int(scale[1]), PB=int(scale[2]), ck=int(scale[3]), gr=gr, gi=gi, Mc=mc,
                nchunks=int(nch[0]), res_w=w)


def debug_post_operands(nmod, eisenstein=False, herk=False):
    """Operand of the post-processing contraction (see gemm2m_debug_post_operands)."""
    import numpy as np
    dims = np.zeros(3, dtype=np.int32)
    consts = np.zeros(19, dtype=np.float64)
    ptr = lambda a: ctypes.c_void_p(a.ctypes.data)
    variant = 2 if herk else 1 if eisenstein else 0
    _check(lib().gemm2m_debug_post_operands(variant, nmod, None, ptr(dims), None), "gemm2m_debug_post_operands")
    digits = np.zeros((2, int(dims[0]), 24), dtype=np.uint8)
    _check(lib().gemm2m_debug_post_operands(variant, nmod, ptr(digits), ptr(dims), ptr(consts)), "gemm2m_debug_post_operands")
    return dict(planes=int(dims[0]), ks=int(dims[1]), nb=int(dims[2]), digits=digits, Mc=consts[0:6], off=consts[6:18].reshape(2, 6),
                inv_M=float(consts[18]))


def debug_residue_reduction(nmod):
    """Constants of the residue kernels' reduction modulo m_j (see gemm2m_debug_residue_reduction)."""
    import numpy as np
    y0 = np.zeros(nmod, dtype=np.int32)
    cq = np.zeros(nmod, dtype=np.float32)
    inv = np.zeros(nmod, dtype=np.float32)
    xmax = np.zeros(nmod, dtype=np.int32)
    margin = np.zeros(nmod, dtype=np.float64)
    ptr = lambda a: ctypes.c_void_p(a.ctypes.data)
    _check(lib().gemm2m_debug_residue_reduction(nmod, ptr(y0), ptr(cq), ptr(inv), ptr(xmax), ptr(margin)),
           "gemm2m_debug_residue_reduction")
    return dict(y0_bits=y0, cq=cq, inv_m=inv, xmax=xmax, margin=margin)


def debug_tables_real(nmod, k):
    """Host-side constants of the real scheme (see gemm2m_debug_tables_real)."""
    import numpy as np
    mods = np.zeros(nmod, dtype=np.int32)
    scale = np.zeros(4, dtype=np.int32)
    g = np.zeros((nmod, 5), dtype=np.float64)
    mc = np.zeros(5, dtype=np.float64)
    nch = np.zeros(1, dtype=np.int32)
    y0 = np.zeros(nmod, dtype=np.int32)
    cq = np.zeros(nmod, dtype=np.float32)
    inv = np.zeros(nmod, dtype=np.float32)
    xmax = np.zeros(nmod, dtype=np.int32)
    margin = np.zeros(nmod, dtype=np.float64)
    ptr = lambda a: ctypes.c_void_p(a.ctypes.data)
    _check(lib().gemm2m_debug_tables_real(nmod, k, ptr(mods), ptr(scale), ptr(g), ptr(mc), ptr(nch), ptr(y0), ptr(cq), ptr(inv),
                                          ptr(xmax), ptr(margin)), "gemm2m_debug_tables_real")
    return dict(moduli=mods, Pt=int(scale[0]), PA=int(scale[1]), PB=int(scale[2]), ck=int(scale[3]), g=g, Mc=mc, nchunks=int(nch[0]),
                y0_bits=y0, cq=cq, inv_m=inv, xmax=xmax, margin=margin)
