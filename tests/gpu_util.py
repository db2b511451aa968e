"""Helpers for the GPU parity tests: column-major numpy <-> torch CUDA tensors, workspace handling, stage dumps."""
import numpy as np
import torch

from paper_2609_05419_b200 import binding as b


def to_dev(a):
    """numpy (rows, cols) array -> CUDA tensor of the same shape stored column-major."""
    a = np.asfortranarray(a)
    return torch.from_numpy(np.ascontiguousarray(a.T)).cuda().t()


def empty_dev(rows, cols, dtype, ld=None, fill=None):
    ld = rows if ld is None else ld
    buf = torch.empty((cols, max(ld, 1)), dtype=dtype, device="cuda")
    if fill is not None:
        buf.fill_(fill)
    return buf[:, :rows].t()


def to_host(t):
    """Column-major CUDA tensor -> numpy Fortran-ordered array."""
    return np.asfortranarray(t.t().contiguous().cpu().numpy().T)


class Workspace:
    def __init__(self, nbytes):
        self.buf = torch.zeros(max(int(nbytes), 256), dtype=torch.uint8, device="cuda")
        b.set_workspace(self.buf)

    def close(self):
        torch.cuda.synchronize()
        b.set_workspace(None)
        self.buf = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def stages(self, op, m, n, k, nmod):
        """Copies of the intermediate stages of the last call: exponents, residue planes, C+- planes."""
        torch.cuda.synchronize()
        lay = b.workspace_layout(op, m, n, k, nmod)
        raw = self.buf.cpu().numpy()
        herk = op == b.OP_ZHERK
        rows_a = n if herk else m
        kp, ldp = lay["kp"], lay["ldp"]
        out = dict(layout=lay)
        out["eA"] = raw[lay["off_exp_a"]: lay["off_exp_a"] + 4 * rows_a].view(np.int32).copy()
        n2 = min(nmod, 22)                      # 2M moduli: planes X+ then X-; 3M moduli (hybrid): X_r, X_i, X_r + X_i
        if op == b.OP_ZGEMM_EISENSTEIN:         # two planes for every modulus of the Eisenstein set
            n2 = nmod
        n3 = nmod - n2

        def split(off, rows, ld):
            flat = raw[off: off + (2 * n2 + 3 * n3) * rows * ld].view(np.int8)
            two = flat[: 2 * n2 * rows * ld].reshape(2, n2, rows, ld)
            three = flat[2 * n2 * rows * ld:].reshape(3, n3, rows, ld)
            return two, three

        if not herk:
            out["Apm"], out["A3"] = split(lay["off_apm"], rows_a, kp)
            out["eB"] = raw[lay["off_exp_b"]: lay["off_exp_b"] + 4 * n].view(np.int32).copy()
            out["Bpm"], out["B3"] = split(lay["off_bpm"], n, kp)
            out["Cpm"], out["C3"] = split(lay["off_cpm"], n, ldp)
        else:
            out["Apm"] = raw[lay["off_apm"]: lay["off_apm"] + 2 * nmod * rows_a * kp].view(np.int8).reshape(2, nmod, rows_a, kp)
            out["Cpm"] = raw[lay["off_cpm"]: lay["off_cpm"] + nmod * n * ldp].view(np.int8).reshape(1, nmod, n, ldp)
        return out


def ulp_distance(x, y):
    """Distance in units of the last place between float64 arrays (same sign assumed or both tiny)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    y = np.ascontiguousarray(y, dtype=np.float64)
    xi = x.view(np.int64).astype(object)
    yi = y.view(np.int64).astype(object)
    fix = lambda v: np.where(v < 0, -(v & 0x7FFFFFFFFFFFFFFF), v)
    return np.abs(fix(xi) - fix(yi)).astype(np.float64)
