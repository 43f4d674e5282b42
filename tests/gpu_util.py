"""Helpers shared by the GPU parity tests: seeded inputs, oracle-quantised weights, tolerance, and
output buffers with guard words on both sides (the bounds check of these tests: a kernel that writes
one element before or past its output changes a guard word)."""
from concurrent.futures import ThreadPoolExecutor
import os

import numpy as np

import oracle
from paper_2605_20706_b200 import synth

RTOL, ATOL = 1e-4, 1e-6           # |y - y_ref| <= RTOL * sum|w x| + ATOL  (fp64 oracle)
NMSE_MAX = 1e-7                   # the paper's op-validation threshold [Sec 3.2]


def quantized_weights(fmt, rows, cols, seed, tensor_id=0, std=0.02, outlier_p=0.0):
    """Oracle-quantised synthetic weight matrix as a flat uint8 array (threads over row slabs)."""
    w = synth.weights(seed, tensor_id, rows, cols, std, outlier_p)
    rb = oracle.row_bytes(fmt, cols)
    out = np.empty(rows * rb, dtype=np.uint8)
    nthr = min(os.cpu_count() or 1, max(1, rows // 64))
    bounds = [rows * i // nthr for i in range(nthr + 1)]

    def job(i):
        r0, r1 = bounds[i], bounds[i + 1]
        if r1 > r0:
            out[r0 * rb:r1 * rb] = oracle.quantize(fmt, w[r0:r1])

    if nthr == 1:
        job(0)
    else:
        with ThreadPoolExecutor(nthr) as pool:
            list(pool.map(job, range(nthr)))
    return out


def check_matvec(y_gpu, y_ref, s_ref, what=""):
    """Element-wise tolerance of the benchmark spec plus the paper's NMSE criterion."""
    y_gpu = np.asarray(y_gpu, dtype=np.float64).reshape(y_ref.shape)
    err = np.abs(y_gpu - y_ref)
    tol = RTOL * s_ref + ATOL
    worst = float((err / tol).max())
    assert np.isfinite(y_gpu).all(), what
    assert worst <= 1.0, "%s: worst error/tolerance ratio %.3g" % (what, worst)
    denom = float((y_ref ** 2).sum())
    if denom > 0:
        nmse = float(((y_gpu - y_ref) ** 2).sum() / denom)
        assert nmse <= NMSE_MAX, "%s: NMSE %.3g" % (what, nmse)
    return worst


GUARD_WORDS = 64                  # 256 bytes on each side: keeps the 16-byte alignment the library asks for
GUARD_PATTERN = 0x5AC3A55A        # as int32; as a float it is a finite number no kernel here produces


class Guarded:
    """A device buffer of `n` 4-byte elements between two runs of guard words.  `.t` is the tensor to hand to
    the library (viewed as `dtype`, shaped `shape`); `.check()` asserts that no guard word changed."""

    def __init__(self, shape, fill=float("nan"), dtype=None):
        import torch
        dtype = dtype or torch.float32
        assert dtype in (torch.float32, torch.int32)
        shape = (shape,) if isinstance(shape, int) else tuple(shape)
        n = int(np.prod(shape))
        self.n = n
        self.raw = torch.full((n + 2 * GUARD_WORDS,), GUARD_PATTERN, dtype=torch.int32, device="cuda")
        self.t = self.raw[GUARD_WORDS:GUARD_WORDS + n].view(dtype).view(shape)
        if fill is not None:
            self.t.fill_(fill)

    def check(self, what=""):
        import torch
        torch.cuda.synchronize()
        lo = self.raw[:GUARD_WORDS].cpu().numpy()
        hi = self.raw[GUARD_WORDS + self.n:].cpu().numpy()
        assert (lo == GUARD_PATTERN).all(), "%s: write before the start of the buffer" % what
        assert (hi == GUARD_PATTERN).all(), "%s: write past the end of the buffer" % what
