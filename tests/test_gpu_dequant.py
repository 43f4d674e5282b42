"""GPU parity of lw_dequant against the oracle: bit-for-bit (uint32 patterns, sign of zero included)."""
import numpy as np
import pytest

import oracle
from paper_2605_20706_b200 import lw, synth

from gpu_util import Guarded

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

FMTS = [lw.F16, lw.Q8_0, lw.Q4_0, lw.Q4_K, lw.Q6_K, lw.Q5_K, lw.Q2_K, lw.Q4_1, lw.Q5_0, lw.Q5_1]


def _gpu_dequant(fmt, blocks, n):
    w = torch.from_numpy(blocks).cuda()
    out = Guarded(n)                           # NaN-filled, guard words on both sides
    lw.dequant(fmt, w, n, out.t)
    torch.cuda.synchronize()
    out.check("dequant output")
    return out.t.cpu().numpy()


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("n", [256, 256 * 3, 256 * 1031, 256 * 20000 + 512])
def test_dequant_bit_exact_on_quantised_weights(fmt, n):
    if fmt in (lw.Q4_K, lw.Q6_K, lw.Q5_K, lw.Q2_K):
        n -= n % 256
    x = synth.normal(21, fmt, n, 0.02, 0.01)
    x[: min(n, 4096)] *= -1.0
    blocks = oracle.quantize(fmt, x)
    want = oracle.dequant(fmt, blocks, n)
    got = _gpu_dequant(fmt, blocks, n)
    assert (got.view(np.uint32) == want.view(np.uint32)).all()
    assert lw.device_status() == 0


@pytest.mark.parametrize("fmt", FMTS)
def test_dequant_bit_exact_on_random_bytes(fmt):
    # arbitrary block contents (every nibble / scale field value), fp16 fields forced finite
    rng = np.random.default_rng(31 + fmt)
    nblk = 4099
    bb, be = oracle.block_bytes(fmt), oracle.block_elems(fmt)
    if fmt == lw.F16:
        nblk, bb, be = 4099 * 32, 2, 1
    raw = rng.integers(0, 256, (nblk, bb), dtype=np.uint8)
    raw[:, 1] &= 0xBB                         # clear one exponent bit of the fp16 at bytes 0-1 -> finite
    if fmt in (lw.Q4_K, lw.Q5_K, lw.Q4_1, lw.Q5_1):
        raw[:, 3] &= 0xBB                     # dmin / m too
    if fmt == lw.Q2_K:                        # fp16 d at bytes 80-81, dmin at 82-83
        raw[:, 81] &= 0xBB
        raw[:, 83] &= 0xBB
        raw[::5, 81] |= 0x80
        raw[::7, 80:82] = 0
        raw[::11, 80:82] = [0x01, 0x00]
    elif fmt == lw.Q6_K:                      # its fp16 factor sits at bytes 208-209
        raw[:, 209] &= 0xBB
        raw[::5, 209] |= 0x80
        raw[::7, 208:210] = 0
        raw[::11, 208:210] = [0x01, 0x00]
    elif fmt != lw.F16:
        raw[::5, 1] |= 0x80                   # plenty of negative scales
        raw[::7, 0:2] = 0                     # zero scales
        raw[::11, 0:2] = [0x01, 0x00]         # subnormal scales
    n = nblk * be
    if fmt == lw.F16:
        n -= n % 32
    blocks = raw.reshape(-1)[: oracle.row_bytes(fmt, n)].copy()
    want = oracle.dequant(fmt, blocks, n)
    got = _gpu_dequant(fmt, blocks, n)
    assert np.isfinite(want).all()
    assert (got.view(np.uint32) == want.view(np.uint32)).all()


def test_dequant_sign_of_zero():
    # q4_0 nibble 8 under a negative scale is -0.0 (IEEE product), not +0.0
    x = np.array([-(i - 16) / 8 for i in range(32)] * 8, dtype=np.float32)
    blocks = oracle.quantize(lw.Q4_0, x)
    got = _gpu_dequant(lw.Q4_0, blocks, 256)
    assert got.view(np.uint32)[15] == 0x80000000
    assert (got.view(np.uint32) == oracle.dequant(lw.Q4_0, blocks, 256).view(np.uint32)).all()


def test_dequant_rejects_bad_arguments_on_device():
    w = torch.zeros(64, dtype=torch.uint8, device="cuda")
    out = torch.zeros(64, dtype=torch.float32, device="cuda")
    L = lw.lib()
    assert L.lw_dequant(lw.Q8_0, w.data_ptr() + 2, 32, out.data_ptr(), None) == lw.ERR_ALIGN
    assert L.lw_dequant(lw.Q8_0, w.data_ptr(), 33, out.data_ptr(), None) == lw.ERR_SHAPE
