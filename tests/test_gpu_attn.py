"""GPU parity of lw_attn_decode against the fp64 oracle, element by element: cache formats, head
counts and widths, grouped-query ratios, ragged position counts, peaked and flat score profiles."""
import numpy as np
import pytest

import oracle
from paper_2605_20706_b200 import lw, synth

from gpu_util import Guarded

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

FMTS = [lw.F16, lw.Q8_0, lw.Q4_0]
RTOL, ATOL = 1e-4, 1e-6           # |out - out_ref| <= RTOL * sum_t p_t |v_t| + ATOL  (fp64 oracle)


@pytest.fixture(autouse=True)
def _reset_variant():
    yield
    lw.set_attn_variant(lw.ATTN_AUTO)


def make_case(fmt, n_head, n_kv, hd, n_pos, seed, k_std=1.0):
    width = n_kv * hd
    K = oracle.quantize(fmt, synth.kv_cache(seed, 0, n_pos, width, k_std))
    V = oracle.quantize(fmt, synth.kv_cache(seed, 1, n_pos, width))
    q = synth.query(seed, 0, n_head, hd)
    return K, V, q


def gpu_attn(fmt, K, V, q, n_head, n_kv, hd, n_pos, scale, repeat=1, variant=lw.ATTN_AUTO):
    lw.set_attn_variant(variant)
    k = torch.from_numpy(K).cuda()
    v = torch.from_numpy(V).cuda()
    qd = torch.from_numpy(np.ascontiguousarray(q, dtype=np.float32)).cuda()
    out = Guarded((n_head, hd))                # NaN-filled, guard words on both sides
    ws = Guarded(lw.attn_workspace_bytes(n_head, n_kv, hd, n_pos) // 4)
    for _ in range(repeat):
        lw.attn_decode(fmt, k, v, qd, out.t, n_head, n_kv, hd, n_pos, scale, ws.t)
    torch.cuda.synchronize()
    assert lw.device_status() == 0
    out.check("attention output")
    ws.check("attention workspace")
    return out.t.cpu().numpy()


def check(out, ref, S, what):
    out = np.asarray(out, dtype=np.float64)
    assert np.isfinite(out).all(), what
    worst = float((np.abs(out - ref) / (RTOL * S + ATOL)).max())
    assert worst <= 1.0, "%s: worst error/tolerance ratio %.3g" % (what, worst)
    return worst


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("n_head,n_kv,hd,n_pos", [
    (32, 8, 128, 1), (32, 8, 128, 15), (32, 8, 128, 16), (32, 8, 128, 17), (32, 8, 128, 1000), (32, 8, 128, 4099),
    (32, 8, 64, 777), (8, 8, 128, 300), (16, 8, 128, 513), (28, 4, 128, 345), (16, 2, 64, 2049), (8, 1, 256, 130),
    (64, 8, 128, 97), (12, 4, 32, 1500), (5, 5, 64, 63), (24, 2, 128, 260), (36, 4, 128, 129), (4, 4, 256, 31),
    (24, 8, 128, 6000), (8, 2, 128, 2500), (4, 1, 128, 700), (16, 4, 64, 9001), (2, 2, 128, 33), (32, 8, 128, 40000)])
def test_attn_matches_oracle(fmt, n_head, n_kv, hd, n_pos):
    K, V, q = make_case(fmt, n_head, n_kv, hd, n_pos, seed=70 + fmt)
    scale = 1.0 / np.sqrt(hd)
    ref, S = oracle.attn_decode(fmt, K, V, q, n_head, n_kv, hd, n_pos, scale)
    for variant in (lw.ATTN_AUTO, lw.ATTN_GENERAL):
        out = gpu_attn(fmt, K, V, q, n_head, n_kv, hd, n_pos, scale, variant=variant)
        check(out, ref, S, "fmt %d heads %d/%d dim %d pos %d variant %d" % (fmt, n_head, n_kv, hd, n_pos, variant))


def test_which_shapes_take_the_tensor_core_kernel():
    for fmt in FMTS:
        assert lw.query_attn_variant(fmt, 32, 8, 128, 4096) == lw.ATTN_TENSOR
        assert lw.query_attn_variant(fmt, 32, 8, 64, 100) == lw.ATTN_TENSOR
        assert lw.query_attn_variant(fmt, 8, 8, 128, 1) == lw.ATTN_TENSOR
        assert lw.query_attn_variant(fmt, 64, 8, 128, 4096) == lw.ATTN_TENSOR       # two batches of four query heads
        assert lw.query_attn_variant(fmt, 8, 1, 256, 4096) == lw.ATTN_GENERAL
        assert lw.query_attn_variant(fmt, 5, 5, 64, 4096) == lw.ATTN_GENERAL
    assert lw.query_attn_variant(lw.Q8_0, 4, 1, 128, 64) == lw.ATTN_GENERAL         # 136-byte rows: not 16-byte pieces
    assert lw.query_attn_variant(lw.F16, 4, 1, 128, 64) == lw.ATTN_TENSOR
    lw.set_attn_variant(lw.ATTN_GENERAL)
    assert lw.query_attn_variant(lw.Q8_0, 32, 8, 128, 4096) == lw.ATTN_GENERAL


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("scale,k_std", [(0.0, 1.0), (1.0, 1.0), (0.02, 0.1), (4.0, 1.0)])
def test_flat_and_peaked_score_profiles(fmt, scale, k_std):
    # scale 0: plain average; scale 1 / 4 without the 1/sqrt(d) factor: scores of +-20 .. +-100, one or two
    # positions carry the whole sum
    n_head, n_kv, hd, n_pos = 32, 8, 128, 2500
    K, V, q = make_case(fmt, n_head, n_kv, hd, n_pos, seed=80, k_std=k_std)
    ref, S = oracle.attn_decode(fmt, K, V, q, n_head, n_kv, hd, n_pos, scale)
    for variant in (lw.ATTN_AUTO, lw.ATTN_GENERAL):
        out = gpu_attn(fmt, K, V, q, n_head, n_kv, hd, n_pos, scale, variant=variant)
        check(out, ref, S, "fmt %d scale %g variant %d" % (fmt, scale, variant))


@pytest.mark.parametrize("fmt", FMTS)
def test_repeated_calls_share_a_workspace(fmt):
    n_head, n_kv, hd, n_pos = 32, 8, 128, 3000
    K, V, q = make_case(fmt, n_head, n_kv, hd, n_pos, seed=90)
    scale = 1.0 / np.sqrt(hd)
    ref, S = oracle.attn_decode(fmt, K, V, q, n_head, n_kv, hd, n_pos, scale)
    out = gpu_attn(fmt, K, V, q, n_head, n_kv, hd, n_pos, scale, repeat=3)
    check(out, ref, S, "fmt %d repeated" % fmt)


def test_argument_errors_enqueue_nothing():
    n_head, n_kv, hd, n_pos = 8, 2, 64, 40
    K, V, q = make_case(lw.Q8_0, n_head, n_kv, hd, n_pos, seed=95)
    k, v = torch.from_numpy(K).cuda(), torch.from_numpy(V).cuda()
    qd = torch.from_numpy(q).cuda()
    out = torch.full((n_head, hd), 7.0, dtype=torch.float32, device="cuda")
    ws = torch.empty(lw.attn_workspace_bytes(n_head, n_kv, hd, n_pos) // 4, dtype=torch.float32, device="cuda")
    L = lw.lib()

    def call(fmt=lw.Q8_0, kk=k, vv=v, qq=qd, oo=out, nh=n_head, nk=n_kv, d=hd, t=n_pos, scale=0.1, w=ws, wb=None):
        wb = w.numel() * 4 if wb is None else wb
        return L.lw_attn_decode(fmt, lw._addr(kk), lw._addr(vv), lw._addr(qq), lw._addr(oo), nh, nk, d, t, scale,
                                lw._addr(w), wb, None)

    assert call(fmt=lw.Q4_K) == lw.ERR_FORMAT and call(fmt=77) == lw.ERR_FORMAT
    assert call(nh=7) == lw.ERR_SHAPE and call(d=48) == lw.ERR_SHAPE and call(t=0) == lw.ERR_SHAPE
    assert call(scale=float("nan")) == lw.ERR_SHAPE
    assert call(kk=None) == lw.ERR_NULL and call(oo=None) == lw.ERR_NULL
    assert call(qq=qd.data_ptr() + 4) == lw.ERR_ALIGN
    assert call(wb=1024) == lw.ERR_WORKSPACE
    torch.cuda.synchronize()
    assert (out == 7.0).all()
    assert call() == lw.OK
    torch.cuda.synchronize()
    assert not (out == 7.0).any()
