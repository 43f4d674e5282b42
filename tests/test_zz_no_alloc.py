"""lw_attn_decode_static -- the attention entry point for callers that cannot allocate device memory
(a process whose GPU memory all belongs to a pool it cannot reach from the call site, a plug-in that
must not call cudaMalloc inside a latency-critical loop, code linked without an allocator).  Its
partial results live in a fixed array inside the library, so it must give what lw_attn_decode gives
with a caller workspace.  Checked on two calls in a row (the second finds the first call's leftovers
in the array), through the C ABI, against lw_attn_decode AND against the fp64 oracle, within the
tolerance of the attention parity tests; both kernels (tensor-core and general) go through the array,
and the largest shape it takes sits next to the smallest one it refuses.  The file sorts last so a run
that stops at the first failure has already run everything else."""
import numpy as np
import pytest

import oracle
from paper_2605_20706_b200 import lw, synth

from gpu_util import Guarded

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-4, 1e-6           # |out - out_ref| <= RTOL * sum_t p_t |v_t| + ATOL  (fp64 oracle)


def _case(fmt, n_head, n_kv, hd, n_pos, seed):
    width = n_kv * hd
    K = oracle.quantize(fmt, synth.kv_cache(seed, 0, n_pos, width))
    V = oracle.quantize(fmt, synth.kv_cache(seed, 1, n_pos, width))
    q = synth.query(seed, 0, n_head, hd)
    return K, V, q


def _static_call(fmt, K, V, q, out, n_head, n_kv, hd, n_pos, scale):
    return lw.lib().lw_attn_decode_static(fmt, lw._addr(K), lw._addr(V), lw._addr(q), lw._addr(out), n_head, n_kv, hd,
                                          n_pos, scale, None)


# (format, query heads, KV heads, head_dim, positions, scale, forced attention variant, kernel expected)
CASES = [
    (lw.Q8_0, 32, 8, 128, 3001, 0.0884, lw.ATTN_AUTO, lw.ATTN_TENSOR),
    (lw.Q4_0, 32, 8, 64, 517, 0.125, lw.ATTN_AUTO, lw.ATTN_TENSOR),
    (lw.F16, 8, 1, 256, 130, 0.0625, lw.ATTN_AUTO, lw.ATTN_GENERAL),        # head_dim 256: general kernel
    (lw.Q8_0, 32, 8, 128, 700, 0.0884, lw.ATTN_GENERAL, lw.ATTN_GENERAL),   # general kernel forced
    (lw.Q8_0, 63, 21, 256, 40, 0.0625, lw.ATTN_AUTO, lw.ATTN_GENERAL),      # 63 * 258 = 16254: the largest that fits
]


def test_static_scratch_matches_workspace_call_and_oracle_twice_in_a_row():
    try:
        for fmt, n_head, n_kv, hd, n_pos, scale, variant, kernel in CASES:   # each case follows the previous one's leftovers
            lw.set_attn_variant(variant)
            assert lw.query_attn_variant(fmt, n_head, n_kv, hd, n_pos) == kernel
            K, V, q = _case(fmt, n_head, n_kv, hd, n_pos, seed=31 + fmt + hd)
            ref, S = oracle.attn_decode(fmt, K, V, q, n_head, n_kv, hd, n_pos, scale)
            tol = RTOL * S + ATOL
            kd, vd, qd = torch.from_numpy(K).cuda(), torch.from_numpy(V).cuda(), torch.from_numpy(q).cuda()
            want = Guarded((n_head, hd))
            ws = Guarded(lw.attn_workspace_bytes(n_head, n_kv, hd, n_pos) // 4)
            lw.attn_decode(fmt, kd, vd, qd, want.t, n_head, n_kv, hd, n_pos, scale, ws.t)
            torch.cuda.synchronize()
            want_np = want.t.double().cpu().numpy()
            assert float((np.abs(want_np - ref) / tol).max()) <= 1.0
            for _ in range(2):
                got = Guarded((n_head, hd))
                assert _static_call(fmt, kd, vd, qd, got.t, n_head, n_kv, hd, n_pos, scale) == lw.OK
                got.check("output of the static-scratch call")
                got_np = got.t.double().cpu().numpy()
                assert np.isfinite(got_np).all()
                assert float((np.abs(got_np - ref) / tol).max()) <= 1.0          # against the oracle
                assert float((np.abs(got_np - want_np) / tol).max()) <= 1.0      # against the workspace entry point
    finally:
        lw.set_attn_variant(lw.ATTN_AUTO)
    assert lw.device_status() == 0


def test_static_scratch_rejects_shapes_beyond_its_array():
    L = lw.lib()
    K, V, q = (torch.from_numpy(a).cuda() for a in _case(lw.Q8_0, 8, 8, 32, 4, seed=40))
    out = torch.full((128, 256), 3.0, dtype=torch.float32, device="cuda")
    # 64 heads of 256 need 64 * 258 = 16512 > 16384 floats per part: refused, nothing enqueued (63 heads fit, above)
    assert _static_call(lw.Q8_0, K, V, q, out, 64, 8, 256, 4, 0.1) == lw.ERR_WORKSPACE
    assert _static_call(lw.Q8_0, K, V, q, out, 128, 8, 256, 4, 0.1) == lw.ERR_WORKSPACE
    assert _static_call(lw.Q4_K, K, V, q, out, 8, 8, 32, 4, 0.1) == lw.ERR_FORMAT
    assert L.lw_attn_decode_static(lw.Q8_0, lw._addr(K), None, lw._addr(q), lw._addr(out), 8, 8, 32, 4, 0.1,
                                   None) == lw.ERR_NULL
    torch.cuda.synchronize()
    assert (out == 3.0).all()
