"""GPU tests of what include/lw.h promises beyond the ordinary parity cases: the error bound of every
kernel variant on activations built to defeat it (huge outliers sitting on zero weights), non-finite
activations, every tunable geometry of the streaming kernels against the oracle, and the bounded-wait
fault path (provoked without anything in flight: one copy is simply never requested)."""
import os
import subprocess
import sys

import numpy as np
import pytest

import oracle
from paper_2605_20706_b200 import lw, synth

from gpu_util import ATOL, RTOL, Guarded, check_matvec, quantized_weights

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

FMTS = [lw.F16, lw.Q8_0, lw.Q4_0, lw.Q4_K, lw.Q6_K, lw.Q5_K, lw.Q2_K, lw.Q4_1, lw.Q5_0, lw.Q5_1]
ALL_VARIANTS = [lw.VARIANT_AUTO, lw.VARIANT_GENERIC, lw.VARIANT_STREAM, lw.VARIANT_IDOT]
# the extra term E = c * sum_k What_k * A_k of the header's accuracy statement, per launched variant
C_EXTRA = {lw.VARIANT_GENERIC: 0.0, lw.VARIANT_STREAM: 2.0 ** -16, lw.VARIANT_IDOT: 2.0 ** -18, lw.VARIANT_TILE: 0.0,
           lw.VARIANT_MMA: 0.0}


@pytest.fixture(autouse=True)
def _reset():
    yield
    lw.set_variant(lw.VARIANT_AUTO)
    lw.set_overlap(False)
    lw.set_tuning()


def _run(fmt, blocks, rows, cols, X, variant=lw.VARIANT_AUTO, batch=1):
    lw.set_variant(variant)
    w = torch.from_numpy(np.ascontiguousarray(blocks)).cuda()
    x = torch.from_numpy(np.ascontiguousarray(X, dtype=np.float32)).cuda()
    y = Guarded((batch, rows))
    lw.matvec(fmt, w, rows, cols, x, y.t, batch)
    torch.cuda.synchronize()
    y.check("Y")
    return y.t.cpu().numpy()


def _extra_term(fmt, blocks, rows, cols, X, c):
    """E of the header: c * sum_k What_k * A_k with What / A the largest decoded |w| / largest |x| of the
    aligned run of 32 columns that contains k."""
    if c == 0.0:
        return np.zeros((1, rows))
    deq = np.abs(oracle.dequant(fmt, blocks, rows * cols).astype(np.float64)).reshape(rows, cols // 32, 32)
    what = deq.max(axis=2)                                             # rows x runs
    a = np.abs(X.astype(np.float64)).reshape(cols // 32, 32).max(axis=1)
    return (c * 32.0 * (what * a[None, :]).sum(axis=1))[None, :]


def _adversarial(fmt, rows, cols, seed, zero_rest_of_vector):
    """Weights with one all-zero column per aligned run of 32 (so that column decodes to zero or next to
    it in every row), activations of 1e-2 everywhere except a value of 1e3..1e6 on exactly those columns."""
    rng = np.random.default_rng(seed)
    w32 = synth.weights(seed, fmt, rows, cols, 0.02, 0.0).copy()
    runs = cols // 32
    hot = np.arange(runs) * 32 + rng.integers(0, 32, runs)
    w32[:, hot] = 0.0
    blocks = oracle.quantize(fmt, w32)
    X = (1e-2 * rng.standard_normal(cols)).astype(np.float32)
    X[hot] = (10.0 ** (3 + np.arange(runs) % 4) * rng.choice([-1.0, 1.0], runs)).astype(np.float32)
    if zero_rest_of_vector:                       # one live run per vector: no other term lends its tolerance
        keep = rng.integers(0, runs)
        mask = np.zeros(cols, bool)
        mask[32 * keep:32 * keep + 32] = True
        X[~mask] = 0.0
    return blocks, X[None, :]


@pytest.mark.parametrize("zero_rest", [False, True])
@pytest.mark.parametrize("variant", ALL_VARIANTS)
@pytest.mark.parametrize("fmt", FMTS)
def test_outliers_on_zero_weights_stay_inside_the_stated_bound(fmt, variant, zero_rest):
    # The streaming variants apply block offsets after the dot product and (IDOT) hold the activations
    # as block fixed point, so an outlier that meets a zero weight leaves an absolute error that the
    # tolerance 1e-4 * sum|w x| + 1e-6 alone does not cover: the header states the extra term, this
    # test asserts it, and asserts that the generic variant needs none.
    rows, cols = 48, 4096
    blocks, X = _adversarial(fmt, rows, cols, seed=90 + fmt, zero_rest_of_vector=zero_rest)
    lw.set_variant(variant)
    launched = lw.query_variant(fmt, rows, cols, 1)
    c = 0.0 if fmt == lw.F16 else C_EXTRA[launched]
    y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, 1)
    y = _run(fmt, blocks, rows, cols, X, variant)
    assert np.isfinite(y).all()
    bound = RTOL * s_ref + ATOL + _extra_term(fmt, blocks, rows, cols, X, c)
    worst = float((np.abs(y.astype(np.float64) - y_ref) / bound).max())
    assert worst <= 1.0, "variant %d launched %d: error / bound = %.3g" % (variant, launched, worst)


@pytest.mark.parametrize("fmt,kernel", [(lw.Q8_0, lw.VARIANT_TILE), (lw.Q4_0, lw.VARIANT_TILE), (lw.Q8_0, lw.VARIANT_MMA),
                                        (lw.Q4_0, lw.VARIANT_MMA), (lw.Q5_0, lw.VARIANT_MMA), (lw.Q6_K, lw.VARIANT_MMA)])
def test_batched_kernels_need_no_extra_term(fmt, kernel):
    # the batched fp32 tile kernel decodes every weight exactly before it multiplies, and the tensor-core kernel
    # multiplies exact integer codes with two bf16 terms that add up to the activation within 2^-16: the plain
    # tolerance holds on the same adversarial activations (eight columns, each with its own outliers), as the
    # header states
    rows, cols, batch = 48, 4096, 8
    cols_x = []
    for b in range(batch):
        blocks, X = _adversarial(fmt, rows, cols, seed=90 + fmt, zero_rest_of_vector=bool(b & 1))
        cols_x.append(np.roll(X[0], 0) * (1.0 + b))
    X = np.stack(cols_x).astype(np.float32)
    y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, batch)
    lw.set_variant(kernel)
    assert lw.query_variant(fmt, rows, cols, batch) == kernel
    y = _run(fmt, blocks, rows, cols, X, kernel, batch)
    worst = float((np.abs(y.astype(np.float64) - y_ref) / (RTOL * s_ref + ATOL)).max())
    assert worst <= 1.0, "kernel %d: error / tolerance = %.3g" % (kernel, worst)
    # and a non-finite activation reaches every output of its column only
    for bad in (np.nan, np.inf, -np.inf):
        Xb = X.copy()
        Xb[3, 100] = bad
        y = _run(fmt, blocks, rows, cols, Xb, kernel, batch)
        assert not np.isfinite(y[3]).any() and np.isfinite(np.delete(y, 3, axis=0)).all()
    # extreme magnitudes survive the split into terms: a huge value (the sums of code * x stay finite up to about
    # 2^115, the limit the header states for the batched kernels) and a denormal
    Xe = np.zeros((batch, cols), np.float32)
    Xe[0, 7] = 1e30
    Xe[1, 9] = 1e-41
    Xe[2, :] = 2.0 ** -100
    y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, Xe, batch)
    y = _run(fmt, blocks, rows, cols, Xe, kernel, batch)
    finite = np.isfinite(y_ref.astype(np.float32))
    assert (np.abs(y.astype(np.float64) - y_ref)[finite] <= (RTOL * s_ref + ATOL)[finite]).all()


@pytest.mark.parametrize("fmt,c_extra", [(lw.Q4_K, 2.0 ** -18), (lw.Q5_K, 2.0 ** -18), (lw.F16, 2.0 ** -30),
                                         (lw.Q4_1, 2.0 ** -18), (lw.Q5_1, 2.0 ** -18), (lw.Q2_K, 2.0 ** -18)])
def test_formats_with_an_extra_term_on_the_tensor_cores_stay_inside_the_stated_bound(fmt, c_extra):
    # q4_K / q5_K in the batched tensor-core kernel apply the sub-block offsets to sums of activations, like the
    # fp32-activation streaming family: the header gives them the extra term with c = 2^-18; f16 holds the
    # activations as two f16 terms relative to each block's largest magnitude, which can lose up to 2^-38 of that
    # magnitude per element (c = 2^-30 stated).  Asserted here on the adversarial activations (eight columns, each
    # with its own outliers); a non-finite activation stays in its column
    rows, cols, batch = 48, 4096, 8
    cols_x = []
    for b in range(batch):
        blocks, X = _adversarial(fmt, rows, cols, seed=90 + fmt, zero_rest_of_vector=bool(b & 1))
        cols_x.append(X[0] * (1.0 + b))
    X = np.stack(cols_x).astype(np.float32)
    y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, batch)
    lw.set_variant(lw.VARIANT_MMA)
    assert lw.query_variant(fmt, rows, cols, batch) == lw.VARIANT_MMA
    y = _run(fmt, blocks, rows, cols, X, lw.VARIANT_MMA, batch)
    for b in range(batch):
        bound = RTOL * s_ref[b] + ATOL + _extra_term(fmt, blocks, rows, cols, X[b:b + 1], c_extra)[0]
        worst = float((np.abs(y[b].astype(np.float64) - y_ref[b]) / bound).max())
        assert worst <= 1.0, "column %d: error / bound = %.3g" % (b, worst)
    Xb = X.copy()
    Xb[3, 100] = np.nan
    y = _run(fmt, blocks, rows, cols, Xb, lw.VARIANT_MMA, batch)
    assert not np.isfinite(y[3]).any() and np.isfinite(np.delete(y, 3, axis=0)).all()


@pytest.mark.parametrize("variant", ALL_VARIANTS)
@pytest.mark.parametrize("fmt", FMTS)
def test_non_finite_activations_reach_the_output(fmt, variant):
    # a NaN or Inf in X must not be rounded away by the fixed-point conversion: every row touches
    # every column, so every output is non-finite, as it is in fp32 / fp64 arithmetic
    rows, cols = 40, 2048
    blocks = quantized_weights(fmt, rows, cols, seed=95, tensor_id=fmt)
    for bad, where in ((np.nan, 5), (np.inf, cols - 1), (-np.inf, 1000)):
        X = synth.activations(95, fmt, 1, cols).copy()
        X[0, where] = bad
        y = _run(fmt, blocks, rows, cols, X, variant)
        assert not np.isfinite(y).any(), "fmt %d variant %d: %r at %d was lost" % (fmt, variant, bad, where)
    # several non-finite values in one run of 16 (the kernels spot them through a sum of integer codes that wraps
    # around for 5, 10 and 15 of them), in runs that belong to different threads, and whole runs of them
    for count in (2, 5, 8, 10, 15, 16):
        X = synth.activations(95, fmt, 1, cols).copy()
        X[0, 512:512 + count] = np.nan
        X[0, 1040:1040 + count:2] = np.inf
        y = _run(fmt, blocks, rows, cols, X, variant)
        assert not np.isfinite(y).any(), "fmt %d variant %d: %d NaNs in a run were lost" % (fmt, variant, count)
    # the same through a grouped call, and a zero elsewhere in the group does not mask it
    X = np.zeros((1, cols), np.float32)
    X[0, 77] = np.nan
    lw.set_variant(variant)
    w = torch.from_numpy(blocks).cuda()
    x = torch.from_numpy(X).cuda()
    ys = [Guarded((1, rows)), Guarded((1, rows))]
    lw.matvec_group(fmt, cols, [(w, rows, x, ys[0].t), (w, rows, x, ys[1].t)])
    torch.cuda.synchronize()
    for y in ys:
        y.check("grouped Y")
        assert not np.isfinite(y.t.cpu().numpy()).any()
    assert lw.device_status() == 0


TUNING_SHAPES = [(lw.Q4_K, 301, 4096), (lw.Q4_0, 150, 14336), (lw.Q8_0, 517, 2048), (lw.F16, 203, 4096),
                 (lw.Q6_K, 77, 4096), (lw.Q2_K, 333, 8192)]


@pytest.mark.parametrize("stage_kb", [0, 24, 40, 64])
@pytest.mark.parametrize("stages", [0, 2, 3, 4])
@pytest.mark.parametrize("groups", [1, 2])
def test_every_tunable_geometry_against_the_oracle(groups, stages, stage_kb):
    # lw_set_tuning changes ring depth, rows per slot and the stage-completion path; each geometry the
    # sweep may launch is checked here against the oracle (not against another kernel of the library)
    lw.set_tuning(groups, stages, stage_kb)
    for fmt, rows, cols in TUNING_SHAPES:
        info = lw.plan_info(fmt, rows, cols)
        assert info["worker_groups"] == groups
        if stage_kb:
            assert info["stage_bytes"] <= max(stage_kb * 1024, lw.row_bytes(fmt, cols) * 4)
        blocks = quantized_weights(fmt, rows, cols, seed=96, tensor_id=fmt, outlier_p=0.01)
        X = synth.activations(96, fmt, 1, cols)
        y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, 1, nthreads=4)
        for overlap in (False, True):
            lw.set_overlap(overlap)
            y = _run(fmt, blocks, rows, cols, X)
            check_matvec(y, y_ref, s_ref, "groups %d slots %d slot %d KB fmt %d" % (groups, stages, stage_kb, fmt))
    assert lw.device_status() == 0


def test_single_group_ctas_from_the_environment_against_the_oracle():
    # LW_WORKER_GROUPS=1 is read once per process, so a child process runs it; the child compares with
    # the oracle
    code = r"""
import numpy as np, torch
import oracle
from paper_2605_20706_b200 import lw, synth
worst = 0.0
for fmt, rows, cols in [(lw.Q4_K, 301, 4096), (lw.Q4_0, 150, 14336), (lw.Q8_0, 37, 2048), (lw.F16, 64, 4096),
                        (lw.Q6_K, 77, 4096), (lw.Q5_K, 77, 4096), (lw.Q2_K, 77, 4096),
                        (lw.Q4_1, 77, 4096), (lw.Q5_0, 77, 4096), (lw.Q5_1, 77, 4096)]:
    assert lw.plan_info(fmt, rows, cols)["worker_groups"] == 1
    blocks = oracle.quantize(fmt, synth.weights(7, fmt, rows, cols, 0.02, 0.0))
    X = synth.activations(7, fmt, 1, cols)
    y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, 1)
    wd, x = torch.from_numpy(blocks).cuda(), torch.from_numpy(X).cuda()
    y = torch.full((rows,), float("nan"), dtype=torch.float32, device="cuda")
    lw.matvec(fmt, wd, rows, cols, x, y)
    torch.cuda.synchronize()
    assert lw.device_status() == 0
    err = np.abs(y.cpu().numpy().astype(np.float64)[None, :] - y_ref)
    worst = max(worst, float((err / (1e-4 * s_ref + 1e-6)).max()))
print("WORST", worst)
assert worst <= 1.0
"""
    env = dict(os.environ, LW_WORKER_GROUPS="1")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env["PYTHONPATH"] = root + os.pathsep + env.get("PYTHONPATH", "")
    out = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stdout + out.stderr


def test_a_copy_that_never_comes_is_reported_and_the_library_stays_usable():
    # lw_debug_drop_copy: the producer thread never requests one unit's copy, so nothing is in flight
    # for it and the group's wait runs out after its limit; the kernel records the fault and returns,
    # lw_device_status reports it once, and the next ordinary call passes parity.
    fmt, rows, cols = lw.Q4_K, 4096, 4096
    blocks = quantized_weights(fmt, rows, cols, seed=97)
    X = synth.activations(97, 0, 1, cols)
    y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, 1, nthreads=8)
    assert lw.device_status() == 0
    w = torch.from_numpy(blocks).cuda()
    x = torch.from_numpy(X).cuda()
    y = Guarded((1, rows))
    lw.debug_drop_copy(1)
    lw.matvec(fmt, w, rows, cols, x, y.t, 1)
    torch.cuda.synchronize()                      # the kernel ends by itself (two bounded waits of ~0.1 s)
    y.check("Y of the faulted call")
    assert lw.device_status() != 0                # the fault was recorded ...
    assert lw.device_status() == 0                # ... and reading it cleared it
    y2 = _run(fmt, blocks, rows, cols, X)         # the request was consumed: this call is an ordinary one
    check_matvec(y2, y_ref, s_ref, "call after the fault")
    assert lw.device_status() == 0


@pytest.mark.parametrize("overlap", [0, 2])
def test_a_copy_that_never_comes_in_the_tensor_core_kernel(overlap):
    # the same aid in the batched tensor-core kernel: from its second stage on a CTA's producer requests nothing, the
    # compute warps' wait for that stage runs out, the fault is recorded, the CTA stops waiting and the kernel ends;
    # the next call is an ordinary one.  Both launch forms (self-clearing cooperative launch, clearing kernel chained
    # by programmatic dependent launch).
    fmt, rows, cols, batch = lw.Q4_0, 4096, 4096, 8
    blocks = quantized_weights(fmt, rows, cols, seed=98)
    X = synth.activations(98, 0, batch, cols)
    y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, batch, nthreads=8)
    assert lw.device_status() == 0
    w = torch.from_numpy(blocks).cuda()
    x = torch.from_numpy(X).cuda()
    y = Guarded((batch, rows))
    lw.set_variant(lw.VARIANT_AUTO)
    lw.set_overlap(overlap)
    try:
        assert lw.query_variant(fmt, rows, cols, batch) == lw.VARIANT_MMA
        lw.debug_drop_copy(1)
        lw.matvec(fmt, w, rows, cols, x, y.t, batch)
        torch.cuda.synchronize()                  # the kernel ends by itself (one bounded wait of ~0.1 s per warp)
        y.check("Y of the faulted call")
        assert lw.device_status() != 0
        assert lw.device_status() == 0
        y2 = _run(fmt, blocks, rows, cols, X, lw.VARIANT_AUTO, batch)
        check_matvec(y2, y_ref, s_ref, "call after the fault")
        assert lw.device_status() == 0
    finally:
        lw.set_overlap(0)
