"""CPU-only checks of the lw library: the shared object loads and exports every symbol the header
declares, the host quantiser reproduces the oracle's bytes, and argument errors are reported
before any CUDA call."""
import os
import re

import numpy as np
import pytest

import oracle
from paper_2605_20706_b200 import build as lw_build
from paper_2605_20706_b200 import lw, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FMTS = [lw.F16, lw.Q8_0, lw.Q4_0, lw.Q4_K, lw.Q6_K, lw.Q5_K, lw.Q2_K, lw.Q4_1, lw.Q5_0, lw.Q5_1]


@pytest.fixture(scope="module", autouse=True)
def _built():
    lw_build.build()


def test_header_symbols_are_exported():
    text = open(os.path.join(ROOT, "include", "lw.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(lw_[a-z0-9_]+)\s*\(", text))
    assert declared, "no declarations found"
    assert declared == set(lw.EXPORTS)
    L = lw.lib()
    for name in declared:
        assert getattr(L, name) is not None


def test_sizes_match_oracle():
    for fmt in FMTS:
        assert lw.block_elems(fmt) == oracle.block_elems(fmt)
        assert lw.block_bytes(fmt) == oracle.block_bytes(fmt)
        for cols in (32, 256, 2048, 4096, 14336, 48, 0, -32):
            assert lw.row_bytes(fmt, cols) == oracle.row_bytes(fmt, cols)
    assert lw.block_elems(29) == 0 and lw.row_bytes(29, 256) == 0


def _adversarial(rng, n):
    x = (rng.standard_normal(n) * 0.02).astype(np.float32)
    x = x.reshape(-1, 256)
    x[1] = 0.0                                    # all-zero super-block
    x[2] = np.abs(x[2])                           # all positive
    x[3] = -np.abs(x[3])                          # all negative
    x[4] = 0.3                                    # constant
    x[5, ::2] = 0.01
    x[5, 1::2] = -0.01                            # ties in |x|
    x[6] *= 1e-6                                  # scales in the fp16 subnormal range
    x[7] *= 1e3
    x[8] = np.where(rng.random(256) < 0.05, x[8] * 10, x[8])
    x[9] = np.round(x[9] * 512) / 512             # many rounding ties
    x[10, 17] = 60000.0                           # largest scales that still fit fp16
    x[11] = np.float32(2.0 ** -24) * rng.integers(-3, 4, 256)
    return x.reshape(-1)


@pytest.mark.parametrize("fmt", FMTS)
def test_host_quantiser_matches_oracle_bytes(fmt):
    rng = np.random.default_rng(100 + fmt)
    x = _adversarial(rng, 256 * 64)
    assert (lw.quantize(fmt, x) == oracle.quantize(fmt, x)).all()
    w = synth.weights(7, fmt, 64, 2048, 0.02, 0.01)
    assert (lw.quantize(fmt, w) == oracle.quantize(fmt, w)).all()
    # wide dynamic range
    y = (rng.standard_normal(256 * 256) * np.exp(rng.uniform(-12, 6, 256 * 256))).astype(np.float32)
    assert (lw.quantize(fmt, y) == oracle.quantize(fmt, y)).all()


@pytest.mark.parametrize("fmt", FMTS)
def test_quantise_errors(fmt):
    x = np.zeros(256, np.float32)
    x[5] = np.nan
    with pytest.raises(lw.LwError) as e:
        lw.quantize(fmt, x)
    assert e.value.code == lw.ERR_NONFINITE
    with pytest.raises(lw.LwError) as e:
        lw.quantize(fmt, np.zeros(40, np.float32))
    assert e.value.code == lw.ERR_SHAPE
    L = lw.lib()
    assert L.lw_quantize(fmt, None, 256, None) == lw.ERR_NULL
    assert L.lw_quantize(11, x.ctypes.data, 256, x.ctypes.data) == lw.ERR_FORMAT
    big = np.full(256, 3e38, np.float32)          # finite input whose scale overflows fp16
    if fmt != lw.F16:
        with pytest.raises(lw.LwError) as e:
            lw.quantize(fmt, big)
        assert e.value.code == lw.ERR_NONFINITE
        with pytest.raises(oracle.OracleError):
            oracle.quantize(fmt, big)


def test_device_calls_validate_before_touching_cuda():
    L = lw.lib()
    a = 0x1000                                    # fake, 16-byte aligned, never dereferenced
    assert L.lw_matvec(lw.Q8_0, None, 4, 64, a, a, 1, None) == lw.ERR_NULL
    assert L.lw_matvec(lw.Q8_0, a, 4, 64, None, a, 1, None) == lw.ERR_NULL
    assert L.lw_matvec(lw.Q8_0, a, 4, 64, a, None, 1, None) == lw.ERR_NULL
    assert L.lw_matvec(42, a, 4, 64, a, a, 1, None) == lw.ERR_FORMAT
    assert L.lw_matvec(lw.Q8_0, a, 0, 64, a, a, 1, None) == lw.ERR_SHAPE
    assert L.lw_matvec(lw.Q8_0, a, 4, 48, a, a, 1, None) == lw.ERR_SHAPE
    assert L.lw_matvec(lw.Q4_K, a, 4, 128, a, a, 1, None) == lw.ERR_SHAPE
    assert L.lw_matvec(lw.Q8_0, a, 4, 64, a, a, 0, None) == lw.ERR_BATCH
    assert L.lw_matvec(lw.Q8_0, a, 4, 64, a, a, 17, None) == lw.ERR_BATCH
    assert L.lw_matvec(lw.Q8_0, a + 2, 4, 64, a, a, 1, None) == lw.ERR_ALIGN
    assert L.lw_matvec(lw.Q8_0, a, 4, 64, a + 4, a, 1, None) == lw.ERR_ALIGN
    assert L.lw_matvec(lw.Q8_0, a, 4, 64, a, a + 8, 1, None) == lw.ERR_ALIGN
    assert L.lw_dequant(lw.Q4_0, None, 64, a, None) == lw.ERR_NULL
    assert L.lw_dequant(lw.Q4_0, a, 40, a, None) == lw.ERR_SHAPE
    assert L.lw_dequant(lw.Q4_0, a + 1, 64, a, None) == lw.ERR_ALIGN
    assert L.lw_dequant(17, a, 64, a, None) == lw.ERR_FORMAT
    item = lw.GroupItem(a, 4, a, a)
    import ctypes as _ct
    assert L.lw_matvec_group(lw.Q8_0, 64, 0, _ct.byref(item), None) == lw.ERR_SHAPE
    assert L.lw_matvec_group(lw.Q8_0, 48, 1, _ct.byref(item), None) == lw.ERR_SHAPE
    assert L.lw_matvec_group(77, 64, 1, _ct.byref(item), None) == lw.ERR_FORMAT
    assert L.lw_matvec_group(lw.Q8_0, 64, 1, None, None) == lw.ERR_NULL
    bad = lw.GroupItem(a + 4, 4, a, a)
    assert L.lw_matvec_group(lw.Q8_0, 64, 1, _ct.byref(bad), None) == lw.ERR_ALIGN
    assert L.lw_matvec_host(lw.Q8_0, a, 4, 64, None, a, a, a, 1, None) == lw.ERR_NULL
    assert L.lw_matvec_host(lw.Q8_0, a, 4, 64, a, a, a, a + 4, 1, None) == lw.ERR_ALIGN


def test_variant_controls():
    assert lw.lib().lw_set_variant(9) == lw.ERR_FORMAT
    lw.set_variant(lw.VARIANT_GENERIC)
    assert lw.query_variant(lw.Q4_K, 4096, 4096, 1) == lw.VARIANT_GENERIC
    lw.set_variant(lw.VARIANT_AUTO)
    assert lw.query_variant(lw.Q4_K, 4096, 4096, 1) == lw.VARIANT_IDOT
    assert lw.query_variant(lw.F16, 4096, 4096, 1) == lw.VARIANT_STREAM
    assert lw.query_variant(lw.Q4_K, 4096, 4096, 2) == lw.VARIANT_IDOT       # one integer-dot pass per column
    assert lw.query_variant(lw.Q4_0, 4096, 4096, 16) == lw.VARIANT_MMA       # tensor-core kernel: q8_0 / q4_0 / q4_K, cols % 256 == 0
    assert lw.query_variant(lw.Q8_0, 128256, 4096, 3) == lw.VARIANT_MMA
    assert lw.query_variant(lw.Q8_0, 128256, 4096, 2) == lw.VARIANT_IDOT        # two columns: one pass per column
    assert lw.query_variant(lw.Q4_0, 4096, 4096 + 512, 16) == lw.VARIANT_MMA
    assert lw.query_variant(lw.Q4_0, 4096, 4096 + 128, 16) == lw.VARIANT_GENERIC  # cols % 256 != 0: no streaming kernel
    lw.set_variant(lw.VARIANT_TILE)
    assert lw.query_variant(lw.Q4_0, 4096, 4096, 16) == lw.VARIANT_TILE      # fp32 tile kernel on request, cols % 1024 == 0
    assert lw.query_variant(lw.Q4_0, 4096, 4096 + 512, 16) != lw.VARIANT_TILE
    lw.set_variant(lw.VARIANT_MMA)
    assert lw.query_variant(lw.Q4_0, 4096, 4096, 2) == lw.VARIANT_MMA
    assert lw.query_variant(lw.Q4_K, 4096, 4096, 8) == lw.VARIANT_MMA         # q4_K as well (with the extra term E)
    assert lw.query_variant(lw.Q5_K, 4096, 4096, 8) == lw.VARIANT_MMA
    assert lw.query_variant(lw.F16, 4096, 4096, 8) == lw.VARIANT_MMA
    assert lw.query_variant(lw.Q6_K, 4096, 4096, 8) == lw.VARIANT_MMA         # q6_K: cols a multiple of 2048
    assert lw.query_variant(lw.Q6_K, 4096, 4096 + 1024, 8) != lw.VARIANT_MMA
    assert lw.query_variant(lw.Q4_0, 4096, 4096, 1) == lw.VARIANT_IDOT        # batch 1: falls back
    lw.set_variant(lw.VARIANT_AUTO)
    assert lw.query_variant(lw.Q4_1, 4096, 4096, 16) == lw.VARIANT_MMA
    assert lw.query_variant(lw.Q2_K, 4096, 4096, 16) == lw.VARIANT_MMA       # q2_K: cols a multiple of 1024
    assert lw.query_variant(lw.Q2_K, 4096, 4096 + 512, 16) == lw.VARIANT_GENERIC   # rows not whole 16-byte pieces
    assert lw.query_variant(lw.Q8_0, 16, 96, 3) == lw.VARIANT_GENERIC       # cols % 256 != 0: tiled fp32 kernel
    assert lw.query_variant(lw.Q6_K, 4096, 4096, 1) == lw.VARIANT_IDOT
    assert lw.query_variant(lw.Q5_K, 4096, 4096, 1) == lw.VARIANT_IDOT
    assert lw.query_variant(lw.Q2_K, 4096, 4096, 1) == lw.VARIANT_IDOT
    assert lw.query_variant(lw.Q2_K, 64, 512, 1) == lw.VARIANT_GENERIC      # 168-byte rows: not whole 16-byte pieces
    for f in (lw.Q4_1, lw.Q5_0, lw.Q5_1):
        assert lw.query_variant(f, 4096, 4096, 1) == lw.VARIANT_IDOT
        assert lw.query_variant(f, 16, 96, 1) == lw.VARIANT_GENERIC
    assert lw.query_variant(lw.Q6_K, 64, 1024, 1) == lw.VARIANT_GENERIC     # q6_K rows must be whole 16-byte pieces
    assert lw.query_variant(lw.F16, 4096, 4096, 2) == lw.VARIANT_STREAM      # f16, up to 4 columns: one pass per column
    assert lw.query_variant(lw.F16, 4096, 4096, 8) == lw.VARIANT_MMA         # f16 from three columns: tensor-core kernel
    assert lw.query_variant(lw.F16, 4096, 4096 + 128, 8) == lw.VARIANT_GENERIC  # cols % 256 != 0: tiled fp32 kernel
    assert lw.query_variant(lw.Q8_0, 64, 32768, 1) == lw.VARIANT_GENERIC     # too wide for one CTA
    lw.set_variant(lw.VARIANT_STREAM)
    assert lw.query_variant(lw.Q4_0, 4096, 4096, 1) == lw.VARIANT_STREAM
    for f in (lw.Q6_K, lw.Q5_K, lw.Q2_K, lw.Q4_1, lw.Q5_0, lw.Q5_1):      # no fp32-activation streaming form
        assert lw.query_variant(f, 4096, 4096, 1) == lw.VARIANT_GENERIC
    lw.set_variant(lw.VARIANT_AUTO)
    assert lw.query_variant(lw.Q4_0, 16, 96, 1) == lw.VARIANT_GENERIC      # cols % 256 != 0
    with pytest.raises(lw.LwError):
        lw.query_variant(lw.Q4_K, 16, 96, 1)
    assert "batch" in lw.status_string(lw.ERR_BATCH)
    lw.set_overlap(False)


def test_tuning_controls_and_plan_info():
    L = lw.lib()
    assert L.lw_set_tuning(3, 0, 0) == lw.ERR_FORMAT and L.lw_set_tuning(0, 5, 0) == lw.ERR_FORMAT
    assert L.lw_set_tuning(0, 0, 200) == lw.ERR_FORMAT and L.lw_set_tuning(-1, 0, 0) == lw.ERR_FORMAT
    try:
        lw.set_tuning()
        auto = lw.plan_info(lw.Q4_K, 4096, 4096)
        assert auto["worker_groups"] == 2 and auto["stages"] == 2 and auto["ctas"] <= 148
        assert auto["stage_bytes"] == auto["stage_rows"] * lw.row_bytes(lw.Q4_K, 4096)
        lw.set_tuning(1, 0, 0)
        one = lw.plan_info(lw.Q4_K, 4096, 4096)
        assert one["worker_groups"] == 1 and one["ctas"] > 148 and one["smem_bytes"] < auto["smem_bytes"]
        lw.set_tuning(2, 2, 24)
        small = lw.plan_info(lw.Q4_K, 4096, 4096)
        assert small["stage_bytes"] <= 24 * 1024 < auto["stage_bytes"]
    finally:
        lw.set_tuning()
    assert lw.plan_info(lw.Q8_0, 64, 96) == dict.fromkeys(auto, 0)          # generic kernels: nothing to plan
    assert L.lw_plan_info(lw.Q8_0, 64, 96, None) == lw.ERR_NULL
    assert L.lw_plan_info(77, 64, 96, None) == lw.ERR_FORMAT



def test_per_shape_tuning_table(tmp_path):
    L = lw.lib()
    try:
        lw.set_tuning()
        lw.clear_shape_tuning()
        auto = lw.plan_info(lw.Q4_K, 512, 2048)
        other = lw.plan_info(lw.Q4_K, 4096, 4096)
        lw.set_shape_tuning(lw.Q4_K, 512, 2048, 1, 2, 45)
        tuned = lw.plan_info(lw.Q4_K, 512, 2048)
        assert tuned["worker_groups"] == 1 and tuned != auto
        assert lw.plan_info(lw.Q4_K, 4096, 4096) == other                   # other shapes keep the heuristics
        assert lw.plan_info(lw.Q4_0, 512, 2048)["worker_groups"] == 2       # and so do other formats
        lw.set_tuning(2, 0, 0)                                              # an explicit process-wide value wins
        assert lw.plan_info(lw.Q4_K, 512, 2048)["worker_groups"] == 2
        lw.set_tuning()
        lw.set_shape_tuning(lw.Q4_K, 512, 2048)                             # all zero: entry removed
        assert lw.plan_info(lw.Q4_K, 512, 2048) == auto
        # the table file the sweep writes
        path = tmp_path / "table.json"
        path.write_text('[{"format": "q8_0", "rows": 512, "cols": 2048, "worker_groups": 1, "stages": 2, "stage_kb": 34, '
                        '"us_heuristics": 3.0, "us_tuned": 2.8}]')
        assert lw.load_tuning_table(str(path)) == 1
        assert lw.plan_info(lw.Q8_0, 512, 2048)["worker_groups"] == 1
        lw.clear_shape_tuning()
        assert lw.plan_info(lw.Q8_0, 512, 2048)["worker_groups"] == 2
        assert L.lw_set_shape_tuning(77, 4, 64, 0, 0, 0) == lw.ERR_FORMAT
        assert L.lw_set_shape_tuning(lw.Q8_0, 4, 48, 0, 0, 0) == lw.ERR_SHAPE
        assert L.lw_set_shape_tuning(lw.Q8_0, 4, 64, 3, 0, 0) == lw.ERR_FORMAT
    finally:
        lw.set_tuning()
        lw.clear_shape_tuning()


def test_attn_host_side_checks():
    L = lw.lib()
    assert lw.attn_workspace_bytes(32, 8, 128, 8192) == 32 * 256 * 130 * 4
    assert lw.attn_workspace_bytes(32, 8, 128, 1) == lw.attn_workspace_bytes(32, 8, 128, 1 << 20)
    for bad in ((32, 7, 128, 10), (32, 8, 96, 10), (32, 8, 128, 0), (0, 1, 128, 10), (2048, 1, 128, 10)):
        assert lw.attn_workspace_bytes(*bad) == 0
    a = 1 << 20                                            # any 16-byte aligned, non-null address: nothing is enqueued
    assert L.lw_attn_decode(lw.Q4_K, a, a, a, a, 32, 8, 128, 10, 1.0, a, 1 << 30, None) == lw.ERR_FORMAT
    assert L.lw_attn_decode(lw.Q8_0, a, a, a, a, 32, 5, 128, 10, 1.0, a, 1 << 30, None) == lw.ERR_SHAPE
    assert L.lw_attn_decode(lw.Q8_0, a, a, a, a, 32, 8, 128, 10, float("inf"), a, 1 << 30, None) == lw.ERR_SHAPE
    assert L.lw_attn_decode(lw.Q8_0, a, None, a, a, 32, 8, 128, 10, 1.0, a, 1 << 30, None) == lw.ERR_NULL
    assert L.lw_attn_decode(lw.Q8_0, a, a, a + 8, a, 32, 8, 128, 10, 1.0, a, 1 << 30, None) == lw.ERR_ALIGN
    assert L.lw_attn_decode(lw.Q8_0, a, a, a, a, 32, 8, 128, 10, 1.0, a, 100, None) == lw.ERR_WORKSPACE
    assert "workspace" in lw.status_string(lw.ERR_WORKSPACE)
    assert L.lw_set_attn_variant(2) == lw.ERR_FORMAT and L.lw_set_attn_variant(-1) == lw.ERR_FORMAT
    assert L.lw_set_attn_variant(1) == lw.OK and L.lw_set_attn_variant(0) == lw.OK
    assert L.lw_query_attn_variant(lw.Q4_K, 32, 8, 128, 10) == lw.ERR_FORMAT
    assert L.lw_query_attn_variant(lw.Q8_0, 32, 5, 128, 10) == lw.ERR_SHAPE
