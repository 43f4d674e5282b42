"""GPU parity at the benchmark's full matrix sizes, in the launch configuration bench.py times
(automatic variant, programmatic overlap on, CUDA-graph replay of consecutive calls): every distinct
matrix shape of the Llama-3.1-8B- and Llama-3.2-1B-shaped decode steps, checked against the fp64
oracle on sampled rows (first, last, ragged ends of CTA row ranges, and random ones)."""
import numpy as np
import pytest

import oracle
from paper_2605_20706_b200 import lw, synth

from gpu_util import Guarded, check_matvec, quantized_weights

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

SHAPES_8B = [("q", 4096, 4096), ("k", 1024, 4096), ("gate", 14336, 4096), ("down", 4096, 14336),
             ("lm_head", 128256, 4096)]
SHAPES_1B = [("q", 2048, 2048), ("k", 512, 2048), ("gate", 8192, 2048), ("down", 2048, 8192),
             ("lm_head", 128256, 2048)]


def _sample_rows(rows, rng, n=1500):
    fixed = [0, 1, 2, 3, rows - 1, rows - 2, rows // 2, rows // 3]
    for step in (4, 16, 48, 52, 100, 436, 868):          # around likely CTA / stage boundaries
        fixed += [r for r in (step - 1, step, step + 1, rows - step, rows - step - 1) if 0 <= r < rows]
    rnd = rng.choice(rows, size=min(n, rows), replace=False).tolist()
    return np.unique(np.array(fixed + rnd, dtype=np.int64))


def _run_case(fmt, rows, cols, seed, outlier_p):
    blocks = quantized_weights(fmt, rows, cols, seed=seed, tensor_id=rows % 97, outlier_p=outlier_p)
    X = synth.activations(seed, rows % 89, 1, cols)
    w = torch.from_numpy(blocks).cuda()
    x = torch.from_numpy(X).cuda()
    guarded = Guarded((1, rows))
    y = guarded.t
    lw.set_variant(lw.VARIANT_AUTO)
    lw.set_overlap(True)
    try:
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            lw.matvec(fmt, w, rows, cols, x, y, 1)
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for _ in range(3):
                lw.matvec(fmt, w, rows, cols, x, y, 1)
        y.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
    finally:
        lw.set_overlap(False)
    assert lw.device_status() == 0
    guarded.check("Y of fmt %d %dx%d" % (fmt, rows, cols))
    got = y.cpu().numpy()
    assert np.isfinite(got).all()
    idx = _sample_rows(rows, np.random.default_rng(seed))
    y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, 1, nthreads=8, row_idx=idx)
    check_matvec(got[:, idx], y_ref, s_ref, "fmt %d %dx%d" % (fmt, rows, cols))


@pytest.mark.parametrize("name,rows,cols", SHAPES_8B)
@pytest.mark.parametrize("fmt", [lw.Q4_K, lw.Q8_0, lw.Q4_0, lw.Q6_K, lw.Q5_K, lw.Q2_K, lw.Q4_1, lw.Q5_0,
                                 lw.Q5_1])
def test_llama8b_shapes(fmt, name, rows, cols):
    _run_case(fmt, rows, cols, seed=4 if fmt == lw.Q4_K else 5, outlier_p=0.01 if fmt == lw.Q4_K else 0.0)


@pytest.mark.parametrize("name,rows,cols", SHAPES_1B)
@pytest.mark.parametrize("fmt", [lw.F16, lw.Q4_0])
def test_llama1b_shapes(fmt, name, rows, cols):
    _run_case(fmt, rows, cols, seed=2 if fmt == lw.F16 else 3, outlier_p=0.0)


@pytest.mark.parametrize("batch", [2, 16])
def test_llama8b_gate_batched(batch):
    fmt, rows, cols = lw.Q4_0, 14336, 4096
    blocks = quantized_weights(fmt, rows, cols, seed=5, tensor_id=7)
    X = synth.activations(5, 7, batch, cols)
    w = torch.from_numpy(blocks).cuda()
    x = torch.from_numpy(X).cuda()
    guarded = Guarded((batch, rows))
    y = guarded.t
    lw.matvec(fmt, w, rows, cols, x, y, batch)
    torch.cuda.synchronize()
    guarded.check("Y of the batched gate")
    idx = _sample_rows(rows, np.random.default_rng(batch), n=400)
    y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, batch, nthreads=8, row_idx=idx)
    check_matvec(y.cpu().numpy()[:, idx], y_ref, s_ref, "batched gate, batch %d" % batch)


LAYER_8B = [("q", 4096, 4096, 0), ("k", 1024, 4096, 0), ("v", 1024, 4096, 0), ("o", 4096, 4096, 1),
            ("gate", 14336, 4096, 2), ("up", 14336, 4096, 2), ("down", 4096, 14336, 3), ("lm_head", 128256, 4096, 4)]
LAYER_1B = [("q", 2048, 2048, 0), ("k", 512, 2048, 0), ("v", 512, 2048, 0), ("o", 2048, 2048, 1),
            ("gate", 8192, 2048, 2), ("up", 8192, 2048, 2), ("down", 2048, 8192, 3), ("lm_head", 128256, 2048, 4)]


@pytest.mark.parametrize("fmt,batch,layer", [(lw.Q4_0, 8, LAYER_8B), (lw.Q4_0, 16, LAYER_8B), (lw.Q8_0, 16, LAYER_8B),
                                             (lw.Q4_K, 8, LAYER_8B), (lw.Q6_K, 16, LAYER_8B), (lw.Q2_K, 5, LAYER_8B),
                                             (lw.F16, 8, LAYER_1B), (lw.F16, 16, LAYER_1B)])
def test_layer_and_lm_head_batched_chain(fmt, batch, layer):
    # the batched step as bench.py issues it: one lw_matvec_sequence_batch call over a layer's mat-vecs and lm_head
    # at their full sizes (q/k/v and gate/up share their activations), weights requested ahead of the dependency
    # wait (overlap level 2), replayed as a CUDA graph; sampled rows of every matrix against the oracle
    xs, items, keep, cases = {}, [], [], []
    for j, (name, rows, cols, xid) in enumerate(layer):
        if xid not in xs:
            X = synth.activations(40 + batch, xid, batch, cols)
            xs[xid] = (X, torch.from_numpy(X).cuda())
        X, xd = xs[xid]
        blocks = quantized_weights(fmt, rows, cols, seed=60 + j, tensor_id=fmt)
        w = torch.from_numpy(blocks).cuda()
        y = Guarded((batch, rows))
        flags = 0 if j and layer[j - 1][3] == xid else lw.SEQ_DEPENDENT
        items.append((w, rows, cols, xd, y.t, flags))
        keep.append((w, y))
        idx = _sample_rows(rows, np.random.default_rng(j), n=300)
        cases.append((name, blocks, rows, cols, X, idx, y))
    lw.set_overlap(2)
    try:
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            lw.matvec_sequence_batch(fmt, items, batch, side)
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for _ in range(2):
                    lw.matvec_sequence_batch(fmt, items, batch, side)
            for _, y in keep:
                y.t.fill_(float("nan"))
            graph.replay()
        torch.cuda.synchronize()
    finally:
        lw.set_overlap(0)
    assert lw.device_status() == 0
    for name, blocks, rows, cols, X, idx, y in cases:
        y.check("Y of %s" % name)
        got = y.t.cpu().numpy()
        assert np.isfinite(got).all(), name
        y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, batch, nthreads=8, row_idx=idx)
        check_matvec(got[:, idx], y_ref, s_ref, "%s, fmt %d, batch %d" % (name, fmt, batch))
