"""GPU parity of lw_matvec against the fp64 oracle, element by element, for every format, kernel
variant and batch size; sizes span several tiles and ragged tails."""
import numpy as np
import pytest

import oracle
from paper_2605_20706_b200 import lw, synth

from gpu_util import Guarded, check_matvec, quantized_weights

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

FMTS = [lw.F16, lw.Q8_0, lw.Q4_0, lw.Q4_K, lw.Q6_K, lw.Q5_K, lw.Q2_K, lw.Q4_1, lw.Q5_0, lw.Q5_1]
VARIANTS = [lw.VARIANT_GENERIC, lw.VARIANT_STREAM, lw.VARIANT_IDOT]


@pytest.fixture(autouse=True)
def _reset_variant():
    yield
    lw.set_variant(lw.VARIANT_AUTO)
    lw.set_overlap(False)


def gpu_matvec(fmt, blocks, rows, cols, X, batch=1, variant=lw.VARIANT_AUTO, overlap=False, repeat=1):
    lw.set_variant(variant)
    lw.set_overlap(overlap)
    w = torch.from_numpy(np.ascontiguousarray(blocks)).cuda()
    x = torch.from_numpy(np.ascontiguousarray(X, dtype=np.float32)).cuda()
    y = Guarded((batch, rows))                  # NaN-filled, guard words on both sides
    for _ in range(repeat):
        lw.matvec(fmt, w, rows, cols, x, y.t, batch)
    torch.cuda.synchronize()
    assert lw.device_status() == 0
    y.check("Y of fmt %d %dx%d batch %d" % (fmt, rows, cols, batch))
    return y.t.cpu().numpy()


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("rows,cols", [(1, 256), (3, 512), (37, 2048), (301, 4096), (150, 14336),
                                       (1024, 4096), (513, 8192), (29, 768)])
def test_matvec_batch1(variant, fmt, rows, cols):
    blocks = quantized_weights(fmt, rows, cols, seed=50, tensor_id=fmt, outlier_p=0.01)
    X = synth.activations(50, rows, 1, cols)
    y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, 1, nthreads=4)
    y = gpu_matvec(fmt, blocks, rows, cols, X, 1, variant)
    check_matvec(y, y_ref, s_ref, "fmt %d %dx%d" % (fmt, rows, cols))


@pytest.mark.parametrize("variant", VARIANTS + [lw.VARIANT_AUTO])
@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("batch", [2, 3, 4, 7, 8, 9, 16])
def test_matvec_batched(variant, fmt, batch):
    # GENERIC: tiled fp32 kernel; IDOT (forced): batched integer-dot kernel in passes of up to 4 columns;
    # AUTO: one pass of the batch-1 integer-dot kernel per column, up to eight columns per launch
    rows, cols = 203, 2048
    blocks = quantized_weights(fmt, rows, cols, seed=51, tensor_id=fmt)
    X = synth.activations(51, batch, batch, cols)
    y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, batch, nthreads=4)
    y = gpu_matvec(fmt, blocks, rows, cols, X, batch, variant)
    check_matvec(y, y_ref, s_ref, "fmt %d batch %d" % (fmt, batch))


@pytest.mark.parametrize("fmt", [lw.Q8_0, lw.Q4_0])
@pytest.mark.parametrize("batch", [2, 3, 4, 5, 8, 9, 13, 16])
@pytest.mark.parametrize("rows,cols", [(1, 1024), (63, 2048), (64, 1024), (65, 4096), (333, 3072), (1000, 14336),
                                       (70000, 1024)])
def test_matvec_tile_kernel(fmt, batch, rows, cols):
    # the batched fp32 tile kernel (on request; q8_0 / q4_0 when cols is a multiple of 1024): ragged row
    # counts around its 64-row stages, one to fourteen column chunks, passes of 4 and 8 columns, several CTAs
    # per SM (70000 rows)
    lw.set_variant(lw.VARIANT_TILE)
    assert lw.query_variant(fmt, rows, cols, batch) == lw.VARIANT_TILE
    blocks = quantized_weights(fmt, rows, cols, seed=59, tensor_id=fmt, outlier_p=0.01)
    X = synth.activations(59, batch, batch, cols)
    y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, batch, nthreads=8)
    y = gpu_matvec(fmt, blocks, rows, cols, X, batch, lw.VARIANT_TILE)
    check_matvec(y, y_ref, s_ref, "tile fmt %d %dx%d batch %d" % (fmt, rows, cols, batch))


@pytest.mark.parametrize("fmt", [lw.Q8_0, lw.Q4_0, lw.Q4_K, lw.Q5_K, lw.F16, lw.Q4_1, lw.Q5_0, lw.Q5_1])
@pytest.mark.parametrize("batch", [2, 3, 7, 8, 9, 16])
@pytest.mark.parametrize("rows,cols", [(1, 256), (15, 512), (16, 1024), (17, 768), (255, 2048), (256, 1024), (257, 4096),
                                       (333, 3072), (1000, 14336), (4096, 1280), (70000, 1024)])
def test_matvec_mma_kernel(fmt, batch, rows, cols):
    # the batched tensor-core kernel (AUTO's choice for every format (q6_K and q2_K: their own test) from three columns on when cols is a
    # multiple of 256): ragged row counts around its 16-row fragments and 256-row stages, chunks of 256 / 512 / 1024 columns,
    # one and two groups of eight columns, more stages than CTAs (70000 rows) and fewer (1 row)
    lw.set_variant(lw.VARIANT_AUTO)
    column_wise = lw.VARIANT_STREAM if fmt == lw.F16 else lw.VARIANT_IDOT
    assert lw.query_variant(fmt, rows, cols, batch) == (lw.VARIANT_MMA if batch >= 3 else column_wise)
    blocks = quantized_weights(fmt, rows, cols, seed=61, tensor_id=fmt, outlier_p=0.01)
    X = synth.activations(61, batch, batch, cols)
    y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, batch, nthreads=8)
    y = gpu_matvec(fmt, blocks, rows, cols, X, batch, lw.VARIANT_MMA)
    check_matvec(y, y_ref, s_ref, "mma fmt %d %dx%d batch %d" % (fmt, rows, cols, batch))
    y = gpu_matvec(fmt, blocks, rows, cols, X, batch, lw.VARIANT_AUTO)
    check_matvec(y, y_ref, s_ref, "auto fmt %d %dx%d batch %d" % (fmt, rows, cols, batch))


@pytest.mark.parametrize("batch", [3, 8, 13, 16])
@pytest.mark.parametrize("fmt,rows,cols", [(lw.Q6_K, 1, 2048), (lw.Q6_K, 17, 2048), (lw.Q6_K, 255, 4096), (lw.Q6_K, 300, 6144),
                                           (lw.Q6_K, 513, 14336), (lw.Q6_K, 4096, 2048), (lw.Q2_K, 1, 1024),
                                           (lw.Q2_K, 17, 3072), (lw.Q2_K, 255, 4096), (lw.Q2_K, 513, 14336),
                                           (lw.Q2_K, 4096, 2048)])
def test_matvec_mma_kernel_offset_fetch(fmt, batch, rows, cols):
    # q6_K and q2_K on the tensor cores: 210- and 84-byte super-blocks, so a stage's row pieces start on a 2-byte
    # (4-byte) grid inside the 16-byte-aligned fetch; all remainders occur from 16 (4) column stages on, q6_K's odd
    # ones with straddled words; cols must be a multiple of 2048 (1024)
    lw.set_variant(lw.VARIANT_AUTO)
    assert lw.query_variant(fmt, rows, cols, batch) == lw.VARIANT_MMA
    assert lw.query_variant(fmt, rows, cols + 256, batch) != lw.VARIANT_MMA
    blocks = quantized_weights(fmt, rows, cols, seed=66, tensor_id=fmt, outlier_p=0.01)
    X = synth.activations(66, batch, batch, cols)
    y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, batch, nthreads=8)
    y = gpu_matvec(fmt, blocks, rows, cols, X, batch, lw.VARIANT_AUTO)
    check_matvec(y, y_ref, s_ref, "mma fmt %d %dx%d batch %d" % (fmt, rows, cols, batch))
    # and two matrices in one launch
    w = torch.from_numpy(blocks).cuda()
    x = torch.from_numpy(X).cuda()
    ys = [Guarded((batch, rows)), Guarded((batch, rows))]
    lw.matvec_group(fmt, cols, [(w, rows, x, ys[0].t), (w, rows, x, ys[1].t)], batch=batch)
    torch.cuda.synchronize()
    for yg in ys:
        yg.check("grouped Y")
        check_matvec(yg.t.cpu().numpy(), y_ref, s_ref, "grouped mma fmt %d" % fmt)
    assert lw.device_status() == 0


@pytest.mark.parametrize("overlap", [0, 1, 2])
@pytest.mark.parametrize("fmt", [lw.Q8_0, lw.Q4_0, lw.Q4_K, lw.Q5_K, lw.F16, lw.Q4_1, lw.Q5_0, lw.Q5_1])
def test_matvec_mma_launch_modes(fmt, overlap):
    # the two ways the tensor-core kernel gets a cleared Y: one cooperative launch whose CTAs clear it and meet at a
    # grid barrier (no overlap), or a clearing kernel chained to it by programmatic dependent launch (overlap 1;
    # 2: weights requested before the previous kernel has completed).  A chain of calls into ping-pong buffers,
    # so a call's Y is the X the call before last read, replayed several times.
    batch, dims = 5, [1024, 768, 2048, 1024, 512]
    mats = [quantized_weights(fmt, dims[j + 1], dims[j], seed=63 + j, tensor_id=fmt) for j in range(len(dims) - 1)]
    wd = [torch.from_numpy(m).cuda() for m in mats]
    x0 = synth.activations(63, 0, batch, dims[0])
    bufs = [torch.zeros(batch * max(dims), dtype=torch.float32, device="cuda") for _ in range(2)]
    lw.set_variant(lw.VARIANT_MMA)
    lw.set_overlap(overlap)
    try:
        for _ in range(3):
            bufs[0][:x0.size] = torch.from_numpy(x0.reshape(-1)).cuda()
            for j in range(len(mats)):
                lw.matvec(fmt, wd[j], dims[j + 1], dims[j], bufs[j & 1], bufs[(j + 1) & 1], batch)
            torch.cuda.synchronize()
            assert lw.device_status() == 0
            got = bufs[len(mats) & 1][:batch * dims[-1]].cpu().numpy().reshape(batch, dims[-1])
            # the chain's rounding differences grow from layer to layer: compare the last layer against the oracle
            # fed with the GPU's own input to that layer
            x_in = bufs[(len(mats) - 1) & 1][:batch * dims[-2]].cpu().numpy().reshape(batch, dims[-2])
            y_ref, s_ref = oracle.matvec(fmt, mats[-1], dims[-1], dims[-2], x_in, batch, nthreads=4)
            check_matvec(got, y_ref, s_ref, "mma chain overlap %d" % overlap)
    finally:
        lw.set_overlap(0)
        lw.set_variant(lw.VARIANT_AUTO)


@pytest.mark.parametrize("variant", VARIANTS)
def test_config1_q8_0_2048(variant):
    # the single q8_0 mat-vec of the first benchmark configuration: every output checked
    rows = cols = 2048
    blocks = quantized_weights(lw.Q8_0, rows, cols, seed=1)
    X = synth.activations(1, 0, 1, cols)
    y_ref, s_ref = oracle.matvec(lw.Q8_0, blocks, rows, cols, X, 1, nthreads=8)
    y = gpu_matvec(lw.Q8_0, blocks, rows, cols, X, 1, variant)
    check_matvec(y, y_ref, s_ref, "config 1")


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("fmt", FMTS)
def test_unit_vectors_recover_dequantised_weights(variant, fmt):
    # x = e_k leaves one non-zero term, which pins the element / nibble order of the mat-vec kernels
    # independently of the dequant kernel.  The generic variant multiplies the exactly decoded weight
    # by 1.0, so it must return it exactly; the streaming variant applies block scales and offsets
    # after the dot product, so it is held to the mat-vec tolerance with S = |w|.
    rows, cols = 9, 512
    blocks = quantized_weights(fmt, rows, cols, seed=52, tensor_id=fmt, outlier_p=0.01)
    deq = oracle.dequant(fmt, blocks, rows * cols).reshape(rows, cols)
    ks = list(range(0, 256, 1))[:: 3] + [256, 300, 511]
    for k in ks:
        X = np.zeros((1, cols), np.float32)
        X[0, k] = 1.0
        y = gpu_matvec(fmt, blocks, rows, cols, X, 1, variant)
        if variant == lw.VARIANT_GENERIC:
            assert (y[0] == deq[:, k]).all(), (fmt, k)
        else:
            w = deq[:, k].astype(np.float64)
            assert (np.abs(y[0] - w) <= 1e-4 * np.abs(w) + 1e-6).all(), (fmt, k)


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("fmt", FMTS)
def test_sparse_and_scaled_activations(variant, fmt):
    # few non-zero activations of awkward magnitude: the tolerance has no sqrt(n) averaging to hide behind
    rows, cols = 64, 4096
    blocks = quantized_weights(fmt, rows, cols, seed=53, tensor_id=fmt)
    rng = np.random.default_rng(53)
    for scale in (1.0, 1e-3, 777.7):
        X = np.zeros((1, cols), np.float32)
        idx = rng.choice(cols, 5, replace=False)
        X[0, idx] = (rng.standard_normal(5) * scale + 0.1 * scale).astype(np.float32)
        y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, 1)
        y = gpu_matvec(fmt, blocks, rows, cols, X, 1, variant)
        check_matvec(y, y_ref, s_ref, "sparse x, scale %g" % scale)
    X = np.full((1, cols), 3.0, np.float32)      # all-positive activations: no cancellation in sum(x)
    y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, 1)
    check_matvec(gpu_matvec(fmt, blocks, rows, cols, X, 1, variant), y_ref, s_ref, "constant x")


@pytest.mark.parametrize("fmt", FMTS)
def test_overlap_mode_and_repeated_calls(fmt):
    rows, cols = 777, 4096
    blocks = quantized_weights(fmt, rows, cols, seed=54, tensor_id=fmt)
    X = synth.activations(54, 0, 1, cols)
    y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, 1, nthreads=4)
    y = gpu_matvec(fmt, blocks, rows, cols, X, 1, lw.VARIANT_AUTO, overlap=True, repeat=5)
    check_matvec(y, y_ref, s_ref, "overlap")


def test_matvec_host_entry_point():
    fmt, rows, cols, batch = lw.Q4_0, 129, 2048, 2
    blocks = quantized_weights(fmt, rows, cols, seed=55)
    X = synth.activations(55, 0, batch, cols)
    y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, batch)
    w = torch.from_numpy(blocks).cuda()
    xh = torch.from_numpy(X.copy()).pin_memory()
    yh = torch.empty((batch, rows), dtype=torch.float32).pin_memory()
    xd = torch.empty((batch, cols), dtype=torch.float32, device="cuda")
    yd = Guarded((batch, rows))
    lw.matvec_host(fmt, w, rows, cols, xh.data_ptr(), yh.data_ptr(), xd, yd.t, batch)
    torch.cuda.synchronize()
    yd.check("Y_dev of the host entry point")
    check_matvec(yh.numpy(), y_ref, s_ref, "host entry point")


def test_matvec_in_cuda_graph():
    fmt, rows, cols = lw.Q4_K, 512, 4096
    blocks = quantized_weights(fmt, rows, cols, seed=56)
    X = synth.activations(56, 0, 1, cols)
    y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, 1, nthreads=4)
    w = torch.from_numpy(blocks).cuda()
    x = torch.from_numpy(X).cuda()
    y = torch.zeros((1, rows), dtype=torch.float32, device="cuda")
    lw.set_overlap(True)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        lw.matvec(fmt, w, rows, cols, x, y, 1)          # warm-up outside capture
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for _ in range(3):
            lw.matvec(fmt, w, rows, cols, x, y, 1)
    y.zero_()
    graph.replay()
    torch.cuda.synchronize()
    check_matvec(y.cpu().numpy(), y_ref, s_ref, "graph replay")
    assert lw.device_status() == 0


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("rows,cols,batch", [(5, 96, 1), (5, 96, 3), (1, 32, 1), (7, 16384, 1), (3, 32768, 1),
                                             (2, 20480, 2), (300, 6400, 1), (300, 6400, 5)])
def test_edge_shapes_and_fallbacks(fmt, rows, cols, batch):
    # cols not a multiple of 256 (generic kernel), the widest row the streaming kernel takes, rows
    # wider than that (fallback), cols not a multiple of the batched kernel's tile, tiny matrices
    if fmt in (lw.Q4_K, lw.Q6_K, lw.Q5_K, lw.Q2_K) and cols % 256:
        with pytest.raises(lw.LwError) as e:
            lw.query_variant(fmt, rows, cols, batch)
        assert e.value.code == lw.ERR_SHAPE
        return
    blocks = quantized_weights(fmt, rows, cols, seed=57, tensor_id=fmt)
    X = synth.activations(57, cols % 1000, batch, cols)
    y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, X, batch)
    y = gpu_matvec(fmt, blocks, rows, cols, X, batch, lw.VARIANT_AUTO)
    check_matvec(y, y_ref, s_ref, "edge %dx%d batch %d" % (rows, cols, batch))


def test_zero_activations_and_zero_weights():
    for fmt in FMTS:
        rows, cols = 33, 1024
        blocks = quantized_weights(fmt, rows, cols, seed=58, tensor_id=fmt)
        X = np.zeros((1, cols), np.float32)
        y = gpu_matvec(fmt, blocks, rows, cols, X, 1)
        assert (y == 0).all()
        zero_w = oracle.quantize(fmt, np.zeros((rows, cols), np.float32))
        X = synth.activations(58, 1, 1, cols)
        y = gpu_matvec(fmt, zero_w, rows, cols, X, 1)
        assert (y == 0).all()


@pytest.mark.parametrize("variant", [lw.VARIANT_AUTO, lw.VARIANT_STREAM, lw.VARIANT_GENERIC])
@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("cols,row_list", [(4096, [4096, 1024, 1024]), (2048, [8192, 8192]), (4096, [37]),
                                           (1024, [5, 1, 300, 64, 7, 129, 2, 33]), (96, [10, 3])])
def test_matvec_group(variant, fmt, cols, row_list):
    # several independent matrices in one call; items share or do not share their activations
    if fmt in (lw.Q4_K, lw.Q6_K, lw.Q5_K, lw.Q2_K) and cols % 256:
        return
    lw.set_variant(variant)
    lw.set_overlap(True)
    items, refs, keep = [], [], []
    for j, rows in enumerate(row_list):
        blocks = quantized_weights(fmt, rows, cols, seed=60 + j, tensor_id=fmt)
        X = synth.activations(60, j % 2, 1, cols)            # alternate between two activation vectors
        w = torch.from_numpy(blocks).cuda()
        x = torch.from_numpy(X).cuda()
        y = Guarded((1, rows))
        keep.append((w, x, y))
        items.append((w, rows, x, y.t))
        refs.append(oracle.matvec(fmt, blocks, rows, cols, X, 1, nthreads=4))
    for _ in range(2):
        lw.matvec_group(fmt, cols, items)
    torch.cuda.synchronize()
    assert lw.device_status() == 0
    for (w, x, y), (y_ref, s_ref) in zip(keep, refs):
        y.check("group item")
        check_matvec(y.t.cpu().numpy(), y_ref, s_ref, "group item")


@pytest.mark.parametrize("overlap", [0, 2])
@pytest.mark.parametrize("batch", [2, 5, 12])
@pytest.mark.parametrize("fmt", [lw.Q8_0, lw.Q4_0, lw.Q4_K, lw.Q5_K, lw.F16, lw.Q4_1, lw.Q5_0, lw.Q5_1])
@pytest.mark.parametrize("cols,row_list,share", [(1024, [300, 77, 1000], True), (2048, [513, 256], True),
                                                 (768, [40, 1, 255, 17, 256, 3, 700, 64], False), (4096, [37], True)])
def test_matvec_group_batch(fmt, batch, overlap, cols, row_list, share):
    # several matrices and several columns in one call: q8_0 / q4_0 go through one launch of the tensor-core kernel
    # (shared or separate activations, ragged row counts around its 256-row stages, both launch modes), q4_K item by
    # item through lw_matvec
    lw.set_variant(lw.VARIANT_AUTO)
    lw.set_overlap(overlap)
    try:
        x_shared = torch.from_numpy(synth.activations(64, 99, batch, cols)).cuda()
        items, refs, keep = [], [], []
        for j, rows in enumerate(row_list):
            blocks = quantized_weights(fmt, rows, cols, seed=64 + j, tensor_id=fmt)
            X = synth.activations(64, 99 if share else j, batch, cols)
            w = torch.from_numpy(blocks).cuda()
            x = x_shared if share else torch.from_numpy(X).cuda()
            y = Guarded((batch, rows))
            keep.append((w, x, y))
            items.append((w, rows, x, y.t))
            refs.append(oracle.matvec(fmt, blocks, rows, cols, X, batch, nthreads=4))
        for _ in range(2):
            lw.matvec_group(fmt, cols, items, batch=batch)
        torch.cuda.synchronize()
        assert lw.device_status() == 0
        for (w, x, y), (y_ref, s_ref) in zip(keep, refs):
            y.check("group item")
            check_matvec(y.t.cpu().numpy(), y_ref, s_ref, "batched group item")
    finally:
        lw.set_overlap(0)


def test_matvec_group_argument_errors():
    L = lw.lib()
    w = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    x = torch.zeros(64, dtype=torch.float32, device="cuda")
    y = torch.zeros(8, dtype=torch.float32, device="cuda")
    with pytest.raises(lw.LwError) as e:
        lw.matvec_group(lw.Q8_0, 64, [(w, 4, x, y)] * 9)
    assert e.value.code == lw.ERR_SHAPE
    with pytest.raises(lw.LwError) as e:
        lw.matvec_group(lw.Q8_0, 64, [(w, 4, x, y), (w, 0, x, y)])
    assert e.value.code == lw.ERR_SHAPE
    with pytest.raises(lw.LwError) as e:
        lw.matvec_group(lw.Q8_0, 64, [(w, 4, None, y)])
    assert e.value.code == lw.ERR_NULL
    assert L.lw_matvec_group(lw.Q8_0, 64, 1, None, None) == lw.ERR_NULL
    with pytest.raises(lw.LwError) as e:
        lw.matvec_group(lw.Q8_0, 64, [(w, 4, x, y)], batch=17)
    assert e.value.code == lw.ERR_BATCH
    with pytest.raises(lw.LwError) as e:
        lw.matvec_group(lw.Q8_0, 64, [(w, 4, x, y)] * 9, batch=4)
    assert e.value.code == lw.ERR_SHAPE
    assert L.lw_matvec_group_batch(lw.Q8_0, 64, 1, None, 4, None) == lw.ERR_NULL
