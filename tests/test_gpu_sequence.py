"""GPU parity of lw_matvec_sequence (the persistent kernel that runs a whole chain of mat-vecs in one
launch) against the fp64 oracle: independent items, phases of several matrices that share their
activations, chains in which every item reads what the previous one wrote, repeated calls, CUDA-graph
replay, and the fall-back for shapes the streaming kernels do not take."""
import numpy as np
import pytest

import oracle
from paper_2605_20706_b200 import lw, synth

from gpu_util import Guarded, check_matvec, quantized_weights

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

MODES = [lw.SEQ_PERSISTENT, lw.SEQ_LAUNCHES]


@pytest.fixture(autouse=True)
def _reset_mode():
    yield
    lw.set_sequence_mode(lw.SEQ_AUTO)
    lw.set_variant(lw.VARIANT_AUTO)


FMTS = [lw.F16, lw.Q8_0, lw.Q4_0, lw.Q4_K, lw.Q6_K, lw.Q5_K, lw.Q2_K, lw.Q4_1, lw.Q5_0, lw.Q5_1]
DEP = lw.SEQ_DEPENDENT


def _workspace():
    ws = Guarded(lw.matvec_sequence_workspace_bytes() // 4, fill=None, dtype=torch.int32)
    return ws


def _layer_like(fmt, cols_a, cols_b, seed, scale_rows=1):
    """A decode-layer-shaped chain: (q, k, v) on x0 | o on x1 | (gate, up) on x2 | down on x3 | ragged extras."""
    r = scale_rows
    spec = [("q", 256 * r + 3, cols_a, 0, DEP), ("k", 64 * r + 1, cols_a, 0, 0), ("v", 64 * r, cols_a, 0, 0),
            ("o", 256 * r, cols_a, 1, DEP), ("gate", 520 * r + 5, cols_a, 2, DEP), ("up", 520 * r + 5, cols_a, 2, 0),
            ("down", 256 * r + 1, cols_b, 3, DEP), ("tiny", 1, cols_a, 4, DEP), ("small", 37, cols_b, 5, 0),
            ("tall", 3000 * r + 7, cols_a, 6, DEP)]
    xs = {}
    items, keep, refs = [], [], []
    for j, (name, rows, cols, xid, flags) in enumerate(spec):
        if xid not in xs:
            X = synth.activations(seed, xid, 1, cols)
            xs[xid] = (X, torch.from_numpy(X).cuda())
        X, xd = xs[xid]
        blocks = quantized_weights(fmt, rows, cols, seed=seed + j, tensor_id=fmt, outlier_p=0.01)
        w = torch.from_numpy(blocks).cuda()
        y = Guarded((1, rows))
        keep.append((w, xd, y))
        items.append((w, rows, cols, xd, y.t, flags))
        refs.append(oracle.matvec(fmt, blocks, rows, cols, X, 1, nthreads=4))
    return items, keep, refs


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("cols_a,cols_b", [(4096, 14336), (2048, 8192), (256, 512)])
def test_sequence_of_layer_shaped_items(fmt, cols_a, cols_b, mode):
    lw.set_sequence_mode(mode)
    if fmt == lw.Q6_K and (cols_a % 2048 or cols_b % 2048):
        cols_a, cols_b = 2048, 6144          # q6_K rows must be whole 16-byte pieces for the streaming kernels
    if fmt == lw.Q2_K and (cols_a % 1024 or cols_b % 1024):
        cols_a, cols_b = 1024, 3072
    items, keep, refs = _layer_like(fmt, cols_a, cols_b, seed=120)
    ws = _workspace()
    for _ in range(2):                        # the second call finds the first call's counter value
        lw.matvec_sequence(fmt, items, ws.t)
    torch.cuda.synchronize()
    assert lw.device_status() == 0
    ws.check("sequence workspace")
    for (w, x, y), (y_ref, s_ref) in zip(keep, refs):
        y.check("sequence item")
        check_matvec(y.t.cpu().numpy(), y_ref, s_ref, "sequence item")


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("fmt", [lw.Q4_K, lw.Q8_0, lw.F16, lw.Q4_0, lw.Q6_K])
def test_chain_where_every_item_reads_the_previous_result(fmt, mode):
    lw.set_sequence_mode(mode)
    # item i+1's X is item i's Y: the grid-wide barrier before a dependent item is what makes this right.
    # Each stage is checked against the oracle applied to the GPU's own previous stage (fp32), so errors
    # do not compound in the comparison.
    dims = [2048, 4096, 2048, 6144, 2048, 4096, 4096, 2048]       # x0 has dims[0] values; stage i maps dims[i] -> dims[i+1]
    X0 = synth.activations(130, 0, 1, dims[0])
    bufs = [torch.from_numpy(X0).cuda()] + [Guarded((1, d)) for d in dims[1:]]
    mats, items = [], []
    for i in range(len(dims) - 1):
        rows, cols = dims[i + 1], dims[i]
        blocks = quantized_weights(fmt, rows, cols, seed=131 + i, tensor_id=fmt, std=1.0 / np.sqrt(cols))
        w = torch.from_numpy(blocks).cuda()
        mats.append((blocks, w, rows, cols))
        x = bufs[i] if i == 0 else bufs[i].t
        items.append((w, rows, cols, x, bufs[i + 1].t, DEP))
    ws = _workspace()
    arr = lw.seq_items(items)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        lw.matvec_sequence(fmt, arr, ws.t, stream=side)          # first call outside capture
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        lw.matvec_sequence(fmt, arr, ws.t, stream=side)
    for b in bufs[1:]:
        b.t.fill_(float("nan"))
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    assert lw.device_status() == 0
    x_prev = X0
    for i, (blocks, w, rows, cols) in enumerate(mats):
        bufs[i + 1].check("stage %d" % i)
        got = bufs[i + 1].t.cpu().numpy()
        y_ref, s_ref = oracle.matvec(fmt, blocks, rows, cols, x_prev, 1, nthreads=8)
        check_matvec(got, y_ref, s_ref, "chain stage %d" % i)
        x_prev = got.astype(np.float32)


@pytest.mark.parametrize("mode", MODES)
def test_sequence_with_host_buffers(mode):
    # lw_matvec_sequence_host: the input block comes from pinned host memory in one copy, the result block
    # goes back in one copy; the items point into the device blocks
    lw.set_sequence_mode(mode)
    fmt = lw.Q4_K
    spec = [(300, 4096, 0, 0), (77, 4096, 0, 0), (512, 4096, 1, DEP), (129, 2048, 2, DEP)]     # rows, cols, which x, flags
    xs = [synth.activations(150, i, 1, c) for i, c in ((0, 4096), (1, 4096), (2, 2048))]
    xoff = [0, 4096, 8192]
    in_host = torch.from_numpy(np.concatenate([x.reshape(-1) for x in xs])).pin_memory()
    in_dev = Guarded(in_host.numel())
    yoff, total = [], 0
    for rows, _, _, _ in spec:
        yoff.append(total)
        total += (rows + 63) & ~63
    out_dev = Guarded(total)
    out_host = torch.full((total,), float("nan"), dtype=torch.float32).pin_memory()
    items, refs, keep = [], [], []
    for j, (rows, cols, xi, flags) in enumerate(spec):
        blocks = quantized_weights(fmt, rows, cols, seed=151 + j)
        w = torch.from_numpy(blocks).cuda()
        keep.append(w)
        items.append((w, rows, cols, in_dev.t.data_ptr() + 4 * xoff[xi], out_dev.t.data_ptr() + 4 * yoff[j], flags))
        refs.append(oracle.matvec(fmt, blocks, rows, cols, xs[xi], 1, nthreads=4))
    ws = _workspace()
    for _ in range(2):
        lw.matvec_sequence_host(fmt, items, in_host, in_dev.t, 4 * in_host.numel(), out_dev.t, out_host, 4 * total, ws.t)
    torch.cuda.synchronize()
    assert lw.device_status() == 0
    in_dev.check("device input block")
    out_dev.check("device output block")
    for j, (rows, _, _, _) in enumerate(spec):
        check_matvec(out_host.numpy()[yoff[j]:yoff[j] + rows], refs[j][0], refs[j][1], "host sequence item %d" % j)
    L = lw.lib()
    import ctypes
    arr = lw.seq_items(items)
    assert L.lw_matvec_sequence_host(fmt, len(items), ctypes.cast(arr, ctypes.c_void_p), None, in_dev.t.data_ptr(), 16,
                                     out_dev.t.data_ptr(), out_host.data_ptr(), 16, ws.t.data_ptr(), 256, None) == lw.ERR_NULL
    assert L.lw_set_sequence_mode(7) == lw.ERR_FORMAT


def test_sequence_falls_back_for_shapes_outside_the_streaming_kernels():
    fmt = lw.Q8_0
    items, keep, refs = [], [], []
    for j, (rows, cols) in enumerate([(10, 96), (33, 4096), (5, 32768)]):
        blocks = quantized_weights(fmt, rows, cols, seed=140 + j)
        X = synth.activations(140, j, 1, cols)
        w, x, y = torch.from_numpy(blocks).cuda(), torch.from_numpy(X).cuda(), Guarded((1, rows))
        keep.append((w, x, y))
        items.append((w, rows, cols, x, y.t, DEP))
        refs.append(oracle.matvec(fmt, blocks, rows, cols, X, 1))
    ws = _workspace()
    lw.matvec_sequence(fmt, items, ws.t)
    torch.cuda.synchronize()
    for (w, x, y), (y_ref, s_ref) in zip(keep, refs):
        y.check("fallback item")
        check_matvec(y.t.cpu().numpy(), y_ref, s_ref, "fallback item")
    # a forced variant takes the same route
    lw.set_variant(lw.VARIANT_GENERIC)
    try:
        items2, keep2, refs2 = _layer_like(lw.Q4_0, 2048, 4096, seed=141)
        lw.matvec_sequence(lw.Q4_0, items2, ws.t)
        torch.cuda.synchronize()
        for (w, x, y), (y_ref, s_ref) in zip(keep2, refs2):
            check_matvec(y.t.cpu().numpy(), y_ref, s_ref, "forced generic")
    finally:
        lw.set_variant(lw.VARIANT_AUTO)
    assert lw.device_status() == 0


def test_sequence_argument_errors_enqueue_nothing():
    L = lw.lib()
    w = torch.zeros(4096 * 34 // 32 * 4, dtype=torch.uint8, device="cuda")
    x = torch.zeros(4096, dtype=torch.float32, device="cuda")
    y = torch.full((8,), 5.0, dtype=torch.float32, device="cuda")
    ws = torch.zeros(64, dtype=torch.int32, device="cuda")
    good = (w, 4, 4096, x, y, 0)

    def call(items, workspace=ws, nbytes=256, fmt=lw.Q8_0):
        arr = lw.seq_items(items)
        import ctypes
        return L.lw_matvec_sequence(fmt, len(items), ctypes.cast(arr, ctypes.c_void_p), lw._addr(workspace), nbytes, None)

    assert call([good], fmt=99) == lw.ERR_FORMAT
    assert call([good], workspace=None) == lw.ERR_NULL
    assert call([good], nbytes=8) == lw.ERR_WORKSPACE
    assert call([good] * 641) == lw.ERR_SHAPE
    assert call([good, (w, 0, 4096, x, y, 0)]) == lw.ERR_SHAPE
    assert call([good, (w, 4, 4010, x, y, 0)]) == lw.ERR_SHAPE
    assert call([good, (w, 4, 4096, None, y, 0)]) == lw.ERR_NULL
    assert call([good, (w, 4, 4096, x, y, 6)]) == lw.ERR_FORMAT
    assert call([(w, 4, 4096, lw._addr(x) + 4, y, 0)]) == lw.ERR_ALIGN
    assert L.lw_matvec_sequence(lw.Q8_0, 1, None, lw._addr(ws), 256, None) == lw.ERR_NULL
    torch.cuda.synchronize()
    assert (y == 5.0).all()


@pytest.mark.parametrize("overlap", [0, 2])
@pytest.mark.parametrize("batch", [1, 4, 11])
@pytest.mark.parametrize("fmt", [lw.Q4_K, lw.Q8_0, lw.F16, lw.Q6_K, lw.Q2_K])
def test_batched_chain_and_its_host_buffer_form(fmt, batch, overlap):
    # lw_matvec_sequence_batch: the chain with several columns per item (one grouped call per run of items that share
    # their X: the tensor-core kernel from two columns on), and lw_matvec_sequence_batch_host around it: the
    # input block from pinned host memory in one copy, the result block back in one copy
    lw.set_overlap(overlap)
    try:
        spec = [(300, 2048, 0, DEP), (77, 2048, 0, 0), (513, 2048, 0, 0), (256, 2048, 1, DEP), (129, 4096, 2, DEP),
                (40, 4096, 2, 0)]                                         # rows, cols, which x, flags
        xs = [synth.activations(170, i, batch, c) for i, c in ((0, 2048), (1, 2048), (2, 4096))]
        xoff = [0, batch * 2048, 2 * batch * 2048]
        in_host = torch.from_numpy(np.concatenate([x.reshape(-1) for x in xs])).pin_memory()
        in_dev = Guarded(in_host.numel())
        yoff, total = [], 0
        for rows, _, _, _ in spec:
            yoff.append(total)
            total += (batch * rows + 63) & ~63
        out_dev = Guarded(total)
        out_host = torch.full((total,), float("nan"), dtype=torch.float32).pin_memory()
        items, refs, keep = [], [], []
        for j, (rows, cols, xi, flags) in enumerate(spec):
            blocks = quantized_weights(fmt, rows, cols, seed=171 + j, tensor_id=fmt)
            w = torch.from_numpy(blocks).cuda()
            keep.append(w)
            items.append((w, rows, cols, in_dev.t.data_ptr() + 4 * xoff[xi], out_dev.t.data_ptr() + 4 * yoff[j], flags))
            refs.append(oracle.matvec(fmt, blocks, rows, cols, xs[xi], batch, nthreads=4))
        for _ in range(2):
            lw.matvec_sequence_batch_host(fmt, items, batch, in_host, in_dev.t, 4 * in_host.numel(), out_dev.t, out_host,
                                          4 * total)
        torch.cuda.synchronize()
        assert lw.device_status() == 0
        in_dev.check("device input block")
        out_dev.check("device output block")
        for j, (rows, _, _, _) in enumerate(spec):
            got = out_host.numpy()[yoff[j]:yoff[j] + batch * rows].reshape(batch, rows)
            check_matvec(got, refs[j][0], refs[j][1], "batched chain item %d" % j)
        # the device-resident form gives the same results
        out_dev.t.fill_(float("nan"))
        lw.matvec_sequence_batch(fmt, items, batch)
        torch.cuda.synchronize()
        for j, (rows, _, _, _) in enumerate(spec):
            got = out_dev.t[yoff[j]:yoff[j] + batch * rows].cpu().numpy().reshape(batch, rows)
            check_matvec(got, refs[j][0], refs[j][1], "batched chain item %d (device)" % j)
        L = lw.lib()
        import ctypes
        arr = lw.seq_items(items)
        assert L.lw_matvec_sequence_batch(fmt, len(items), ctypes.cast(arr, ctypes.c_void_p), 17, None) == lw.ERR_BATCH
        assert L.lw_matvec_sequence_batch(fmt, 0, ctypes.cast(arr, ctypes.c_void_p), 4, None) == lw.ERR_SHAPE
        assert L.lw_matvec_sequence_batch_host(fmt, len(items), ctypes.cast(arr, ctypes.c_void_p), 4, None,
                                               in_dev.t.data_ptr(), 16, out_dev.t.data_ptr(), out_host.data_ptr(), 16,
                                               None) == lw.ERR_NULL
    finally:
        lw.set_overlap(0)


@pytest.mark.parametrize("overlap", [0, 2])
def test_batched_chain_over_ping_pong_buffers(overlap):
    # every item's Y is the buffer the item before it read its X from: the chain call must not let a launch clear
    # the next launch's outputs here (they overlap its own input) and falls back to the clearing kernel
    fmt, batch, dims = lw.Q4_0, 6, [1024, 768, 2048, 512, 1024]
    mats = [quantized_weights(fmt, dims[j + 1], dims[j], seed=180 + j, tensor_id=fmt) for j in range(len(dims) - 1)]
    wd = [torch.from_numpy(m).cuda() for m in mats]
    x0 = synth.activations(180, 0, batch, dims[0])
    bufs = [Guarded(batch * max(dims)), Guarded(batch * max(dims))]
    bufs[0].t[:x0.size] = torch.from_numpy(x0.reshape(-1)).cuda()
    items = [(wd[j], dims[j + 1], dims[j], bufs[j & 1].t, bufs[(j + 1) & 1].t, DEP) for j in range(len(mats))]
    lw.set_overlap(overlap)
    try:
        lw.matvec_sequence_batch(fmt, items, batch)
        torch.cuda.synchronize()
        assert lw.device_status() == 0
        for b in bufs:
            b.check("ping-pong buffer")
        # the last layer against the oracle fed with the GPU's own input to that layer
        x_in = bufs[(len(mats) - 1) & 1].t[:batch * dims[-2]].cpu().numpy().reshape(batch, dims[-2])
        got = bufs[len(mats) & 1].t[:batch * dims[-1]].cpu().numpy().reshape(batch, dims[-1])
        y_ref, s_ref = oracle.matvec(fmt, mats[-1], dims[-1], dims[-2], x_in, batch, nthreads=4)
        check_matvec(got, y_ref, s_ref, "ping-pong chain")
        # and the first layer, recomputed alone
        y1 = Guarded((batch, dims[1]))
        lw.matvec(fmt, wd[0], dims[1], dims[0], torch.from_numpy(x0).cuda(), y1.t, batch)
        torch.cuda.synchronize()
        y_ref, s_ref = oracle.matvec(fmt, mats[0], dims[1], dims[0], x0, batch, nthreads=4)
        check_matvec(y1.t.cpu().numpy(), y_ref, s_ref, "first layer")
    finally:
        lw.set_overlap(0)


def _host_chain(fmt, batch, layout, n_items=24, rows=1500, cols=4096, seed=190):
    """A chain of dependent items with one X each, the X in the input block and the Y in the result block in the
    order `layout` gives; with "hole", item 0 writes into a gap of the input block instead."""
    order = list(range(n_items))
    if layout == "descending":
        order = order[::-1]
    elif layout == "shuffled":
        order = [int(v) for v in np.random.default_rng(5).permutation(n_items)]
    xw, yw = batch * cols, (batch * rows + 63) & ~63
    hole = yw if layout == "hole" else 0
    in_words, out_words = n_items * xw + hole, n_items * yw
    in_np = np.full(in_words, np.nan, dtype=np.float32)
    xs, items, refs, keep = [], [], [], []
    in_dev, out_dev = Guarded(in_words), Guarded(out_words)
    for j in range(n_items):
        X = synth.activations(seed, j, batch, cols)
        in_np[order[j] * xw:(order[j] + 1) * xw] = X.reshape(-1)
        blocks = quantized_weights(fmt, rows, cols, seed=seed + 1 + j, tensor_id=fmt)
        w = torch.from_numpy(blocks).cuda()
        keep.append(w)
        y_ptr = out_dev.t.data_ptr() + 4 * order[j] * yw
        if hole and j == 0:
            y_ptr = in_dev.t.data_ptr() + 4 * n_items * xw         # behind every X: the last piece of a piecewise copy
        items.append((w, rows, cols, in_dev.t.data_ptr() + 4 * order[j] * xw, y_ptr, DEP))
        refs.append(oracle.matvec(fmt, blocks, rows, cols, X, batch, nthreads=4))
    in_host = torch.from_numpy(in_np).pin_memory()
    out_host = torch.full((out_words,), float("nan"), dtype=torch.float32).pin_memory()
    return dict(items=items, refs=refs, keep=keep, in_host=in_host, in_dev=in_dev, out_dev=out_dev, out_host=out_host,
                order=order, yw=yw, xw=xw, rows=rows, hole=hole, n=n_items, batch=batch)


def _check_host_chain(c, what):
    torch.cuda.synchronize()
    assert lw.device_status() == 0
    c["in_dev"].check("device input block")
    c["out_dev"].check("device output block")
    batch, rows = c["batch"], c["rows"]
    for j in range(c["n"]):
        if c["hole"] and j == 0:
            got = c["in_dev"].t[c["n"] * c["xw"]:c["n"] * c["xw"] + batch * rows].cpu().numpy()
        else:
            got = c["out_host"].numpy()[c["order"][j] * c["yw"]:c["order"][j] * c["yw"] + batch * rows]
        check_matvec(got.reshape(batch, rows), c["refs"][j][0], c["refs"][j][1], "%s item %d" % (what, j))
    # the whole input block is on the device afterwards, whether an item read it or not
    n_x = c["n"] * c["xw"]
    assert torch.equal(c["in_dev"].t[:n_x].cpu(), c["in_host"][:n_x])


@pytest.mark.parametrize("graph", [False, True])
@pytest.mark.parametrize("layout", ["ascending", "descending", "shuffled", "hole"])
@pytest.mark.parametrize("mode", MODES)
def test_host_chain_whose_blocks_are_copied_in_pieces(mode, layout, graph):
    # blocks of several hundred KB: the input block goes in piece by piece beside the kernels and the result block
    # leaves piece by piece; whatever the order of the activations and results inside the blocks, the outcome is
    # that of one copy before and one copy behind the chain.  "hole": an item writes into the input block, which
    # a late piece must not overwrite.
    lw.set_sequence_mode(mode)
    fmt = lw.Q4_K
    c = _host_chain(fmt, 1, layout)
    ws = _workspace()

    def call(stream=None):
        lw.matvec_sequence_host(fmt, c["items"], c["in_host"], c["in_dev"].t, 4 * c["in_host"].numel(), c["out_dev"].t,
                                c["out_host"], 4 * c["out_host"].numel(), ws.t, stream=stream)
    if not graph:
        for _ in range(2):                         # on the default stream, twice in a row
            call()
        _check_host_chain(c, "eager, default stream")
        return
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        call(side)
        side.synchronize()
        _check_host_chain(c, "eager")
        if graph:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                call(side)
            for _ in range(3):
                c["out_host"].fill_(float("nan"))
                c["in_dev"].t.fill_(float("nan"))
                g.replay()
                torch.cuda.synchronize()
                _check_host_chain(c, "replay")


@pytest.mark.parametrize("overlap", [0, 2])
@pytest.mark.parametrize("layout", ["ascending", "shuffled", "hole"])
@pytest.mark.parametrize("fmt,batch", [(lw.Q4_0, 3), (lw.Q8_0, 8), (lw.F16, 2)])
def test_batched_host_chain_whose_blocks_are_copied_in_pieces(fmt, batch, layout, overlap):
    lw.set_overlap(overlap)
    try:
        c = _host_chain(fmt, batch, layout, n_items=12, rows=700, cols=2048, seed=230)
        side = torch.cuda.Stream()

        def call(stream):
            lw.matvec_sequence_batch_host(fmt, c["items"], batch, c["in_host"], c["in_dev"].t, 4 * c["in_host"].numel(),
                                          c["out_dev"].t, c["out_host"], 4 * c["out_host"].numel(), stream)
        with torch.cuda.stream(side):
            call(side)
            side.synchronize()
            _check_host_chain(c, "eager")
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                call(side)
            for _ in range(2):
                c["out_host"].fill_(float("nan"))
                c["in_dev"].t.fill_(float("nan"))
                g.replay()
                torch.cuda.synchronize()
                _check_host_chain(c, "replay")
    finally:
        lw.set_overlap(0)


def test_host_chain_called_while_another_is_being_captured():
    # a captured call holds the library's copy streams until its capture ends; a call on another stream in the
    # meantime must run at once on copy streams of its own, not land in that graph
    lw.set_sequence_mode(lw.SEQ_LAUNCHES)
    fmt = lw.Q8_0
    a = _host_chain(fmt, 1, "ascending", n_items=10, rows=900, cols=4096, seed=260)
    b = _host_chain(fmt, 1, "ascending", n_items=10, rows=900, cols=4096, seed=280)
    ws_a, ws_b = _workspace(), _workspace()

    def call(c, ws, stream):
        lw.matvec_sequence_host(fmt, c["items"], c["in_host"], c["in_dev"].t, 4 * c["in_host"].numel(), c["out_dev"].t,
                                c["out_host"], 4 * c["out_host"].numel(), ws.t, stream=stream)
    side, other = torch.cuda.Stream(), torch.cuda.Stream()
    call(a, ws_a, side)                                      # warm-up outside capture
    side.synchronize()
    a["out_host"].fill_(float("nan"))
    a["in_dev"].t.fill_(float("nan"))
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side, capture_error_mode="relaxed"):
        call(a, ws_a, side)
        call(b, ws_b, other)                                 # not captured: runs now
        other.synchronize()
        _check = b["out_host"].numpy().copy()
    assert np.isfinite(_check).any(), "the call on the other stream did not run while the capture was open"
    _check_host_chain(b, "beside an open capture")
    assert not np.isfinite(a["out_host"].numpy()).any(), "the captured call ran before its graph was replayed"
    g.replay()
    _check_host_chain(a, "captured beside another call")
