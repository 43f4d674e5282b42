// C ABI of the lw library: argument validation, variant selection and launch.
#include <cuda_runtime.h>

#include <atomic>
#include <cstdlib>

#include "lw_internal.h"

namespace lw {

static std::atomic<int> g_variant{-1};   // -1: not initialised (environment not read yet)
static std::atomic<int> g_overlap{0};
static std::atomic<int> g_sequence_mode{LW_SEQ_AUTO};

static int forced_variant() {
    int v = g_variant.load(std::memory_order_relaxed);
    if (v >= 0) return v;
    v = LW_VARIANT_AUTO;
    if (const char* env = std::getenv("LW_FORCE_VARIANT")) {
        const int e = std::atoi(env);
        if (e >= LW_VARIANT_AUTO && e <= LW_VARIANT_MMA) v = e;
    }
    int expected = -1;
    g_variant.compare_exchange_strong(expected, v);
    return g_variant.load();
}

// Does the current device take cooperative launches (kernels whose CTAs wait for one another)?
static bool cooperative_launch_ok() {
    static int coop[64] = {0};          // 0 unknown, 1 yes, -1 no
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    if (coop[dev] == 0) {
        int v = 0;
        coop[dev] = (cudaDeviceGetAttribute(&v, cudaDevAttrCooperativeLaunch, dev) == cudaSuccess && v) ? 1 : -1;
    }
    return coop[dev] == 1;
}

static bool misaligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

static int check_matvec_args(int fmt, const void* W, int64_t rows, int64_t cols, const void* X,
                             const void* Y, int batch) {
    if (lw_block_elems(fmt) == 0) return LW_ERR_FORMAT;
    if (!W || !X || !Y) return LW_ERR_NULL;
    if (rows < 1 || lw_row_bytes(fmt, cols) == 0) return LW_ERR_SHAPE;
    if (batch < 1 || batch > 16) return LW_ERR_BATCH;
    if (misaligned16(W) || misaligned16(X) || misaligned16(Y)) return LW_ERR_ALIGN;
    return LW_OK;
}

// Batch 2..16 without a forced variant: may the columns be run one by one through the batch-1
// streaming kernel (grouped launches of up to kColumnsPerLaunch columns)?  Measured on the 1B f16
// shapes: 0.87 / 1.37 ms per step at batch 2 / 4 against 1.31 / 1.65 ms for the tiled fp32 kernel,
// but 2.69 / 5.32 ms against 2.19 / 4.51 ms at batch 8 / 16.
constexpr int kColumnsPerLaunch = 4;
constexpr int kTileMinColumns = 7;
constexpr int kMmaMinColumns = 3;
static bool columnwise(int fmt, int64_t rows, int64_t cols, int batch) {
    if (fmt == LW_F16 && batch > 4) return false;      // f16 from 5 columns: the tiled fp32 kernel is faster
    return batch > 1 && forced_variant() == LW_VARIANT_AUTO && rows <= INT32_MAX &&
           matvec_stream_supported(fmt, rows, cols, 1) &&
           matvec_group_supported(fmt, cols, batch < kColumnsPerLaunch ? batch : kColumnsPerLaunch);
}

static int pick_variant(int fmt, int64_t rows, int64_t cols, int batch) {
    const int forced = forced_variant();
    // batch 2..16: the tensor-core kernel where it applies (every format, cols a multiple of 256, q6_K of 2048, q2_K
    // of 1024; all columns in one pass over the weights).  Measured on the 8B shapes (ms per step, q4_0, one call
    // per mat-vec): 2.3 / 2.3 / 2.3 / 3.1 for 3 / 4 / 8 / 16 columns, against 2.2 / 3.7 / 7.3 for 2 / 4 / 8 columns
    // through the batch-1 kernel and 5.6 / 10.9 for 8 / 16 through the fp32 tile kernel: AUTO takes it from three
    // columns on.  The fp32 tile kernel stays for forced selection.
    if (matvec_mma_supported(fmt, rows, cols, batch) &&
        (forced == LW_VARIANT_MMA || (forced == LW_VARIANT_AUTO && batch >= kMmaMinColumns)))
        return LW_VARIANT_MMA;
    if (matvec_tile_supported(fmt, rows, cols, batch) &&
        (forced == LW_VARIANT_TILE || (forced == LW_VARIANT_AUTO && batch >= kTileMinColumns)))
        return LW_VARIANT_TILE;
    if (columnwise(fmt, rows, cols, batch)) return fmt == LW_F16 ? LW_VARIANT_STREAM : LW_VARIANT_IDOT;
    if (forced == LW_VARIANT_GENERIC || !matvec_stream_supported(fmt, rows, cols, batch)) return LW_VARIANT_GENERIC;
    if (batch > 1) {
        // Batched integer-dot kernel up to 4 columns (measured faster on B200: 3.7 / 6.6 ms per 8B q4_0
        // step at batch 2 / 4 against 6.4 / 7.9 ms); from 5 columns the tiled fp32 kernel wins unless forced.
        if (forced == LW_VARIANT_STREAM) return LW_VARIANT_GENERIC;
        return (batch <= 4 || forced == LW_VARIANT_IDOT) ? LW_VARIANT_IDOT : LW_VARIANT_GENERIC;
    }
    if (fmt == LW_F16) return LW_VARIANT_STREAM;
    // the fp32-activation streaming family exists for q8_0, q4_0 and q4_K; for the later formats a forced
    // STREAM falls back to the next simpler variant
    if (forced == LW_VARIANT_STREAM) return fmt <= LW_Q4_K ? LW_VARIANT_STREAM : LW_VARIANT_GENERIC;
    return LW_VARIANT_IDOT;
}

}  // namespace lw

using namespace lw;

extern "C" {

size_t lw_block_elems(int fmt) {
    switch (fmt) {
        case LW_F16: return 1;
        case LW_Q8_0: return 32;
        case LW_Q4_0: return 32;
        case LW_Q4_K: return 256;
        case LW_Q6_K: return 256;
        case LW_Q5_K: return 256;
        case LW_Q2_K: return 256;
        case LW_Q4_1: return 32;
        case LW_Q5_0: return 32;
        case LW_Q5_1: return 32;
        default: return 0;
    }
}

size_t lw_block_bytes(int fmt) {
    switch (fmt) {
        case LW_F16: return 2;
        case LW_Q8_0: return 34;
        case LW_Q4_0: return 18;
        case LW_Q4_K: return 144;
        case LW_Q6_K: return 210;
        case LW_Q5_K: return 176;
        case LW_Q2_K: return 84;
        case LW_Q4_1: return 20;
        case LW_Q5_0: return 22;
        case LW_Q5_1: return 24;
        default: return 0;
    }
}

size_t lw_row_bytes(int fmt, int64_t cols) {
    const size_t be = lw_block_elems(fmt);
    if (be == 0 || cols <= 0) return 0;
    const int64_t quantum = (fmt == LW_Q4_K || fmt == LW_Q6_K || fmt == LW_Q5_K || fmt == LW_Q2_K) ? 256 : 32;
    if (cols % quantum != 0) return 0;
    return (size_t)(cols / (int64_t)be) * lw_block_bytes(fmt);
}

const char* lw_status_string(int status) {
    switch (status) {
        case LW_OK: return "ok";
        case LW_ERR_FORMAT: return "unknown format or option value";
        case LW_ERR_SHAPE: return "bad shape: rows < 1 or cols/n not a whole number of blocks";
        case LW_ERR_NULL: return "null pointer";
        case LW_ERR_ALIGN: return "device pointer not 16-byte aligned";
        case LW_ERR_BATCH: return "batch outside 1..16";
        case LW_ERR_NONFINITE: return "non-finite input or scale";
        case LW_ERR_CUDA: return "CUDA runtime error";
        case LW_ERR_DEVICE: return "device-side fault recorded";
        case LW_ERR_WORKSPACE: return "workspace smaller than lw_attn_workspace_bytes (or shape beyond the built-in scratch)";
        default: return "unknown status";
    }
}

int lw_quantize(int fmt, const float* src, int64_t n, void* dst) { return quantize_host(fmt, src, n, dst); }

int lw_dequant(int fmt, const void* W_blocks, int64_t n, float* out, void* stream) {
    if (lw_block_elems(fmt) == 0) return LW_ERR_FORMAT;
    if (!W_blocks || !out) return LW_ERR_NULL;
    if (lw_row_bytes(fmt, n) == 0) return LW_ERR_SHAPE;
    if (misaligned16(W_blocks) || misaligned16(out)) return LW_ERR_ALIGN;
    return launch_dequant(fmt, W_blocks, n, out, static_cast<cudaStream_t>(stream)) == 0 ? LW_OK : LW_ERR_CUDA;
}

int lw_matvec(int fmt, const void* W_blocks, int64_t rows, int64_t cols, const float* X, float* Y,
              int batch, void* stream) {
    const int rc = check_matvec_args(fmt, W_blocks, rows, cols, X, Y, batch);
    if (rc != LW_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int err;
    const int variant = pick_variant(fmt, rows, cols, batch);
    if (variant == LW_VARIANT_MMA) {
        // without overlap: one cooperative launch that clears Y itself; with it: a clearing kernel and the main
        // kernel chained by programmatic dependent launch
        const int ov = g_overlap.load();
        err = launch_matvec_mma(fmt, W_blocks, rows, cols, X, Y, batch, ov, ov == 0 && cooperative_launch_ok(), s);
    } else if (variant == LW_VARIANT_TILE && forced_variant() == LW_VARIANT_AUTO) {
        // passes of seven or eight columns through the tile kernel, the remainder through the batch-1 kernel
        const int tiled = batch - (batch % 8 >= kTileMinColumns ? 0 : batch % 8);
        err = launch_matvec_tile(fmt, W_blocks, rows, cols, X, Y, tiled, s);
        if (err == 0 && tiled < batch) {
            const int rc2 = lw_matvec(fmt, W_blocks, rows, cols, X + (int64_t)tiled * cols, Y + (int64_t)tiled * rows,
                                      batch - tiled, stream);
            if (rc2 != LW_OK) return rc2;
        }
    } else if (variant == LW_VARIANT_TILE) {
        err = launch_matvec_tile(fmt, W_blocks, rows, cols, X, Y, batch, s);
    } else if (columnwise(fmt, rows, cols, batch)) {
        // One streaming pass per activation column, four columns per grouped launch (their CTAs walk
        // the same matrix at the same time, so most of the re-reads hit L2): on B200 this beats both
        // batched kernels at every batch size 2..16.
        err = 0;
        for (int b0 = 0; b0 < batch && err == 0; b0 += kColumnsPerLaunch) {
            const int n = batch - b0 < kColumnsPerLaunch ? batch - b0 : kColumnsPerLaunch;
            const void* W[8];
            const float* Xs[8];
            float* Ys[8];
            int64_t rws[8];
            for (int j = 0; j < n; ++j) {
                W[j] = W_blocks;
                Xs[j] = X + (int64_t)(b0 + j) * cols;
                Ys[j] = Y + (int64_t)(b0 + j) * rows;
                rws[j] = rows;
            }
            err = launch_matvec_stream_group(fmt, true, cols, n, W, rws, Xs, Ys, g_overlap.load() != 0, s);
        }
    } else if (variant != LW_VARIANT_GENERIC && batch > 1)
        err = launch_matvec_stream_batched(fmt, W_blocks, rows, cols, X, Y, batch, g_overlap.load() != 0, s);
    else if (variant != LW_VARIANT_GENERIC)
        err = launch_matvec_stream(fmt, variant == LW_VARIANT_IDOT, W_blocks, rows, cols, X, Y,
                                   g_overlap.load() != 0, s);
    else
        err = launch_matvec_generic(fmt, W_blocks, rows, cols, X, Y, batch, s);
    return err == 0 ? LW_OK : LW_ERR_CUDA;
}

int lw_matvec_group_batch(int fmt, int64_t cols, int n_items, const lw_group_item* items, int batch, void* stream) {
    if (batch == 1) return lw_matvec_group(fmt, cols, n_items, items, stream);
    if (lw_block_elems(fmt) == 0) return LW_ERR_FORMAT;
    if (!items) return LW_ERR_NULL;
    if (n_items < 1 || n_items > 8) return LW_ERR_SHAPE;
    const void* W[8];
    const float* X[8];
    float* Y[8];
    int64_t rows[8];
    for (int j = 0; j < n_items; ++j) {
        const int rc = check_matvec_args(fmt, items[j].W_blocks, items[j].rows, cols, items[j].X, items[j].Y, batch);
        if (rc != LW_OK) return rc;
        W[j] = items[j].W_blocks;
        X[j] = items[j].X;
        Y[j] = items[j].Y;
        rows[j] = items[j].rows;
    }
    const int forced = forced_variant();
    if ((forced == LW_VARIANT_AUTO || forced == LW_VARIANT_MMA) && matvec_mma_group_supported(fmt, cols, n_items, rows, batch)) {
        const int ov = g_overlap.load();
        const int err = launch_matvec_mma_group(fmt, cols, n_items, W, rows, X, Y, batch, ov,
                                                ov == 0 && cooperative_launch_ok(), static_cast<cudaStream_t>(stream), false, 0,
                                                nullptr, nullptr);
        return err == 0 ? LW_OK : LW_ERR_CUDA;
    }
    for (int j = 0; j < n_items; ++j) {
        const int rc = lw_matvec(fmt, W[j], rows[j], cols, X[j], Y[j], batch, stream);
        if (rc != LW_OK) return rc;
    }
    return LW_OK;
}

int lw_matvec_group(int fmt, int64_t cols, int n_items, const lw_group_item* items, void* stream) {
    if (lw_block_elems(fmt) == 0) return LW_ERR_FORMAT;
    if (!items) return LW_ERR_NULL;
    if (n_items < 1 || n_items > 8) return LW_ERR_SHAPE;
    for (int j = 0; j < n_items; ++j) {
        const int rc = check_matvec_args(fmt, items[j].W_blocks, items[j].rows, cols, items[j].X, items[j].Y, 1);
        if (rc != LW_OK) return rc;
    }
    const int forced = forced_variant();
    const bool has_fp32_stream = fmt <= LW_Q4_K;
    if (forced != LW_VARIANT_GENERIC && !(forced == LW_VARIANT_STREAM && !has_fp32_stream) &&
        matvec_group_supported(fmt, cols, n_items)) {
        const void* W[8];
        const float* X[8];
        float* Y[8];
        int64_t rows[8];
        for (int j = 0; j < n_items; ++j) {
            W[j] = items[j].W_blocks;
            X[j] = items[j].X;
            Y[j] = items[j].Y;
            rows[j] = items[j].rows;
        }
        const bool idot = forced != LW_VARIANT_STREAM && fmt != LW_F16;
        const int err = launch_matvec_stream_group(fmt, idot, cols, n_items, W, rows, X, Y, g_overlap.load() != 0,
                                                   static_cast<cudaStream_t>(stream));
        return err == 0 ? LW_OK : LW_ERR_CUDA;
    }
    for (int j = 0; j < n_items; ++j) {
        const int rc = lw_matvec(fmt, items[j].W_blocks, items[j].rows, cols, items[j].X, items[j].Y, 1, stream);
        if (rc != LW_OK) return rc;
    }
    return LW_OK;
}

int64_t lw_matvec_sequence_workspace_bytes(void) { return 256; }

static int check_sequence(int fmt, int n_items, const lw_seq_item* items, void* workspace, int64_t workspace_bytes) {
    if (lw_block_elems(fmt) == 0) return LW_ERR_FORMAT;
    if (!items || !workspace) return LW_ERR_NULL;
    if (n_items < 1 || n_items > 640) return LW_ERR_SHAPE;
    if (misaligned16(workspace)) return LW_ERR_ALIGN;
    if (workspace_bytes < lw_matvec_sequence_workspace_bytes()) return LW_ERR_WORKSPACE;
    for (int j = 0; j < n_items; ++j) {
        const int rc = check_matvec_args(fmt, items[j].W_blocks, items[j].rows, items[j].cols, items[j].X, items[j].Y, 1);
        if (rc != LW_OK) return rc;
        if (items[j].flags & ~LW_SEQ_DEPENDENT) return LW_ERR_FORMAT;
    }
    return LW_OK;
}

// The chain, arguments already checked.  `pipe` (may be null) carries the copies of the host form: it is told
// before and behind every launch which items the launch runs.
static int run_sequence(int fmt, int n_items, const lw_seq_item* items, void* workspace, void* stream, HostPipe* pipe) {
    const bool can = cooperative_launch_ok();
    const bool streaming = forced_variant() == LW_VARIANT_AUTO && matvec_sequence_supported(fmt, n_items, items);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (streaming && can && g_sequence_mode.load() == LW_SEQ_PERSISTENT) {
        // one kernel for the whole chain: nothing to overlap copies with from the host
        if (pipe) pipe->whole_copies_only();
        if (pipe && !pipe->begin()) return LW_ERR_CUDA;
        const int err = launch_matvec_sequence(fmt, n_items, items, static_cast<unsigned*>(workspace), s);
        if (err != 0) return LW_ERR_CUDA;
        return !pipe || pipe->end() ? LW_OK : LW_ERR_CUDA;
    }
    if (pipe && !pipe->begin()) return LW_ERR_CUDA;
    if (streaming) {
        // One launch per phase (consecutive items that share their X and are not flagged dependent), chained
        // with programmatic dependent launch: stream order provides every dependency, and a kernel waits for
        // its predecessor before it requests any of W or X.
        int j = 0;
        while (j < n_items) {
            int n = 1;
            while (j + n < n_items && n < 8 && !(items[j + n].flags & LW_SEQ_DEPENDENT) && items[j + n].X == items[j].X &&
                   items[j + n].cols == items[j].cols)
                ++n;
            const void* W[8];
            const float* X[8];
            float* Y[8];
            int64_t rows[8];
            for (int k = 0; k < n; ++k) {
                W[k] = items[j + k].W_blocks;
                X[k] = items[j + k].X;
                Y[k] = items[j + k].Y;
                rows[k] = items[j + k].rows;
            }
            if (pipe && !pipe->before(j, n)) return LW_ERR_CUDA;
            const int err = n == 1 ? launch_matvec_stream(fmt, fmt != LW_F16, W[0], rows[0], items[j].cols, X[0], Y[0], true, s)
                                   : launch_matvec_stream_group(fmt, fmt != LW_F16, items[j].cols, n, W, rows, X, Y, true, s);
            if (err != 0) return LW_ERR_CUDA;
            if (pipe && !pipe->after(j, n)) return LW_ERR_CUDA;
            j += n;
        }
        return !pipe || pipe->end() ? LW_OK : LW_ERR_CUDA;
    }
    for (int j = 0; j < n_items; ++j) {
        if (pipe && !pipe->before(j, 1)) return LW_ERR_CUDA;
        const int rc = lw_matvec(fmt, items[j].W_blocks, items[j].rows, items[j].cols, items[j].X, items[j].Y, 1, stream);
        if (rc != LW_OK) return rc;
        if (pipe && !pipe->after(j, 1)) return LW_ERR_CUDA;
    }
    return !pipe || pipe->end() ? LW_OK : LW_ERR_CUDA;
}

int lw_matvec_sequence(int fmt, int n_items, const lw_seq_item* items, void* workspace, int64_t workspace_bytes,
                       void* stream) {
    const int rc = check_sequence(fmt, n_items, items, workspace, workspace_bytes);
    return rc != LW_OK ? rc : run_sequence(fmt, n_items, items, workspace, stream, nullptr);
}

int lw_matvec_sequence_host(int fmt, int n_items, const lw_seq_item* items, const void* in_host, void* in_dev,
                            int64_t in_bytes, const void* out_dev, void* out_host, int64_t out_bytes, void* workspace,
                            int64_t workspace_bytes, void* stream) {
    if (!in_host || !in_dev || !out_dev || !out_host) return LW_ERR_NULL;
    if (in_bytes < 0 || out_bytes < 0) return LW_ERR_SHAPE;
    // validate everything before the first copy is queued: a call that fails enqueues nothing
    const int rc = check_sequence(fmt, n_items, items, workspace, workspace_bytes);
    if (rc != LW_OK) return rc;
    HostPipe pipe(n_items, items, 1, in_host, in_dev, in_bytes, out_dev, out_host, out_bytes, static_cast<cudaStream_t>(stream));
    return run_sequence(fmt, n_items, items, workspace, stream, &pipe);
}

static int check_sequence_batch(int fmt, int n_items, const lw_seq_item* items, int batch) {
    if (lw_block_elems(fmt) == 0) return LW_ERR_FORMAT;
    if (!items) return LW_ERR_NULL;
    if (n_items < 1 || n_items > 640) return LW_ERR_SHAPE;
    for (int j = 0; j < n_items; ++j) {
        const int rc = check_matvec_args(fmt, items[j].W_blocks, items[j].rows, items[j].cols, items[j].X, items[j].Y, batch);
        if (rc != LW_OK) return rc;
        if (items[j].flags & ~LW_SEQ_DEPENDENT) return LW_ERR_FORMAT;
    }
    return LW_OK;
}

// Do the byte ranges [a, a + na) and [b, b + nb) overlap?
static bool ranges_overlap(const void* a, int64_t na, const void* b, int64_t nb) {
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return a0 < b0 + (uintptr_t)nb && b0 < a0 + (uintptr_t)na;
}

static int run_sequence_batch(int fmt, int n_items, const lw_seq_item* items, int batch, void* stream, HostPipe* pipe) {
    // One grouped call per run of consecutive items that share their X and their width and are not flagged
    // dependent; stream order provides every dependency.  Where two consecutive runs both take the tensor-core
    // kernel under lw_set_overlap, and the outputs of the second overlap nothing the first reads or writes, the
    // first clears them at its end and the second needs no clearing kernel in front of it.
    const int forced = forced_variant();
    const int ov = g_overlap.load();
    const bool mma_allowed = forced == LW_VARIANT_AUTO || forced == LW_VARIANT_MMA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    auto run_length = [&](int j) {
        int n = 1;
        while (j + n < n_items && n < 8 && !(items[j + n].flags & LW_SEQ_DEPENDENT) && items[j + n].X == items[j].X &&
               items[j + n].cols == items[j].cols)
            ++n;
        return n;
    };
    auto takes_mma = [&](int j, int n) {
        int64_t rows[8];
        for (int k = 0; k < n; ++k) rows[k] = items[j + k].rows;
        return mma_allowed && matvec_mma_group_supported(fmt, items[j].cols, n, rows, batch);
    };
    int j = 0;
    bool pre_cleared = false;
    if (pipe && !pipe->begin()) return LW_ERR_CUDA;
    while (j < n_items) {
        const int n = run_length(j);
        const bool mma = takes_mma(j, n);
        if (pipe && !pipe->before(j, n)) return LW_ERR_CUDA;
        // can this run clear the next run's outputs?
        int n_next = 0;
        float* next_y[8];
        int64_t next_n[8];
        if (mma && ov >= 1 && j + n < n_items) {
            const int jn = j + n, nn = run_length(jn);
            bool ok = takes_mma(jn, nn);
            for (int a = 0; a < nn && ok; ++a) {
                const int64_t ybytes = 4 * (int64_t)batch * items[jn + a].rows;
                for (int b = 0; b < n && ok; ++b)
                    ok = !ranges_overlap(items[jn + a].Y, ybytes, items[j + b].X, 4 * (int64_t)batch * items[j + b].cols) &&
                         !ranges_overlap(items[jn + a].Y, ybytes, items[j + b].Y, 4 * (int64_t)batch * items[j + b].rows) &&
                         !ranges_overlap(items[jn + a].Y, ybytes, items[j + b].W_blocks,
                                         (int64_t)items[j + b].rows * (int64_t)lw_row_bytes(fmt, items[j + b].cols));
            }
            if (ok) {
                n_next = nn;
                for (int a = 0; a < nn; ++a) {
                    next_y[a] = items[jn + a].Y;
                    next_n[a] = (int64_t)batch * items[jn + a].rows;
                }
            }
        }
        if (mma) {
            const void* W[8];
            const float* X[8];
            float* Y[8];
            int64_t rows[8];
            for (int k = 0; k < n; ++k) {
                W[k] = items[j + k].W_blocks;
                X[k] = items[j + k].X;
                Y[k] = items[j + k].Y;
                rows[k] = items[j + k].rows;
            }
            const int err = launch_matvec_mma_group(fmt, items[j].cols, n, W, rows, X, Y, batch, ov,
                                                    ov == 0 && cooperative_launch_ok(), s, pre_cleared, n_next, next_y, next_n);
            if (err != 0) return LW_ERR_CUDA;
        } else {
            lw_group_item g[8];
            for (int k = 0; k < n; ++k) {
                g[k].W_blocks = items[j + k].W_blocks;
                g[k].rows = items[j + k].rows;
                g[k].X = items[j + k].X;
                g[k].Y = items[j + k].Y;
            }
            const int rc2 = lw_matvec_group_batch(fmt, items[j].cols, n, g, batch, stream);
            if (rc2 != LW_OK) return rc2;
        }
        if (pipe && !pipe->after(j, n)) return LW_ERR_CUDA;
        pre_cleared = n_next > 0;
        j += n;
    }
    return !pipe || pipe->end() ? LW_OK : LW_ERR_CUDA;
}

int lw_matvec_sequence_batch(int fmt, int n_items, const lw_seq_item* items, int batch, void* stream) {
    const int rc = check_sequence_batch(fmt, n_items, items, batch);
    return rc != LW_OK ? rc : run_sequence_batch(fmt, n_items, items, batch, stream, nullptr);
}

int lw_matvec_sequence_batch_host(int fmt, int n_items, const lw_seq_item* items, int batch, const void* in_host,
                                  void* in_dev, int64_t in_bytes, const void* out_dev, void* out_host, int64_t out_bytes,
                                  void* stream) {
    if (!in_host || !in_dev || !out_dev || !out_host) return LW_ERR_NULL;
    if (in_bytes < 0 || out_bytes < 0) return LW_ERR_SHAPE;
    const int rc = check_sequence_batch(fmt, n_items, items, batch);      // a call that fails enqueues nothing
    if (rc != LW_OK) return rc;
    HostPipe pipe(n_items, items, batch, in_host, in_dev, in_bytes, out_dev, out_host, out_bytes, static_cast<cudaStream_t>(stream));
    return run_sequence_batch(fmt, n_items, items, batch, stream, &pipe);
}

int lw_set_sequence_mode(int mode) {
    if (mode < LW_SEQ_AUTO || mode > LW_SEQ_LAUNCHES) return LW_ERR_FORMAT;
    g_sequence_mode.store(mode);
    return LW_OK;
}

int lw_matvec_host(int fmt, const void* W_blocks, int64_t rows, int64_t cols, const float* X_host,
                   float* Y_host, float* X_dev, float* Y_dev, int batch, void* stream) {
    if (!X_host || !Y_host) return LW_ERR_NULL;
    const int rc = check_matvec_args(fmt, W_blocks, rows, cols, X_dev, Y_dev, batch);
    if (rc != LW_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(X_dev, X_host, sizeof(float) * (size_t)batch * (size_t)cols,
                        cudaMemcpyHostToDevice, s) != cudaSuccess) return LW_ERR_CUDA;
    const int mv = lw_matvec(fmt, W_blocks, rows, cols, X_dev, Y_dev, batch, stream);
    if (mv != LW_OK) return mv;
    if (cudaMemcpyAsync(Y_host, Y_dev, sizeof(float) * (size_t)batch * (size_t)rows,
                        cudaMemcpyDeviceToHost, s) != cudaSuccess) return LW_ERR_CUDA;
    return LW_OK;
}

int lw_set_variant(int variant) {
    if (variant < LW_VARIANT_AUTO || variant > LW_VARIANT_MMA) return LW_ERR_FORMAT;
    g_variant.store(variant);
    return LW_OK;
}

int lw_query_variant(int fmt, int64_t rows, int64_t cols, int batch) {
    if (lw_block_elems(fmt) == 0) return LW_ERR_FORMAT;
    if (rows < 1 || lw_row_bytes(fmt, cols) == 0) return LW_ERR_SHAPE;
    if (batch < 1 || batch > 16) return LW_ERR_BATCH;
    return pick_variant(fmt, rows, cols, batch);
}

int lw_set_tuning(int worker_groups, int stages, int stage_kb) {
    if (worker_groups < 0 || worker_groups > 2 || stages < 0 || stages > 4 || stage_kb < 0 || stage_kb > 96)
        return LW_ERR_FORMAT;
    set_stream_tuning(worker_groups, stages, stage_kb);
    return LW_OK;
}

int lw_set_shape_tuning(int fmt, int64_t rows, int64_t cols, int worker_groups, int stages, int stage_kb) {
    if (lw_block_elems(fmt) == 0) return LW_ERR_FORMAT;
    if (rows < 1 || lw_row_bytes(fmt, cols) == 0) return LW_ERR_SHAPE;
    if (worker_groups < 0 || worker_groups > 2 || stages < 0 || stages > 4 || stage_kb < 0 || stage_kb > 96)
        return LW_ERR_FORMAT;
    set_shape_tuning(fmt, rows, cols, worker_groups, stages, stage_kb);
    return LW_OK;
}

int lw_clear_shape_tuning(void) {
    clear_shape_tuning();
    return LW_OK;
}

int lw_plan_info(int fmt, int64_t rows, int64_t cols, int* out6) {
    if (lw_block_elems(fmt) == 0) return LW_ERR_FORMAT;
    if (!out6) return LW_ERR_NULL;
    if (rows < 1 || lw_row_bytes(fmt, cols) == 0) return LW_ERR_SHAPE;
    if (!stream_plan_info(fmt, rows, cols, &out6[0], &out6[1], &out6[2], &out6[3], &out6[4], &out6[5])) {
        for (int i = 0; i < 6; ++i) out6[i] = 0;       // shape not covered by the streaming kernels
    }
    return LW_OK;
}

int lw_probe_read(const void* src, int64_t bytes, void* stream) {
    if (!src) return LW_ERR_NULL;
    if (bytes < 16 || bytes % 16 != 0) return LW_ERR_SHAPE;
    if (misaligned16(src)) return LW_ERR_ALIGN;
    return launch_probe_read(src, bytes, static_cast<cudaStream_t>(stream)) == 0 ? LW_OK : LW_ERR_CUDA;
}

int lw_debug_drop_copy(int unit) {
    set_drop_unit(unit);
    return LW_OK;
}

int lw_set_overlap(int enabled) {
    if (enabled < 0 || enabled > 2) return LW_ERR_FORMAT;
    g_overlap.store(enabled);
    return LW_OK;
}

int lw_set_attn_variant(int variant) {
    if (variant != 0 && variant != 1) return LW_ERR_FORMAT;
    set_attn_variant(variant);
    return LW_OK;
}

int lw_query_attn_variant(int kv_fmt, int64_t n_head, int64_t n_kv_head, int64_t head_dim, int64_t n_pos) {
    if (kv_fmt != LW_F16 && kv_fmt != LW_Q8_0 && kv_fmt != LW_Q4_0) return LW_ERR_FORMAT;
    if (!attn_shape_supported(kv_fmt, n_head, n_kv_head, head_dim, n_pos)) return LW_ERR_SHAPE;
    return attn_variant_of(kv_fmt, n_head, n_kv_head, head_dim, n_pos);
}

int64_t lw_attn_workspace_bytes(int64_t n_head, int64_t n_kv_head, int64_t head_dim, int64_t n_pos) {
    if (!attn_shape_supported(LW_F16, n_head, n_kv_head, head_dim, n_pos)) return 0;
    return attn_workspace_bytes(n_head, n_kv_head, head_dim, n_pos);
}

int lw_attn_decode(int kv_fmt, const void* K_blocks, const void* V_blocks, const float* q, float* out, int64_t n_head,
                   int64_t n_kv_head, int64_t head_dim, int64_t n_pos, float scale, void* workspace,
                   int64_t workspace_bytes, void* stream) {
    if (kv_fmt != LW_F16 && kv_fmt != LW_Q8_0 && kv_fmt != LW_Q4_0) return LW_ERR_FORMAT;
    if (!attn_shape_supported(kv_fmt, n_head, n_kv_head, head_dim, n_pos) || !std::isfinite(scale)) return LW_ERR_SHAPE;
    if (!K_blocks || !V_blocks || !q || !out || !workspace) return LW_ERR_NULL;
    if (misaligned16(K_blocks) || misaligned16(V_blocks) || misaligned16(q) || misaligned16(out) || misaligned16(workspace))
        return LW_ERR_ALIGN;
    if (workspace_bytes < attn_workspace_bytes(n_head, n_kv_head, head_dim, n_pos)) return LW_ERR_WORKSPACE;
    return launch_attn_decode(kv_fmt, K_blocks, V_blocks, q, out, n_head, n_kv_head, head_dim, n_pos, scale, workspace,
                              static_cast<cudaStream_t>(stream)) == 0 ? LW_OK : LW_ERR_CUDA;
}

int lw_device_status(int* status_out) {
    if (!status_out) return LW_ERR_NULL;
    int* word = device_fault_word();
    if (!word) return LW_ERR_CUDA;
    if (cudaDeviceSynchronize() != cudaSuccess) return LW_ERR_CUDA;
    int value = 0;
    if (cudaMemcpy(&value, word, sizeof value, cudaMemcpyDeviceToHost) != cudaSuccess) return LW_ERR_CUDA;
    if (value != 0 && cudaMemset(word, 0, sizeof value) != cudaSuccess) return LW_ERR_CUDA;
    *status_out = value;
    return LW_OK;
}

}  // extern "C"
