/* lw.h -- C ABI of the B200 fused dequantize + matrix-vector library.
 *
 * One hot path: the decode-phase product y = W x where W is stored in a block-quantised weight
 * format and is decoded in registers while it streams from HBM [paper Sec 3.2, the
 * decode-phase mat-vec kernel of the matrix-multiplication paragraph; Sec 3.3, weights decoded in registers].
 *
 * Formats [Sec 2.2]: f16; the "basic" symmetric 32-weight blocks q8_0 and q4_0; the K-quants q4_K
 * (256-weight super-block, eight 32-weight sub-blocks with 6-bit scale/min pairs quantised against
 * fp16 super-block factors) and q6_K (sixteen 16-weight sub-blocks with int8 scales against one fp16
 * factor).  Byte layouts are the public ggml ones:
 *   f16 : little-endian IEEE binary16 per weight
 *   q8_0: 34 bytes = fp16 d, 32 x int8 q               value = d * q
 *   q4_0: 18 bytes = fp16 d, 16 bytes; byte j = q[j] | q[j+16] << 4   value = d * (q - 8)
 *   q4_K: 144 bytes = fp16 d, fp16 dmin, 12 bytes of packed 6-bit (sc, m) x 8, 128 bytes of nibbles;
 *         byte 32g+l holds weight 64g+l (low nibble, sub-block 2g) and weight 64g+32+l (high
 *         nibble, sub-block 2g+1);                     value = d*sc*q - dmin*m
 *   q4_1: 20 bytes = fp16 d, fp16 m, nibbles as q4_0     value = d * q + m
 *   q5_0: 22 bytes = fp16 d, 4 bytes qh, nibbles         value = d * (q - 16), q = nibble | bit << 4,
 *         bit i of the little-endian 32-bit word qh belonging to weight i
 *   q5_1: 24 bytes = fp16 d, fp16 m, qh, nibbles         value = d * q + m
 *   q2_K: 84 bytes = 16 bytes of (scale | min << 4) pairs (one per run of 16 weights), 64 bytes of 2-bit
 *         codes, fp16 d, fp16 dmin; weight 32j+l (j < 4, l < 32) of half h (128 weights) sits in bits
 *         2j, 2j+1 of code byte 32h + l and uses pair 8h + 2j + l/16;   value = d*scale*q - dmin*min
 *   q5_K: 176 bytes = fp16 d, fp16 dmin, the 12 packed (sc, m) bytes of q4_K, 32 bytes qh, 128 bytes of
 *         nibbles; the 5-bit code of weight 64g+l is the low nibble of nibble byte 32g+l | bit 2g of
 *         qh[l] << 4, that of weight 64g+32+l the high nibble | bit 2g+1 of qh[l] << 4;
 *                                                       value = d*sc*q - dmin*m
 *   q6_K: 210 bytes = 128 bytes ql, 64 bytes qh, 16 x int8 scale, fp16 d (256 weights).  Weight 32j+l
 *         (j < 4, l < 32) of half h (128 weights) keeps the low 4 bits of its 6-bit code q in ql byte
 *         64h + l + 32(j mod 2) (low nibble for j < 2, high for j >= 2), the high 2 bits in bits
 *         2j, 2j+1 of qh byte 32h + l, and uses scale 8h + 2j + l/16;   value = d*scale*(q - 32)
 *         [Sec 2.2 K-quants; the first of the further formats the decode-routine design admits,
 *         Sec 3.3].  Streaming (integer-dot) kernel when cols is a multiple of 2048, so that a row
 *         is a whole number of 16-byte pieces; generic kernels otherwise.
 *
 * Conventions for every call:
 *   - "device" pointers are CUDA device addresses on the current device; "host" pointers are
 *     ordinary host memory.  The library never allocates, frees or retains any buffer and never
 *     synchronises the stream unless a call says so.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Device calls
 *     only enqueue work; they can be captured into a CUDA graph.
 *   - Arguments are validated on the host first; a call that returns an error has enqueued nothing.
 *   - Return value: LW_OK (0) or a negative lw_status.  No exceptions, aborts or device traps.
 */
#ifndef LW_H_
#define LW_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { LW_F16 = 0, LW_Q8_0 = 1, LW_Q4_0 = 2, LW_Q4_K = 3, LW_Q6_K = 4, LW_Q5_K = 5, LW_Q2_K = 6,
               LW_Q4_1 = 7, LW_Q5_0 = 8, LW_Q5_1 = 9 } lw_format;

typedef enum {
    LW_OK = 0,
    LW_ERR_FORMAT = -1,    /* unknown lw_format */
    LW_ERR_SHAPE = -2,     /* rows < 1, cols / n not a whole number of blocks (32; 256 for the K-quants) */
    LW_ERR_NULL = -3,      /* a required pointer is NULL */
    LW_ERR_ALIGN = -4,     /* a device pointer is not 16-byte aligned */
    LW_ERR_BATCH = -5,     /* batch outside 1..16 */
    LW_ERR_NONFINITE = -6, /* quantiser input (or a resulting fp16 scale) is Inf/NaN */
    LW_ERR_CUDA = -7,      /* the CUDA runtime reported an error (no device, launch failure, ...) */
    LW_ERR_DEVICE = -8,    /* a kernel recorded a device-side fault (bounded wait gave up) */
    LW_ERR_WORKSPACE = -9  /* workspace_bytes below what lw_attn_workspace_bytes returns, or a shape beyond
                              the built-in scratch of lw_attn_decode_static */
} lw_status;

/* Weights per block: 1 (f16), 32, 32, 256, 256, 256, 256, 32, 32, 32.  0 for an unknown format. */
size_t lw_block_elems(int fmt);
/* Bytes per block: 2, 34, 18, 144, 210, 176, 84, 20, 22, 24.  0 for an unknown format. */
size_t lw_block_bytes(int fmt);
/* Bytes of one row of `cols` weights; 0 if cols is not a positive multiple of 32 (256 for the K-quants). */
size_t lw_row_bytes(int fmt, int64_t cols);
/* Static description of a status code. */
const char* lw_status_string(int status);

/* Host-side quantiser [Eq. 1: q = round((x - mu)/s), x^ = s*q + mu, scale from the block's range].
 *   q8_0: d = amax/127, q = roundf(x/d);   q4_0: d = (signed extreme)/-8, q = min(15,(int)(x/d+8.5));
 *   q4_K: per sub-block offset -min(0, min x) and step (range)/15, both rounded to 6 bits against
 *         fp16 d = max step/63 and dmin = max offset/63 (a deterministic min/max rule);
 *   q4_1 / q5_1: d = (max - min)/(15 or 31), m = min, q = min(top, (int)((x - min)/d + 0.5));
 *   q5_0: d = (signed extreme)/-16, q = min(31, (int)(x/d + 16.5));
 *   q5_K: the q4_K rule with step (range)/31 and 5-bit codes;
 *   q2_K: the same rule on runs of 16 with step (range)/3, rounded to 4 bits against d = max step/15
 *         and dmin = max offset/15;
 *   q6_K: per run of 16 a step (signed extreme)/-32, rounded to int8 against fp16 d = max|step|/127;
 *         q = clamp(round(x/(d*scale)) + 32, 0, 63) (a deterministic rule of this library);
 *   f16 : round to nearest even.
 * src: host, n floats.  dst: host, lw_row_bytes(fmt, n) bytes, fully overwritten.  n must be a
 * whole number of blocks.  Pure CPU code: makes no CUDA call.  Single-threaded; callers may run
 * disjoint ranges from several threads. */
int lw_quantize(int fmt, const float* src, int64_t n, void* dst);

/* Stand-alone dequantisation [Sec 3.3 decode routines]: out[i] = decode(W_blocks)[i] as fp32,
 * bit-exact IEEE results (the products are exact; q4_K's final subtraction rounds once).
 * W_blocks: device, lw_row_bytes(fmt, n) bytes, 16-byte aligned, read-only.
 * out: device, n floats, 16-byte aligned, fully overwritten.  Asynchronous on `stream`. */
int lw_dequant(int fmt, const void* W_blocks, int64_t n, float* out, void* stream);

/* Fused dequantise + mat-vec [Sec 3.2, 3.3]: Y[b*rows + r] = sum_k decode(W)[r][k] * X[b*cols + k],
 * fp32 accumulation, for b < batch (1..16).  The batched kernels reuse every decoded block for all
 * their columns: without a forced variant every format, with cols a multiple of 256 (q6_K: of 2048,
 * q2_K: of 1024), runs on the tensor cores from three columns on (LW_VARIANT_MMA); two columns, and other
 * widths of the streaming shapes, run one streaming pass per column instead (four columns per launch), which
 * measures faster on B200 than the older batched kernels.
 * W_blocks: device, rows * lw_row_bytes(fmt, cols) bytes, row-major without padding, 16-byte
 *           aligned, read-only.
 * X: device, batch * cols floats, each activation vector contiguous, 16-byte aligned, read-only.
 * Y: device, batch * rows floats, 16-byte aligned, fully overwritten (never accumulated into).
 * Asynchronous on `stream`.
 * Accuracy.  With w the decoded weights and S = sum_k |w_k x_k|, every result satisfies
 *     |y - y_exact| <= 1e-4 * S + 1e-6 + E .
 * E = 0 for LW_VARIANT_GENERIC and for f16 at batch 1 and 2 (each weight is decoded exactly and then multiplied:
 * plain fp32 accumulation), for any finite input, and for the batched LW_VARIANT_TILE and LW_VARIANT_MMA on
 * q8_0, q4_0, q5_0 and q6_K (exact integer codes times the activations -- exact in TILE, to 2^-16 of each one's
 * own magnitude in MMA -- and block sums scaled in fp32) as long as |x| <= 2^115, which keeps a block's sum of
 * code * x finite.  The streaming variants multiply the integer codes first and apply
 * block scales and offsets to the sums, and LW_VARIANT_IDOT holds the activations as block fixed point
 * (23 bits + sign relative to the largest magnitude in each run of 16 or 32), so an activation that is
 * huge compared with its neighbours and meets a weight that is zero or nearly so leaves an absolute error
 * that S does not cover.  For them
 *     E = c * sum_k What_k * A_k ,   c = 2^-18 (IDOT, the default for the quantised formats; MMA on q4_K, q5_K, q2_K,
 *                                    q4_1 and q5_1), 2^-16 (STREAM), 2^-30 (MMA on f16: activations as two f16
 *                                    terms relative to their block's largest),
 * where, over the aligned run of 32 columns that contains k, A_k is the largest |x| and What_k the largest
 * decoded |w|.  This holds for weights made by lw_quantize, and for any block whose scale * code and offset
 * terms are at most four times its largest decoded magnitude.  The constants are worst-case figures (the
 * largest c observed on inputs built to provoke the term is 2^-26 for IDOT and 2^-22 for STREAM); on
 * Gaussian activations and weights the measured error stays below 0.001 of 1e-4 * S.
 * A NaN or Inf activation makes every output of its column's rows non-finite in every variant. */
int lw_matvec(int fmt, const void* W_blocks, int64_t rows, int64_t cols,
              const float* X, float* Y, int batch, void* stream);

/* Same product with HOST activations and results: copies X_host -> X_dev, runs lw_matvec, copies
 * Y_dev -> Y_host, all asynchronously on `stream` (pinned host memory makes the copies truly
 * asynchronous).  X_dev / Y_dev are caller-provided device staging buffers of batch*cols and
 * batch*rows floats.  The caller synchronises the stream before reading Y_host. */
int lw_matvec_host(int fmt, const void* W_blocks, int64_t rows, int64_t cols,
                   const float* X_host, float* Y_host, float* X_dev, float* Y_dev,
                   int batch, void* stream);

/* Several independent mat-vecs of one format and one width in a single launch, batch 1 [Sec 3.1,
 * 3.2: the runtime groups operations into compute passes to cut submission and synchronisation
 * cost].  Typical groups are the q/k/v projections and the gate/up projections of a layer, which
 * read the same activations and do not depend on each other.  Each item is what lw_matvec takes:
 * W (device, rows * lw_row_bytes(fmt, cols) bytes), X (device, cols floats), Y (device, rows floats),
 * all 16-byte aligned; items must not overlap in Y.  1 <= n_items <= 8.  When the shape is not
 * covered by the streaming kernels the items are run one after the other with lw_matvec.
 * `items` is host memory, read during the call only. */
typedef struct {
    const void* W_blocks;
    int64_t rows;
    const float* X;
    float* Y;
} lw_group_item;
int lw_matvec_group(int fmt, int64_t cols, int n_items, const lw_group_item* items, void* stream);

/* The same with `batch` activation columns per item (1..16): X of an item is batch * cols floats, Y batch * rows
 * floats, laid out as in lw_matvec.  batch 1 is lw_matvec_group.  From two columns on, every format with cols a
 * multiple of 256 run all items in ONE launch of the tensor-core kernel (LW_VARIANT_MMA, unless another variant
 * is forced; items that follow one another and share their X pointer share its converted copy); everything else
 * is run item by item with lw_matvec.  Errors as lw_matvec (LW_ERR_BATCH for batch outside 1..16); a call that
 * fails validation enqueues nothing. */
int lw_matvec_group_batch(int fmt, int64_t cols, int n_items, const lw_group_item* items, int batch, void* stream);

/* A whole chain of batch-1 mat-vecs of one format in ONE call [Sec 3.1, 3.2: the runtime groups operations
 * into compute passes; the whole mat-vec chain of a decode step is one pass here].  The items run in the
 * order given.  Consecutive items that read the same X (same pointer, same cols) and are not flagged
 * dependent form one phase whose rows are shared out over all SMs together (q/k/v, gate/up).  An item
 * flagged LW_SEQ_DEPENDENT reads (X) or overwrites (Y) memory that an earlier item of the sequence writes
 * or reads: before it starts, every earlier item has finished device-wide.  Without the flag an item may
 * run concurrently with its predecessors.  Two implementations (lw_set_sequence_mode):
 *   LW_SEQ_LAUNCHES   one grouped launch per phase, chained with programmatic dependent launch (a kernel's
 *                     CTAs are placed and set up while its predecessor finishes and wait for it before they
 *                     touch W or X); the default (LW_SEQ_AUTO) because it measures faster on B200;
 *   LW_SEQ_PERSISTENT one persistent kernel, one CTA per SM, launched cooperatively, with a grid-wide barrier
 *                     before each dependent item; the weight ring keeps filling across item boundaries
 *                     (weights are constant data), so a boundary costs a barrier and the activation fetch
 *                     instead of a launch with a cold pipeline.
 * Each item is what lw_matvec takes at batch 1 (W: rows * lw_row_bytes(fmt, cols) bytes; X: cols floats;
 * Y: rows floats; all device, 16-byte aligned); n_items <= 640, at most 320 phases.
 * workspace: device, at least lw_matvec_sequence_workspace_bytes() bytes, 16-byte aligned, owned by the
 *           caller, need not be initialised (the call clears what it needs on `stream` first); sequences that
 *           may run concurrently need separate workspaces.
 * `items` is host memory, read during the call only.  Results and accuracy are those of lw_matvec.
 * When a shape is not covered by the streaming kernels or a variant is forced, the items are issued one
 * after the other with lw_matvec on `stream` (stream order then provides every dependency); a device that
 * cannot launch cooperatively gets LW_SEQ_LAUNCHES.  Asynchronous on `stream`; can be captured into a CUDA graph.
 * Errors: as lw_matvec per item, LW_ERR_SHAPE for n_items outside 1..640, LW_ERR_WORKSPACE. */
typedef struct {
    const void* W_blocks;
    int64_t rows;
    int64_t cols;
    const float* X;
    float* Y;
    int flags;              /* 0 or LW_SEQ_DEPENDENT */
} lw_seq_item;
enum { LW_SEQ_DEPENDENT = 1 };
int64_t lw_matvec_sequence_workspace_bytes(void);
int lw_matvec_sequence(int fmt, int n_items, const lw_seq_item* items, void* workspace, int64_t workspace_bytes,
                       void* stream);
typedef enum { LW_SEQ_AUTO = 0, LW_SEQ_PERSISTENT = 1, LW_SEQ_LAUNCHES = 2 } lw_sequence_mode;
/* Process-wide choice of the implementation behind lw_matvec_sequence; LW_ERR_FORMAT for another value. */
int lw_set_sequence_mode(int mode);

/* lw_matvec_sequence with HOST activations and results: copies in_bytes from in_host to in_dev (the block that
 * holds the chain's input activations; the items' X pointers point into in_dev), runs the chain, copies out_bytes
 * from out_dev to out_host (the block the items' Y pointers point into).  In stream order the call is one
 * operation on `stream`: it starts after everything enqueued before it and `stream` has finished it when both
 * blocks are complete; it is asynchronous (pinned host memory makes the copies truly asynchronous) and can be
 * captured into a CUDA graph.  The result is that of one copy in, the chain, one copy out.  Blocks above 128 KB
 * move in pieces on two copy streams of the library beside the kernels (LW_SEQ_LAUNCHES only): the input block in
 * address order, a launch waiting only for the pieces up to the end of the activations it reads; a piece of the
 * result block as soon as no later item writes into it.  Activations and results laid out in the order of the
 * items overlap best; any layout is correct.  When an item writes into the input block, that block is copied
 * whole before the first kernel.  in_host must not change and out_host must not be read until the stream has
 * finished the call.  in_dev / out_dev are caller-provided device buffers; a size of 0 skips that copy.
 * The library creates its copy streams and events at the first call that needs them (per device, and one more set
 * per call that runs concurrently or per stream capture that is open at the same time) and keeps them; calls
 * from several host threads, captured or not, do not disturb one another.
 * Errors as lw_matvec_sequence; a call that fails validation enqueues nothing. */
int lw_matvec_sequence_host(int fmt, int n_items, const lw_seq_item* items, const void* in_host, void* in_dev,
                            int64_t in_bytes, const void* out_dev, void* out_host, int64_t out_bytes, void* workspace,
                            int64_t workspace_bytes, void* stream);

/* The chain with `batch` activation columns per item (1..16): X of an item is batch * cols floats, Y batch * rows,
 * laid out as in lw_matvec.  Runs of consecutive items that share their X pointer and width and are not flagged
 * LW_SEQ_DEPENDENT go into one lw_matvec_group_batch call each (one launch of the tensor-core kernel where it
 * applies); stream order provides every dependency.  Under lw_set_overlap a launch of that kernel also clears the
 * outputs of the launch after it where they overlap nothing it reads or writes (checked on the host), which saves the
 * clearing kernel in between.  No workspace.  Errors as lw_matvec_sequence, LW_ERR_BATCH for
 * batch outside 1..16; a call that fails validation enqueues nothing. */
int lw_matvec_sequence_batch(int fmt, int n_items, const lw_seq_item* items, int batch, void* stream);

/* The same with the step's inputs and results in HOST memory, as lw_matvec_sequence_host (blocks above 128 KB move
 * in pieces beside the kernels; same rules). */
int lw_matvec_sequence_batch_host(int fmt, int n_items, const lw_seq_item* items, int batch, const void* in_host,
                                  void* in_dev, int64_t in_bytes, const void* out_dev, void* out_host, int64_t out_bytes,
                                  void* stream);

/* Kernel-variant selection [Sec 3.2: the kernel library picks a variant from the tensor context;
 * tunable work-group and tile sizes].  LW_VARIANT_AUTO lets the launch heuristics decide. */
typedef enum {
    LW_VARIANT_AUTO = 0,
    LW_VARIANT_GENERIC = 1, /* one warp per row, plain loads; any legal shape and batch */
    LW_VARIANT_STREAM = 2,  /* bulk-copy ring into shared memory, fp32 activations held in registers, one
                               512-thread CTA per SM; needs cols % 256 == 0, cols <= 16384 and rows that are
                               whole 16-byte pieces; batch 1.  Exists for f16, q8_0, q4_0 and q4_K; forced on
                               one of the six later formats it falls back to LW_VARIANT_GENERIC */
    LW_VARIANT_IDOT = 3,    /* same streaming skeleton, but activations are converted once per call to
                               24-bit block fixed point (one fp32 scale per 16 or 32 values) and the
                               products run as exact integer dot products (dp4a); error per
                               activation <= 2^-22 of its group's largest magnitude (see the accuracy
                               statement of lw_matvec).  All nine quantised formats (f16 falls back to
                               LW_VARIANT_STREAM).  q8_0, q4_0 and q4_K also have a batched form (2..16
                               columns, fixed-point activations kept in shared memory) */
    LW_VARIANT_TILE = 4,    /* batch 2..16 only: fp32 tile kernel, a lane owns rows, every weight is decoded once
                               (exactly) and multiplied with all columns of a pass (up to 8) by packed fp32 FMAs,
                               activations read from shared memory by broadcast; q8_0 and q4_0, cols a multiple
                               of 1024.  E = 0 in the accuracy statement of lw_matvec; a row's sum is completed
                               with atomic additions (one per 1024 columns), so the last bits of a result can
                               differ from run to run.  Not chosen by AUTO (LW_VARIANT_MMA covers its shapes and
                               is faster); forced, it runs passes of 8 and 4 columns */
    LW_VARIANT_MMA = 5      /* batch 2..16 only: tensor-core kernel (mma m16n8k16, bf16 operands, fp32 accumulation).
                               A weight's integer code is exact in bf16 and the block scale is applied in fp32 to each
                               block's sum; every fp32 activation is cut into two bf16 terms that add up to it within
                               2^-16 of its magnitude (an error that scales with |w x| term by term and stays at
                               0.15 of the tolerance at worst), so E = 0 in the accuracy statement of lw_matvec for
                               q8_0, q4_0, q5_0 and q6_K (cols a multiple of 2048).  q4_K, q5_K, q2_K (cols a multiple of 1024), q4_1 and q5_1 as well: there the codes are
                               multiplied the same way, and the sub-block offsets
                               (dmin * m) are applied to fp32 sums of each sub-block's activations, which brings the
                               extra term E back with c = 2^-18.  cols a multiple of 256; all columns in one pass
                               over the weights.  f16 as well: the weights are the A operand as they lie in
                               memory, the activations two f16 terms of x * s with s a power of two per block of
                               32 and column (E with c = 2^-30).  A row's sum is completed
                               with atomic additions (one per chunk of up to 1024 columns), so the last bits of a
                               result can differ from run to run.  AUTO takes it from 3 columns on */
} lw_variant;
/* Process-wide; returns LW_ERR_FORMAT for an unknown value.  Also settable once at load time
 * through the environment variable LW_FORCE_VARIANT (a number).  A forced variant that does not
 * support the problem (shape, batch, format) falls back to the next simpler one.  AUTO picks, when
 * the shape qualifies: IDOT for the quantised formats (batch 3..16: MMA where it applies,
 * else IDOT's batch-1 kernel once per column), STREAM for f16 up to batch 4 (likewise); otherwise GENERIC. */
int lw_set_variant(int variant);
/* The variant lw_matvec would launch for this problem (after forcing and shape checks), or a
 * negative lw_status. */
int lw_query_variant(int fmt, int64_t rows, int64_t cols, int batch);

/* Tunable work-group and tile sizes of the streaming kernels [Sec 3.2: the kernels expose their
 * work-group and tile sizes as tunables; Sec 3.1: empirical tuning].  worker_groups: 1 = two 256-thread
 * CTAs per SM, 2 = one 512-thread CTA of two worker groups per SM; stages: ring slots per group (2..4);
 * stage_kb: target size of a ring slot in KB.  0 leaves a parameter to the launch heuristics.
 * Process-wide, meant to be changed between launches (a sweep: python -m paper_2605_20706_b200.autotune);
 * the environment variables LW_WORKER_GROUPS, LW_STAGES, LW_STAGE_KB give the initial values.
 * Returns LW_ERR_FORMAT for values outside 0..2, 0..4, 0..96. */
int lw_set_tuning(int worker_groups, int stages, int stage_kb);
/* The same tunables for ONE shape [Sec 3.2: the kernel library selects a tuned variant from the tensor context;
 * Sec 3.1: the tuning table comes from an empirical sweep].  The launch heuristics consult these entries for
 * every parameter that lw_set_tuning leaves at 0; a grouped launch or a sequence phase is looked up by the sum
 * of its rows.  The sweep (python -m paper_2605_20706_b200.autotune --table FILE) writes the table,
 * lw.load_tuning_table(FILE) of the Python binding installs it.  All three values 0 removes the entry;
 * lw_clear_shape_tuning removes all.  Process-wide, meant to be changed between launches. */
int lw_set_shape_tuning(int fmt, int64_t rows, int64_t cols, int worker_groups, int stages, int stage_kb);
int lw_clear_shape_tuning(void);

/* What the launch heuristics choose for one batch-1 mat-vec under the current tuning: out6 =
 * {worker groups, ring slots per group, rows per slot, bytes per slot, CTAs, shared memory per CTA};
 * all zero when the shape goes to the generic kernels.  Host only, no CUDA work besides a device
 * query. */
int lw_plan_info(int fmt, int64_t rows, int64_t cols, int* out6);

/* Overlap of consecutive calls on one stream (programmatic dependent launch): when enabled, the
 * launches carry the programmatic-serialisation attribute, so a mat-vec kernel's CTAs may be placed and
 * run their set-up (barrier initialisation, launch latency) while the previous kernel on the stream is
 * still finishing; they wait for that kernel to complete before they request any of W or X or write Y.
 * enabled = 2: the same, and the batched tensor-core kernel (LW_VARIANT_MMA) may start streaming W before
 * the previous kernel has completed -- only for weights that no work still pending on the stream writes
 * (model parameters); X and Y are still not touched before.  Other values: LW_ERR_FORMAT.
 * The batched tensor-core kernel adds into Y, which has to be clear first: with overlap off it is launched
 * cooperatively (one CTA on every SM) and its CTAs clear Y themselves before a grid-wide barrier; with overlap on a
 * small clearing kernel is chained in front of it.
 * Default off (0).  Process-wide. */
int lw_set_overlap(int enabled);

/* Decode attention of ONE query token over a block-quantised KV cache [Sec 3.2 "FlashAttention": the
 * decode variant keeps a running maximum, exponential sum and output accumulator per query row while the
 * cached K/V stream by, and accepts q4_0 / q8_0 caches by dequantising their blocks as they are read;
 * Sec 3.3: the mat-vec decode routines are reused for the cache].  For every query head h, with KV head
 * g = h / (n_head / n_kv_head):
 *     s_t = scale * sum_d q[h][d] * K[t][g][d],  p = softmax_t(s),  out[h][:] = sum_t p_t * V[t][g][:]
 * kv_fmt: LW_F16, LW_Q8_0 or LW_Q4_0.
 * K_blocks, V_blocks: device, position-major caches: n_pos rows of n_kv_head * head_dim values each,
 *           every row block-quantised on its own (lw_row_bytes(kv_fmt, n_kv_head * head_dim) bytes, no
 *           padding), 16-byte aligned, read-only.
 * q: device, n_head * head_dim floats; out: device, n_head * head_dim floats, fully overwritten.
 * n_head a multiple of n_kv_head, n_head <= 1024; head_dim in {32, 64, 128, 256}; n_pos >= 1.
 * workspace: device scratch of at least lw_attn_workspace_bytes(...) bytes, 16-byte aligned, owned by the
 *           caller; its contents are overwritten and need not be initialised; calls that may run
 *           concurrently need separate workspaces.
 * Asynchronous on `stream` (two kernels).  Results satisfy |out - exact| <= 1e-4 * sum_t p_t |V| + 1e-6.
 * Errors: LW_ERR_FORMAT, LW_ERR_SHAPE (also a non-finite scale), LW_ERR_NULL, LW_ERR_ALIGN,
 * LW_ERR_WORKSPACE, LW_ERR_CUDA. */
int lw_attn_decode(int kv_fmt, const void* K_blocks, const void* V_blocks, const float* q, float* out,
                   int64_t n_head, int64_t n_kv_head, int64_t head_dim, int64_t n_pos, float scale,
                   void* workspace, int64_t workspace_bytes, void* stream);

/* Kernel choice of lw_attn_decode.  0 (default): the tensor-core kernel where the shape allows it (head_dim
 * 64 or 128, 1 / 2 / 4 / 8 KV heads, cache rows a multiple of 16 bytes; it reads the cache once per four
 * query heads of a KV head), the general CUDA-core kernel otherwise; 1: the general kernel always.  Process-wide; returns
 * LW_ERR_FORMAT for another value.  lw_query_attn_variant tells what a shape gets under the current
 * setting: 1 = general, 2 = tensor-core (or LW_ERR_FORMAT / LW_ERR_SHAPE); host only apart from a device
 * query. */
int lw_set_attn_variant(int variant);
int lw_query_attn_variant(int kv_fmt, int64_t n_head, int64_t n_kv_head, int64_t head_dim, int64_t n_pos);

/* Bytes of workspace lw_attn_decode needs for a shape (an upper bound over its kernels: 256 partial
 * results of head_dim + 2 floats per query head); 0 for an unsupported shape.  Host only. */
int64_t lw_attn_workspace_bytes(int64_t n_head, int64_t n_kv_head, int64_t head_dim, int64_t n_pos);

/* lw_attn_decode without a workspace argument (the paper has no counterpart: this entry point exists for
 * the integration, not for the method).  It is for callers that cannot obtain device memory at call time:
 * a serving process that handed the whole GPU to its own pool at start-up and has no pool handle where the
 * attention is called, a plug-in whose host forbids cudaMalloc because that call synchronises the device
 * in the middle of a latency-critical decode loop, or firmware-style code that is linked without an
 * allocator at all.  The partial results go to a 16 MiB array that is part of the library's device image
 * (every GPU that loads the library holds it until the process exits), which limits the shape to
 * n_head * (head_dim + 2) <= 16384 (for example 64 heads of 128 or 32 heads of 256); larger shapes return
 * LW_ERR_WORKSPACE and enqueue nothing.  The call allocates and frees nothing.
 * The first call on each device looks the array's device address up (once per device, with that device
 * current); make that first call outside any stream capture.
 * All calls on a device share the one array, which keeps whatever the previous call left there (nothing
 * in it has to start at zero: every partial result is written before it is read).  Two calls that may
 * overlap on the GPU (different streams, or one stream with overlap enabled) race on it; keep them
 * ordered, or use lw_attn_decode with separate workspaces.
 * All other arguments, results and errors are those of lw_attn_decode. */
int lw_attn_decode_static(int kv_fmt, const void* K_blocks, const void* V_blocks, const float* q, float* out,
                          int64_t n_head, int64_t n_kv_head, int64_t head_dim, int64_t n_pos, float scale,
                          void* stream);

/* Reads and clears the device-side fault word of the current device (0 = no fault).  Kernels
 * never trap or spin forever: a bounded wait that gives up records a code here and the kernel
 * finishes.  This call synchronises the device.  Returns LW_OK, LW_ERR_NULL or LW_ERR_CUDA. */
int lw_device_status(int* status_out);

/* Measurement aid (the paper has no counterpart): streams `bytes` bytes at `src` (device, 16-byte aligned, a
 * multiple of 16 bytes) through the copy pipeline of the streaming mat-vec kernels -- one CTA per SM, rings of
 * 1-D bulk copies into shared memory, L2 evict-first -- and does nothing with them.  Timing it gives the
 * read-only bandwidth ceiling of that pipeline on the device.  Asynchronous on `stream`. */
int lw_probe_read(const void* src, int64_t bytes, void* stream);

/* Testing aid for that fault path (the paper has no counterpart).  After lw_debug_drop_copy(u), u >= 0, the
 * next batch-1 lw_matvec of a q4_K matrix that takes the streaming kernel (a separate build of it: the kernels
 * of ordinary calls carry no trace of this aid) never requests the copy of the u-th row unit of each CTA: nothing is in flight for it, the wait for it runs out after its limit (about 0.1 s), the kernel
 * records a fault, requests nothing further and returns; the rows of that unit and of the units after it are
 * left unwritten.  The batched tensor-core kernel has the same aid for q4_0 with up to 8 columns: the launch that
 * consumes the request asks for no copy from each CTA's u-th stage on, the wait for that stage runs out, the fault
 * is recorded and the kernel returns (its results are meaningless).  The request is consumed by the first launch of
 * either kind; u < 0 cancels it.  Always returns LW_OK. */
int lw_debug_drop_copy(int unit);

#ifdef __cplusplus
}
#endif
#endif /* LW_H_ */
