// Internal declarations shared by the translation units of the lw library.
#ifndef LW_INTERNAL_H_
#define LW_INTERNAL_H_

#include <cstddef>
#include <cstdint>

#include "lw.h"

namespace lw {

// Device-side fault codes recorded in the status word (see lw_device_status).
enum DeviceFault : int {
    FAULT_NONE = 0,
    FAULT_BULK_WAIT_TIMEOUT = 1,   // a bounded wait on a bulk-copy barrier gave up
    FAULT_DRAIN_TIMEOUT = 2,       // the end-of-kernel drain of copies in flight gave up
    FAULT_GRID_BARRIER_TIMEOUT = 3 // a CTA of the sequence kernel gave up waiting for the other CTAs
};

int quantize_host(int fmt, const float* src, int64_t n, void* dst);

#ifdef __CUDACC__
// Each returns a cudaError_t cast to int (0 = success); arguments are already validated.
int launch_dequant(int fmt, const void* W, int64_t n, float* out, cudaStream_t stream);
int launch_matvec_generic(int fmt, const void* W, int64_t rows, int64_t cols, const float* X,
                          float* Y, int batch, cudaStream_t stream);
// Streaming variant: `supported` tells whether the shape qualifies.
bool matvec_stream_supported(int fmt, int64_t rows, int64_t cols, int batch);
// integer_dot selects the dp4a family (ignored for f16, which has none).
int launch_matvec_stream(int fmt, bool integer_dot, const void* W, int64_t rows, int64_t cols, const float* X,
                         float* Y, bool overlap, cudaStream_t stream);
// Batched (2..16 columns) integer-dot streaming kernel; Y[b*rows + r] strides by `rows`.
int launch_matvec_stream_batched(int fmt, const void* W, int64_t rows, int64_t cols, const float* X, float* Y,
                                 int batch, bool overlap, cudaStream_t stream);
// Grouped launch: n_items independent matrices of one format and width in one grid (batch 1).
bool matvec_group_supported(int fmt, int64_t cols, int n_items);
int launch_matvec_stream_group(int fmt, bool integer_dot, int64_t cols, int n_items, const void* const* W,
                               const int64_t* rows, const float* const* X, float* const* Y, bool overlap,
                               cudaStream_t stream);
// Sequence of batch-1 mat-vecs in one persistent launch (grid-wide barrier before dependent items).
// `counter` is a device word owned by the caller (cleared on the stream by the launch).
bool matvec_sequence_supported(int fmt, int n_items, const lw_seq_item* items);
int launch_matvec_sequence(int fmt, int n_items, const lw_seq_item* items, unsigned* counter, cudaStream_t stream);
// Read-only streaming probe over `bytes` bytes (a multiple of 16) at `src`.
int launch_probe_read(const void* src, int64_t bytes, cudaStream_t stream);
// Batched fp32 tile kernel (2..16 columns, every decoded weight used for all columns of a pass): q8_0 and
// q4_0, cols a multiple of 1024.
bool matvec_tile_supported(int fmt, int64_t rows, int64_t cols, int batch);
int launch_matvec_tile(int fmt, const void* W, int64_t rows, int64_t cols, const float* X, float* Y, int batch,
                       cudaStream_t stream);
// Batched tensor-core kernel (2..16 columns; weights as exact bf16 codes, activations as three bf16 terms, fp32
// accumulation; f16: f16 operands): every format, cols a multiple of 256 (q6_K: of 2048, q2_K: of 1024).  The launch clears Y first (the kernel adds into it).
bool matvec_mma_supported(int fmt, int64_t rows, int64_t cols, int batch);
int launch_matvec_mma(int fmt, const void* W, int64_t rows, int64_t cols, const float* X, float* Y, int batch,
                      int overlap, bool self_clear, cudaStream_t stream);
// The same for up to eight matrices of one format and width in one launch (each with its own X and Y).
bool matvec_mma_group_supported(int fmt, int64_t cols, int n_items, const int64_t* rows, int batch);
// pre_cleared: the launch before on the stream cleared these outputs; next_*: outputs of the launch after, to be
// cleared by this one at its end (n_next = 0: none).
int launch_matvec_mma_group(int fmt, int64_t cols, int n_items, const void* const* W, const int64_t* rows,
                            const float* const* X, float* const* Y, int batch, int overlap, bool self_clear,
                            cudaStream_t stream, bool pre_cleared, int n_next, float* const* next_y,
                            const int64_t* next_n);
// Tunables of the streaming kernels (0 = automatic) and the geometry they lead to for a shape.
void set_stream_tuning(int worker_groups, int stages, int stage_kb);
// Per-shape tunables (all zero erases the entry); make_plan uses them where the process-wide ones are 0.
void set_shape_tuning(int fmt, int64_t rows, int64_t cols, int worker_groups, int stages, int stage_kb);
void clear_shape_tuning();
// Testing aid: the next single-matrix streaming launch never requests the copy of pool unit `unit` (< 0: none).
void set_drop_unit(int unit);
int take_drop_unit();     // the pending request (-1: none), consumed
bool stream_plan_info(int fmt, int64_t rows, int64_t cols, int* groups, int* stages, int* stage_rows, int* stage_bytes,
                      int* grid, int* smem_bytes);
// Decode attention over a quantised KV cache: shape check, parts the positions are cut into, bytes of
// workspace that is always enough, launch (arguments already validated; returns a cudaError_t as int).
bool attn_shape_supported(int fmt, int64_t n_head, int64_t n_kv_head, int64_t head_dim, int64_t n_pos);
int attn_parts(int64_t n_head, int64_t n_kv_head, int64_t head_dim, int64_t n_pos);
int64_t attn_workspace_bytes(int64_t n_head, int64_t n_kv_head, int64_t head_dim, int64_t n_pos);
int launch_attn_decode(int fmt, const void* K, const void* V, const float* q, float* out, int64_t n_head,
                       int64_t n_kv_head, int64_t head_dim, int64_t n_pos, float scale, void* workspace,
                       cudaStream_t stream);
// Kernel choice of the attention: 0 automatic, 1 general kernel only; and what a shape gets (1 general, 2 tensor-core).
void set_attn_variant(int variant);
int attn_variant_of(int fmt, int64_t n_head, int64_t n_kv_head, int64_t head_dim, int64_t n_pos);
// Address of the per-device fault word (device memory), or nullptr on error.
int* device_fault_word();

// Host <-> device copies of a chain's input and result blocks, in pieces that overlap with the chain's kernels
// (lw_hostpipe.cu).  The chain code calls begin() first, before(j, n) ahead of the launch that runs items
// j .. j+n-1, after(j, n) behind it, and end() last; every call returns false on a CUDA error.
class HostPipe {
public:
    HostPipe(int n_items, const lw_seq_item* items, int batch, const void* in_host, void* in_dev, int64_t in_bytes,
             const void* out_dev, void* out_host, int64_t out_bytes, cudaStream_t stream);
    ~HostPipe();
    HostPipe(const HostPipe&) = delete;
    HostPipe& operator=(const HostPipe&) = delete;
    void whole_copies_only();      // one copy in before the first kernel, one copy out behind the last (call before begin)
    bool begin();
    bool before(int j, int n);     // the caller's stream waits for the input pieces these items read
    bool after(int j, int n);      // result pieces that no later item writes may leave
    bool end();                    // the rest of both blocks; the caller's stream waits for all copies
private:
    struct State;
    cudaEvent_t event();
    bool copy_in(int64_t upto);
    bool copy_out(int64_t upto);
    const char* in_host_;
    char* in_dev_;
    int64_t in_bytes_;
    const char* out_dev_;
    char* out_host_;
    int64_t out_bytes_;
    cudaStream_t s_;
    State* st_;
};
#endif

}  // namespace lw
#endif
