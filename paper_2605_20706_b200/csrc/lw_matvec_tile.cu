// Batched mat-vec (2..16 activation columns) that decodes every weight once and uses it for all the
// columns of a pass [paper Sec 3.2: the mat-vec kernel hands over to a tiled kernel as the number of
// activation columns grows; the benchmark spec asks for batch 1-16 columns reusing each decoded block].
// Plain fp32 FMAs on the CUDA cores, no tensor cores.
//
// From two columns on the path is bound by instruction issue, not by HBM (the weights of a pass after the
// first come from L2), so the kernel is organised around the FMA pipe:
//   * A lane owns ROWS (two of them), not a slice of the columns: the activations a warp needs at any time
//     are the same for all its lanes, so they are fetched from shared memory with broadcast loads (one
//     wavefront per 16 bytes) and a decoded weight pair meets BB columns with BB packed FMAs
//     (fma.rn.f32x2: two FMAs per issue slot, which leaves issue slots for the decode and the loads).
//   * The 16 warps of a CTA split the columns of a chunk of 1024 (one 64-weight unit per warp and row);
//     their partial sums are combined through a small table, in a fixed order.
//   * Weights are decoded exactly ((q - 8) resp. the int8 code as floats, then one multiply by the block
//     scale per block and column), so the accuracy is that of the generic kernels.
//   * Weights reach shared memory with 16-byte cp.async copies into padded rows (a lane reads its own row;
//     the padding spreads a warp's 32 rows over eight banks), double-buffered against the products.
// The work is cut into items of 64 rows x one chunk, numbered chunk-major and shared out evenly over the CTAs
// (one per SM): also a matrix of few rows keeps every SM busy.  An item's sums are added into Y (cleared
// before the launch) with atomic adds, because the other chunks of the same rows may belong to other CTAs;
// the order of those (at most cols / 1024) additions is not fixed, so the last bits of a result can differ
// from run to run.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "lw_internal.h"
#include "lw_stream_common.cuh"

namespace lw {
namespace {

constexpr int kTileThreads = 512;
constexpr int kTileWarps = kTileThreads / 32;
constexpr int kTileRows = 64;                 // rows per stage: two per lane
constexpr int kChunkCols = 64 * kTileWarps;   // 1024: one 64-weight unit per warp

struct TileParams {
    const uint8_t* W;
    const float* X;      // batch columns, each `cols` floats
    float* Y;            // Y[b * rows + r]
    int64_t rows;
    int64_t cols;
    int64_t row_bytes;
    int batch;           // columns of this pass (<= BB)
    int chunk_words;     // 32-bit words of one row's share of a chunk
    int row_stride;      // words between rows of a stage in shared memory (a multiple of four, 20 modulo 32)
    uint32_t x_off, w_off, p_off, y_off;     // byte offsets: activations, weight stages, partial table, row sums
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// Four consecutive floats of shared memory as two packed pairs, loaded straight into 64-bit registers (the
// operand form of the packed FMAs: no moves between the load and the arithmetic).
// `base` is a shared-memory address (32 bits), BYTES a compile-time offset: no address arithmetic per load.
template <int BYTES>
__device__ __forceinline__ void lds_pairs(uint32_t base, f2& lo, f2& hi) {
    asm volatile("ld.shared.v2.b64 {%0, %1}, [%2+%3];" : "=l"(lo), "=l"(hi) : "r"(base), "n"(BYTES));
}
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// One 64-weight unit of a row (two blocks), read from the lane's row in shared memory.  `emit(k, pair0, pair1)`
// receives, for k = 0, 4, 8, ..., 60 in some order, the exactly decoded weights k..k+3 as two packed pairs
// (before the block scale); `scale(blk)` the fp16 block scale of block 0 / 1.
struct TileQ40 {
    static constexpr int kFmt = LW_Q4_0;
    static constexpr int kUnitWords = 9;          // 2 x 18 bytes
    uint32_t w[kUnitWords];
    __device__ __forceinline__ void load(const uint32_t* p) {
#pragma unroll
        for (int i = 0; i < kUnitWords; ++i) w[i] = p[i];
    }
    __device__ __forceinline__ float scale(int blk) const { return blk == 0 ? half_lo_to_float(w[0]) : half_hi_to_float(w[4]); }
    // nibble word i (0..3) of block blk: weights 4i..4i+3 in the low nibbles, 16+4i.. in the high ones
    __device__ __forceinline__ uint32_t nibbles(int blk, int i) const {
        return blk == 0 ? __byte_perm(w[i], w[i + 1], 0x5432u) : w[5 + i];
    }
    // weights of group g of block blk (g = 0..7: k = 4g..4g+3 inside the block) as floats q - 8
    __device__ __forceinline__ void group(int blk, int g, f2& p0, f2& p1) const {
        const uint32_t q = nibbles(blk, g & 3);
        const uint32_t m = (g < 4 ? q : (q >> 4)) & 0x0F0F0F0Fu;
        const f2 bias = pack2(-136.f, -136.f);                       // (128 + q) - 136 = q - 8, exactly
        p0 = add2(pack2u(byte_to_128_plus<0>(m), byte_to_128_plus<1>(m)), bias);
        p1 = add2(pack2u(byte_to_128_plus<2>(m), byte_to_128_plus<3>(m)), bias);
    }
};

struct TileQ80 {
    static constexpr int kFmt = LW_Q8_0;
    static constexpr int kUnitWords = 17;         // 2 x 34 bytes
    uint32_t w[kUnitWords];
    __device__ __forceinline__ void load(const uint32_t* p) {
#pragma unroll
        for (int i = 0; i < kUnitWords; ++i) w[i] = p[i];
    }
    __device__ __forceinline__ float scale(int blk) const { return blk == 0 ? half_lo_to_float(w[0]) : half_hi_to_float(w[8]); }
    __device__ __forceinline__ void group(int blk, int g, f2& p0, f2& p1) const {
        const uint32_t q = (blk == 0 ? __byte_perm(w[g], w[g + 1], 0x5432u) : w[9 + g]) ^ 0x80808080u;   // code + 128
        const f2 bias = pack2(-8388736.f, -8388736.f);               // -(2^23 + 128)
        p0 = add2(pack2u(byte_to_2p23_plus<0>(q), byte_to_2p23_plus<1>(q)), bias);
        p1 = add2(pack2u(byte_to_2p23_plus<2>(q), byte_to_2p23_plus<3>(q)), bias);
    }
};

template <class T, int BB>
__global__ void __launch_bounds__(kTileThreads, 1) matvec_tile_kernel(const TileParams p) {
    extern __shared__ __align__(128) uint8_t smem[];
    float* xs = reinterpret_cast<float*>(smem + p.x_off);            // [BB][kChunkCols]
    uint32_t* wst = reinterpret_cast<uint32_t*>(smem + p.w_off);     // two stages of kTileRows x row_stride words
    float* ptab = reinterpret_cast<float*>(smem + p.p_off);          // [kTileWarps][BB][kTileRows]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // Work items: (chunk c of 1024 columns) x (stage s of 64 rows), numbered chunk-major; a CTA takes a
    // contiguous range of them, so it changes chunk -- and reloads its activations -- at most a few times.
    const int n_stages = (int)((p.rows + kTileRows - 1) / kTileRows);
    const int n_chunks = (int)(p.cols / kChunkCols);
    const int64_t items = (int64_t)n_stages * n_chunks;
    const int64_t first = items * blockIdx.x / gridDim.x, last = items * (blockIdx.x + 1) / gridDim.x;
    const int stride = p.row_stride, chunk_words = p.chunk_words;
    const int stage_words = kTileRows * stride;

    // queues the copies of item `it` into buffer `buf`: word j of row r <- W[64 s + r][chunk c][j]; a warp takes
    // every 16th row, its lanes the words of that row's piece
    auto issue_item = [&](int64_t it, int buf) {
        const int c = (int)(it / n_stages), st = (int)(it - (int64_t)c * n_stages);
        const int64_t r_base = (int64_t)st * kTileRows;
        const int n = (int)(p.rows - r_base < kTileRows ? p.rows - r_base : kTileRows);
        const uint8_t* src0 = p.W + r_base * p.row_bytes + (int64_t)c * chunk_words * 4;
        const uint32_t dst0 = smem_u32(wst + buf * stage_words);
        // 16-byte pieces (a row's share of a chunk is a whole number of them, and so is the padded row in shared
        // memory); measured 5 % faster than 4-byte copies into conflict-free odd-stride rows
        constexpr int kPieces = T::kUnitWords * kTileWarps / 4;
        for (int i = tid; i < n * kPieces; i += kTileThreads) {
            const int r = i / kPieces, j = i - r * kPieces;
            cp_async16(dst0 + 4u * (uint32_t)(r * stride) + 16u * j, src0 + (int64_t)r * p.row_bytes + 16 * j);
        }
        cp_async_commit();
    };

    if (first < last) issue_item(first, 0);
    int cur_chunk = -1;
    for (int64_t it = first; it < last; ++it) {
        const int buf = (int)(it - first) & 1;
        const int c = (int)(it / n_stages), st = (int)(it - (int64_t)c * n_stages);
        if (c != cur_chunk) {
            // this chunk's activations: xs[b][k] = X[b][c * 1024 + k]; columns beyond the batch are zero.  (The
            // barrier that ended the previous item has passed: nobody reads the previous chunk any more.)
            cur_chunk = c;
            for (int i = tid; i < BB * (kChunkCols / 4); i += kTileThreads) {
                const int b = i / (kChunkCols / 4), k4 = i - b * (kChunkCols / 4);
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (b < p.batch) v = __ldg(reinterpret_cast<const float4*>(p.X + (int64_t)b * p.cols + (int64_t)c * kChunkCols) + k4);
                *reinterpret_cast<float4*>(xs + b * kChunkCols + 4 * k4) = v;
            }
        }
        // queue the next item (the buffer it goes to was released by the barrier that ended the previous item)
        if (it + 1 < last) {
            issue_item(it + 1, buf ^ 1);
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();                   // this item's weights and the chunk's activations are in place
        const int64_t r_base = (int64_t)st * kTileRows;
        const int n = (int)(p.rows - r_base < kTileRows ? p.rows - r_base : kTileRows);
        // lane's two rows of the stage, this warp's 64 columns of the chunk
        if (lane < n) {
            f2 y2[2][BB];
#pragma unroll
            for (int rr = 0; rr < 2; ++rr)
#pragma unroll
                for (int b = 0; b < BB; ++b) y2[rr][b] = 0;
            const bool two = lane + 32 < n;
            const uint32_t* base = wst + buf * stage_words + warp * T::kUnitWords;
            T u0, u1;
            u0.load(base + lane * stride);
            u1.load(base + (two ? lane + 32 : lane) * stride);
            const uint32_t xw = smem_u32(xs + warp * 64);
#pragma unroll
            for (int blk = 0; blk < 2; ++blk) {
                f2 acc[2][BB];
#pragma unroll
                for (int g = 0; g < 8; ++g) {
                    f2 a0, a1, b0, b1;
                    u0.group(blk, g, a0, a1);
                    u1.group(blk, g, b0, b1);
                    const uint32_t xk = xw + 4u * (32 * blk + 4 * g);
#pragma unroll
                    for (int b = 0; b < BB; b += 2) {
                        // two columns at a time, so that the two FMAs into one accumulator are four issues apart
                        f2 x01, x23, z01, z23;
                        if (b == 0) {
                            lds_pairs<0>(xk, x01, x23);              // same address in every lane
                            lds_pairs<4 * kChunkCols>(xk, z01, z23);
                        } else if (b == 2) {
                            lds_pairs<8 * kChunkCols>(xk, x01, x23);
                            lds_pairs<12 * kChunkCols>(xk, z01, z23);
                        } else if (b == 4) {
                            lds_pairs<16 * kChunkCols>(xk, x01, x23);
                            lds_pairs<20 * kChunkCols>(xk, z01, z23);
                        } else {
                            lds_pairs<24 * kChunkCols>(xk, x01, x23);
                            lds_pairs<28 * kChunkCols>(xk, z01, z23);
                        }
                        if (g == 0) {              // the block's first products start its sums
                            acc[0][b] = mul2(a0, x01);
                            acc[0][b + 1] = mul2(a0, z01);
                            acc[1][b] = mul2(b0, x01);
                            acc[1][b + 1] = mul2(b0, z01);
                        } else {
                            acc[0][b] = fma2(a0, x01, acc[0][b]);
                            acc[0][b + 1] = fma2(a0, z01, acc[0][b + 1]);
                            acc[1][b] = fma2(b0, x01, acc[1][b]);
                            acc[1][b + 1] = fma2(b0, z01, acc[1][b + 1]);
                        }
                        acc[0][b] = fma2(a1, x23, acc[0][b]);
                        acc[0][b + 1] = fma2(a1, z23, acc[0][b + 1]);
                        acc[1][b] = fma2(b1, x23, acc[1][b]);
                        acc[1][b + 1] = fma2(b1, z23, acc[1][b + 1]);
                    }
                }
                const float d0 = u0.scale(blk), d1 = u1.scale(blk);
                const f2 dd0 = pack2(d0, d0), dd1 = pack2(d1, d1);
#pragma unroll
                for (int b = 0; b < BB; ++b) {
                    y2[0][b] = fma2(dd0, acc[0][b], y2[0][b]);
                    y2[1][b] = fma2(dd1, acc[1][b], y2[1][b]);
                }
            }
            float* pt = ptab + warp * (kTileRows * BB) + lane;         // [warp][column][row]: lanes write consecutive words
#pragma unroll
            for (int b = 0; b < BB; ++b) pt[b * kTileRows] = hsum2(y2[0][b]);
            if (two) {
#pragma unroll
                for (int b = 0; b < BB; ++b) pt[b * kTileRows + 32] = hsum2(y2[1][b]);
            }
        }
        __syncthreads();                   // partial sums of the item are complete; its weight buffer is free
        // fold the 16 warps' partial sums, in warp order, and add the item's share to Y (other chunks of the same
        // rows are added by other items, possibly of other CTAs: Y was cleared before the launch)
        for (int i = tid; i < kTileRows * BB; i += kTileThreads) {
            const int b = i / kTileRows, r = i - b * kTileRows;
            if (b < p.batch && r < n) {
                float s = 0.f;
#pragma unroll
                for (int w = 0; w < kTileWarps; ++w) s += ptab[w * kTileRows * BB + i];
                atomicAdd(p.Y + (int64_t)b * p.rows + r_base + r, s);
            }
        }
    }
}

template <class T, int BB>
int launch_tile(TileParams& p, int grid, size_t smem_bytes, cudaStream_t stream) {
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return (int)e;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        e = cudaFuncSetAttribute(matvec_tile_kernel<T, BB>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return (int)e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    matvec_tile_kernel<T, BB><<<(unsigned)grid, kTileThreads, smem_bytes, stream>>>(p);
    return (int)cudaGetLastError();
}

int tile_sm_count() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
    return n;
}

}  // namespace

bool matvec_tile_supported(int fmt, int64_t rows, int64_t cols, int batch) {
    if (fmt != LW_Q4_0 && fmt != LW_Q8_0) return false;
    if (batch < 2 || batch > 16) return false;
    if (cols % kChunkCols != 0) return false;
    return rows >= 1 && rows <= (int64_t)1 << 30;
}

// Batch 2..16 in passes of up to 8 columns.  Arguments are validated; returns a cudaError_t as int.
int launch_matvec_tile(int fmt, const void* W, int64_t rows, int64_t cols, const float* X, float* Y, int batch,
                       cudaStream_t stream) {
    const int grid = tile_sm_count();
    // the kernel adds every (chunk, stage) item's share into Y
    cudaError_t e = cudaMemsetAsync(Y, 0, sizeof(float) * (size_t)batch * (size_t)rows, stream);
    if (e != cudaSuccess) return (int)e;
    const int unit_words = fmt == LW_Q4_0 ? 9 : 17;
    for (int b0 = 0; b0 < batch;) {
        const int left = batch - b0;
        const int bb = left > 4 ? 8 : 4;
        const int nb = left < bb ? left : bb;
        TileParams p{};
        p.W = static_cast<const uint8_t*>(W);
        p.X = X + (int64_t)b0 * cols;
        p.Y = Y + (int64_t)b0 * rows;
        p.rows = rows;
        p.cols = cols;
        p.row_bytes = (int64_t)lw_row_bytes(fmt, cols);
        p.batch = nb;
        p.chunk_words = unit_words * kTileWarps;
        // rows padded to a multiple of four words (16-byte copies) that is 20 modulo 32: a lane reads its own row,
        // so the 32 rows of a warp spread over eight banks (4-way conflicts on the 18 or 34 unit loads per item,
        // which is cheap next to the products; an odd stride would be conflict-free but forces 4-byte copies)
        p.row_stride = p.chunk_words + ((20 - p.chunk_words % 32) + 32) % 32;
        const size_t x_bytes = (size_t)bb * kChunkCols * 4;
        const size_t w_bytes = 2 * (size_t)kTileRows * p.row_stride * 4;
        const size_t p_bytes = (size_t)kTileWarps * kTileRows * bb * 4;
        p.x_off = 0;
        p.w_off = (uint32_t)x_bytes;
        p.p_off = (uint32_t)((p.w_off + w_bytes + 15) & ~(size_t)15);
        p.y_off = 0;
        const size_t smem_bytes = p.p_off + p_bytes;
        if (smem_bytes > 227 * 1024) return (int)cudaErrorInvalidValue;
        int err;
        if (fmt == LW_Q4_0) err = bb == 8 ? launch_tile<TileQ40, 8>(p, grid, smem_bytes, stream) : launch_tile<TileQ40, 4>(p, grid, smem_bytes, stream);
        else err = bb == 8 ? launch_tile<TileQ80, 8>(p, grid, smem_bytes, stream) : launch_tile<TileQ80, 4>(p, grid, smem_bytes, stream);
        if (err != 0) return err;
        b0 += nb;
    }
    return 0;
}

}  // namespace lw
