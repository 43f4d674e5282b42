// Batched mat-vec on the tensor cores (batch 2..16; all ten formats) [paper Sec 3.2: from a handful of columns on
// the mat-vec turns into a small mat-mat product, a dense contraction; Sec 3.3: one decode routine per format
// spliced into a common skeleton].
//
// With several columns the products, not the weight bytes, bound an fp32 kernel (74 TFLOP/s of packed FMAs at
// best, against the 98 / 196 TFLOP/s that 8 / 16 columns need to keep up with the weight stream of q4_0).  This
// kernel computes Y[b][r] = sum_k W[r][k] X[b][k] with mma.sync.m16n8k16 (bf16 x bf16 -> f32) and loses nothing
// to the narrow operand type:
//   * the integer code of a weight (q - 8 in [-8, 7], resp. an int8) is exact in bf16; the fp16 block scale is
//     applied in fp32 to each block's sum, as in the definition;
//   * an fp32 activation is cut into two bf16 terms: x1 = x cut off after eight significant bits, x2 = the rest
//     rounded to eight: x1 + x2 = x (1 + e) with |e| <= 2^-16, so code * x1 + code * x2, accumulated in fp32 by the
//     tensor core, is the product with the activation to 2^-16 relative -- 0.15 of the tolerance if every term of a
//     row erred the same way, and an error that scales with |w x| term by term (an activation that meets a zero
//     weight contributes exactly nothing).  Three terms (x exactly, -DLW_MMA_TERMS=3) measured 13 % slower at 8
//     columns and 23 % at 16, where the tensor pipe binds.  A NaN or Inf stays non-finite (in x1 or x2).
// The accuracy is that of the fp32 kernels' contract: |y - y_ref| <= 1e-4 * sum|w x| + 1e-6 with no extra term
// (q4_0, q8_0; q4_K's sub-block offsets go onto fp32 sums of the activations and bring an extra term back, see MmaQ4K).
//
// Why mma.sync and not tcgen05.mma here: the A operand is the decoded weight, which exists only in registers
// (18- and 34-byte blocks decode to fragments with byte permutes); tcgen05.mma reads A from shared or tensor
// memory, so every weight would take one more store and a proxy fence, for an N of 8..48 whose tensor time is
// already far below the decode time.  The warp-level form takes the fragments straight from the decode.
//
// Layout of the work.  A stage is 256 rows x 256 columns of weights (36 KB of q4_0, 68 KB of q8_0), brought in
// by a producer thread with one tiled bulk-tensor copy (the matrix as a 2-D tensor of 32-bit words; rows beyond
// the matrix arrive as zeros) into a ring of stages (full / empty mbarriers).  One 1-D bulk copy per row piece
// was measured at about 40 ns per copy, 10 us per stage.
// Each of 16 compute warps owns 16 rows of the stage (the M of the mma) and walks the stage's four 64-weight
// units; a lane (g = lane / 4, t = lane % 4) reads word t of the quants of rows g and g + 8, which holds
// exactly the eight weights of its A fragments once the k index inside a block is permuted -- the same
// permutation is applied to the activations when a lane loads its B fragments, and a sum does not care.
// The activations of a chunk of up to 1024 columns sit in shared memory as one bf16 plane per term.  Stages are
// numbered chunk-major, (row stage, sub-stage)-minor and dealt out in equal contiguous ranges to one CTA per
// SM, so a matrix of few rows still keeps every SM busy; sums stay in registers while a CTA stays inside one
// (chunk, row stage) and are then added into Y, which the host clears before the launch, with atomic adds
// (the other chunks of the same rows may belong to other CTAs).  The order of those adds is not fixed: results
// may differ in the last bits from run to run, within the tolerance.
//
// All waits are bounded: a wait that gives up records a fault code, the CTA stops waiting and copying, the
// producer drains what it has in flight, and the kernel terminates (its results are then meaningless and
// lw_device_status reports the fault).
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "lw.h"
#include "lw_internal.h"
#include "lw_stream_common.cuh"

namespace lw {
namespace {

#ifndef LW_MMA_WARPS
#define LW_MMA_WARPS 16
#endif
constexpr int kMmaWarps = LW_MMA_WARPS;               // compute warps
constexpr int kCtasPerSm = 16 / kMmaWarps;
constexpr int kSmemPerCta = kCtasPerSm == 1 ? 227 * 1024 : 113 * 1024;
constexpr int kXR = 8 * 64 / (32 * kMmaWarps);        // quads per thread, piece and group of eight columns
constexpr int kMmaComputeThreads = 32 * kMmaWarps;
constexpr int kMmaThreads = kMmaComputeThreads + 32;  // plus the producer warp
constexpr int kStageRows = 16 * kMmaWarps;            // 256
constexpr int kStageCols = 256;
constexpr int kStageUnits = kStageCols / 64;
constexpr int kMaxRing = 4;
constexpr int kXPad = 64;                             // bytes after each column of a plane: 16-byte loads of lanes
                                                      // (g, t) at 64 g + 16 t cover 128 distinct bytes per quarter warp
#ifndef LW_MMA_TERMS
#define LW_MMA_TERMS 2
#endif
constexpr int kTerms = LW_MMA_TERMS;                  // terms an activation is cut into (planes in shared memory)
constexpr int kTabRow = 72;                           // bytes between rows of a warp's scale table: 64 of entries + 8, so the
                                                      // eight rows a warp reads at once (8-byte entries) fall into different banks
constexpr int kSxBlockBytes = 64;                     // block sums of the activations: [block of 32][16 columns] floats
constexpr int kMmaHeader = 128;                       // barriers, the stop flag and the grid barrier's generation
constexpr uint32_t kGridPolls = 1u << 20;             // polls of the generation word (~0.5 us each) before giving up

// Grid barrier of the self-clearing launches: {count, generation}.  A launch holds every SM (one CTA per SM,
// cooperative), so two launches never use it at the same time; the last CTA to arrive resets the count and
// bumps the generation, which leaves the words ready for the next launch whatever happened in this one.
__device__ unsigned g_mma_grid_barrier[2] = {0u, 0u};

constexpr int kMmaMaxItems = 8;                       // matrices of one width per launch

// One matrix of a launch: its row stages are numbered rs_begin .. rs_begin + ceil(rows / 256) - 1 in the launch.
struct MmaItem {
    const float* X;
    float* Y;
    int64_t rows;
    int rs_begin;
    int same_x_end;       // first row stage (of the launch) after the run of matrices that share this X
};

struct MmaMaps {
    CUtensorMap m[kMmaMaxItems];
};

struct MmaParams {
    int* fault;
    int64_t cols;
    MmaItem item[kMmaMaxItems];
    int n_items;
    int total_rs;         // row stages of all matrices
    int batch;            // columns of this launch (<= 8 NT)
    int chunk_cols;       // 256, 512 or 1024: columns whose activations are resident at a time
    int ring;             // stages in the ring (2..kMaxRing)
    int early_weights;    // the weight copies may start before the previous kernel on the stream has completed
    int self_clear;       // cooperative launch: the CTAs clear Y themselves and meet at a grid barrier before the
                          // first sum is added (no clearing kernel in front)
    unsigned* grid_bar;   // {arrival count, generation} of that barrier, owned by the library
    uint32_t x_off, w_off;
    uint32_t sx_off, tab_off;   // block sums of the activations and the warps' scale tables (formats that need them)
    int drop_stage;       // testing aid (separate kernel build): the CTA's stage from which on no copy is requested
    // Outputs of the NEXT launch on the stream, cleared by this one at its end (a chain call passes them when they
    // overlap nothing this launch reads or writes): the next launch then needs no clearing kernel in front of it.
    float* next_y[kMmaMaxItems];
    int64_t next_n[kMmaMaxItems];     // floats
    int n_next;
};

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void compute_barrier() {
    asm volatile("bar.sync 1, %0;" ::"n"(kMmaComputeThreads) : "memory");
}
__device__ __forceinline__ uint32_t sub_bf16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
// Shared-memory loads at `base` + a compile-time byte offset: no address arithmetic per load.
template <int OFF>
__device__ __forceinline__ uint32_t lds32(uint32_t base) {
    uint32_t v;
    asm volatile("ld.shared.b32 %0, [%1+%2];" : "=r"(v) : "r"(base), "n"(OFF));
    return v;
}
template <int OFF>
__device__ __forceinline__ float lds_half(uint32_t base) {
    unsigned short h;
    asm volatile("ld.shared.u16 %0, [%1+%2];" : "=h"(h) : "r"(base), "n"(OFF));
    return __half2float(__ushort_as_half(h));
}
template <int OFF>
__device__ __forceinline__ void lds64(uint32_t base, uint32_t& a, uint32_t& b) {
    asm volatile("ld.shared.v2.b32 {%0, %1}, [%2+%3];" : "=r"(a), "=r"(b) : "r"(base), "n"(OFF));
}
template <int OFF>
__device__ __forceinline__ void lds_f32x2(uint32_t base, float& a, float& b) {
    asm volatile("ld.shared.v2.f32 {%0, %1}, [%2+%3];" : "=f"(a), "=f"(b) : "r"(base), "n"(OFF));
}
template <int OFF>
__device__ __forceinline__ void lds128(uint32_t base, uint32_t& a, uint32_t& b, uint32_t& c, uint32_t& d) {
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4+%5];" : "=r"(a), "=r"(b), "=r"(c), "=r"(d) : "r"(base), "n"(OFF));
}
// D = A (16 x 16, row) * B (16 x 8, col) + D, bf16 operands, fp32 accumulators
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// The same with D = A * B (the first product of a sum)
__device__ __forceinline__ void mma_bf16_first(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm("{\n\t.reg .f32 z;\n\tmov.f32 z, 0f00000000;\n\t"
                 "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
                 "{z, z, z, z};\n\t}"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// One box of the 2-D tensor behind `map` (x = first 32-bit word of the row piece, y = first row) into shared
// memory at `dst` (128-byte aligned); completion is counted in bytes on `bar`.  x * 4 must be a multiple of 16.
__device__ __forceinline__ void tensor_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar,
                                               uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%2, %3}], [%4], %5;" ::"r"(smem_u32(dst)),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}

// Two bytes of `v` (I and I + 1) as the bf16 pair (128 + byte I, 128 + byte I + 1): each byte lands in the seven
// mantissa bits of 128.0 (0x4300), so it must be below 128.
template <int I>
__device__ __forceinline__ uint32_t bytes_to_bf16_128_plus(uint32_t v) {
    return __byte_perm(v, 0x43434343u, I == 0 ? 0x4140u : 0x4342u);
}

// A lane's weights of one block of one row: four bf16 pairs.  p[0], p[1] = weights 4t .. 4t+3 of the block,
// p[2], p[3] = weights 16+4t .. 16+4t+3 (the k order the B fragments follow).  `wt` = shared-memory address of
// the row's piece of the stage plus 4 t (t = lane % 4), OFF = byte offset of the two-block unit from there.
struct MmaQ40 {
    static constexpr int kStageRows = 256;          // 16 warps x 16 rows
    static constexpr bool kF16 = false;
    static constexpr bool kQ6K = false;
    static constexpr bool kQ2K = false;
    static constexpr int kPiece = 8 * 18;               // bytes of a row's 256 columns
    static constexpr int kXWords = kPiece / 4;          // 32-bit words between consecutive stages of a row
    static constexpr bool kHasMin = false;              // no per-block offset term
    static constexpr int kTableBytes = 0;               // no per-warp table of decoded scales
    static __device__ __forceinline__ void prepare(uint32_t, uint32_t, int) {}
    template <int U, int BLK, int ROW>
    static __device__ __forceinline__ void block(uint32_t wt, uint32_t, int, uint32_t (&p)[4]) {
        constexpr int OFF = ROW + 36 * U;               // the two-block unit
        uint32_t q;
        if (BLK == 0)                                   // quants at bytes 2..17: word t straddles two words
            q = __byte_perm(lds32<OFF>(wt), lds32<OFF + 4>(wt), 0x5432u);
        else                                            // quants at bytes 20..35
            q = lds32<OFF + 20>(wt);
        const uint32_t lo = q & 0x0F0F0F0Fu, hi = (q >> 4) & 0x0F0F0F0Fu;
        const uint32_t bias = 0x43084308u;              // (136, 136): (128 + q) - 136 = q - 8, exactly
        p[0] = sub_bf16x2(bytes_to_bf16_128_plus<0>(lo), bias);
        p[1] = sub_bf16x2(bytes_to_bf16_128_plus<2>(lo), bias);
        p[2] = sub_bf16x2(bytes_to_bf16_128_plus<0>(hi), bias);
        p[3] = sub_bf16x2(bytes_to_bf16_128_plus<2>(hi), bias);
    }
    // `row` = address of the row's piece (without the lane's 4 t); the block's scale (and offset: none)
    template <int U, int BLK, int ROW>
    static __device__ __forceinline__ void scales(uint32_t row, uint32_t, float& d, float& m) {
        d = lds_half<ROW + 36 * U + 18 * BLK>(row);
        m = 0.f;
    }
};

struct MmaQ80 {
    static constexpr int kStageRows = 256;          // 16 warps x 16 rows
    static constexpr bool kF16 = false;
    static constexpr bool kQ6K = false;
    static constexpr bool kQ2K = false;
    static constexpr int kPiece = 8 * 34;
    static constexpr int kXWords = kPiece / 4;
    static constexpr bool kHasMin = false;
    static constexpr int kTableBytes = 0;
    static __device__ __forceinline__ void prepare(uint32_t, uint32_t, int) {}
    // An int8 code c as bf16: 0x4300 | (c & 0x7F) is 128 + (c & 0x7F), and 0x4300 | (c & 0x80) is 128 or 256;
    // their difference is c.
    static __device__ __forceinline__ uint32_t pair(uint32_t v) {
        return sub_bf16x2(v & 0xFF7FFF7Fu, v & 0xFF80FF80u);
    }
    template <int U, int BLK, int ROW>
    static __device__ __forceinline__ void block(uint32_t wt, uint32_t, int, uint32_t (&p)[4]) {
        constexpr int OFF = ROW + 68 * U;
        uint32_t qa, qb;                                // quant words t and 4 + t of the block
        if (BLK == 0) {                                 // quants at bytes 2..33
            qa = __byte_perm(lds32<OFF>(wt), lds32<OFF + 4>(wt), 0x5432u);
            qb = __byte_perm(lds32<OFF + 16>(wt), lds32<OFF + 20>(wt), 0x5432u);
        } else {                                        // quants at bytes 36..67
            qa = lds32<OFF + 36>(wt);
            qb = lds32<OFF + 52>(wt);
        }
        p[0] = pair(__byte_perm(qa, 0x43434343u, 0x4140u));
        p[1] = pair(__byte_perm(qa, 0x43434343u, 0x4342u));
        p[2] = pair(__byte_perm(qb, 0x43434343u, 0x4140u));
        p[3] = pair(__byte_perm(qb, 0x43434343u, 0x4342u));
    }
    template <int U, int BLK, int ROW>
    static __device__ __forceinline__ void scales(uint32_t row, uint32_t, float& d, float& m) {
        d = lds_half<ROW + 68 * U + 34 * BLK>(row);
        m = 0.f;
    }
};

// q4_K: a row's 256 columns are one 144-byte super-block {d, dmin (fp16), 12 bytes of 6-bit scales and offsets, 128
// bytes of nibbles}; sub-blocks 2 U and 2 U + 1 are the low and high nibbles of bytes 32 U .. 32 U + 31, and a weight
// is d * sc * q - dmin * m.  The kernel multiplies the codes q (exact in bf16) and applies d * sc to the sum and
// dmin * m to the sum of the sub-block's activations, like the fp32-activation streaming family: an activation that
// is huge beside its neighbours and meets a weight near zero leaves an absolute error (the extra term E of the
// accuracy statement).  The 6-bit fields are unpacked once per warp and stage into a table of (d * sc, dmin * m).
struct MmaQ4K {
    static constexpr int kStageRows = 256;          // 16 warps x 16 rows
    static constexpr bool kF16 = false;
    static constexpr bool kQ6K = false;
    static constexpr bool kQ2K = false;
    static constexpr int kPiece = 144;
    static constexpr int kXWords = kPiece / 4;
    static constexpr bool kHasMin = true;
    static constexpr int kTableBytes = 16 * kTabRow;    // per warp: 16 rows x 8 sub-blocks x (d * sc, dmin * m)
    // `rows` = address of the warp's first row piece of the stage, `tab` = the warp's table; lane: row lane / 2,
    // sub-blocks 4 (lane % 2) .. + 3
    static __device__ __forceinline__ void prepare(uint32_t rows, uint32_t tab, int lane) {
        const uint32_t row = rows + (uint32_t)(lane >> 1) * kPiece;
        const uint32_t dd = lds32<0>(row), w0 = lds32<4>(row), w1 = lds32<8>(row), w2 = lds32<12>(row);
        const float d = __half2float(__ushort_as_half((unsigned short)(dd & 0xFFFFu)));
        const float dmin = __half2float(__ushort_as_half((unsigned short)(dd >> 16)));
        const bool upper = lane & 1;
        const uint32_t out = tab + (uint32_t)(lane >> 1) * kTabRow + (upper ? 32u : 0u);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t sc, mn;
            if (!upper) {
                sc = (w0 >> (8 * j)) & 63u;
                mn = (w1 >> (8 * j)) & 63u;
            } else {
                sc = ((w2 >> (8 * j)) & 0xFu) | (((w0 >> (8 * j + 6)) & 3u) << 4);
                mn = ((w2 >> (8 * j + 4)) & 0xFu) | (((w1 >> (8 * j + 6)) & 3u) << 4);
            }
            const float dsc = d * (float)sc, dmn = dmin * (float)mn;
            asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(out + 8u * j), "f"(dsc), "f"(dmn) : "memory");
        }
    }
    template <int U, int BLK, int ROW>
    static __device__ __forceinline__ void block(uint32_t wt, uint32_t, int, uint32_t (&p)[4]) {
        constexpr int OFF = ROW + 16 + 32 * U;          // the 32 bytes of sub-blocks 2 U (low nibbles), 2 U + 1 (high)
        uint32_t qa = lds32<OFF>(wt), qb = lds32<OFF + 16>(wt);         // bytes 4t .. 4t+3 and 16+4t .. 16+4t+3
        if (BLK == 1) {
            qa >>= 4;
            qb >>= 4;
        }
        qa &= 0x0F0F0F0Fu;
        qb &= 0x0F0F0F0Fu;
        const uint32_t bias = 0x43004300u;              // (128, 128): (128 + q) - 128 = q, exactly
        p[0] = sub_bf16x2(bytes_to_bf16_128_plus<0>(qa), bias);
        p[1] = sub_bf16x2(bytes_to_bf16_128_plus<2>(qa), bias);
        p[2] = sub_bf16x2(bytes_to_bf16_128_plus<0>(qb), bias);
        p[3] = sub_bf16x2(bytes_to_bf16_128_plus<2>(qb), bias);
    }
    // ROW / kPiece = row of the warp's 16 (g or g + 8 is added by the caller through `tabg`): tab entry of row g
    template <int U, int BLK, int ROW>
    static __device__ __forceinline__ void scales(uint32_t, uint32_t tabg, float& d, float& m) {
        lds_f32x2<(ROW / kPiece) * kTabRow + 8 * (2 * U + BLK)>(tabg, d, m);
    }
};

// q5_K: q4_K's layout with 32 bytes of fifth bits between the scales and the nibbles (176 bytes per 256 weights): bit
// s of byte l is the high bit of weight l of sub-block s, so a code is 0..31 -- still exact in bf16.
struct MmaQ5K {
    static constexpr int kStageRows = 256;          // 16 warps x 16 rows
    static constexpr bool kF16 = false;
    static constexpr bool kQ6K = false;
    static constexpr bool kQ2K = false;
    static constexpr int kPiece = 176;
    static constexpr int kXWords = kPiece / 4;
    static constexpr bool kHasMin = true;
    static constexpr int kTableBytes = MmaQ4K::kTableBytes;
    static __device__ __forceinline__ void prepare(uint32_t rows, uint32_t tab, int lane) {
        // the same header {d, dmin, 12 bytes of 6-bit fields} at the same offsets, rows 176 bytes apart
        const uint32_t row = rows + (uint32_t)(lane >> 1) * kPiece;
        const uint32_t dd = lds32<0>(row), w0 = lds32<4>(row), w1 = lds32<8>(row), w2 = lds32<12>(row);
        const float d = __half2float(__ushort_as_half((unsigned short)(dd & 0xFFFFu)));
        const float dmin = __half2float(__ushort_as_half((unsigned short)(dd >> 16)));
        const bool upper = lane & 1;
        const uint32_t out = tab + (uint32_t)(lane >> 1) * kTabRow + (upper ? 32u : 0u);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t sc, mn;
            if (!upper) {
                sc = (w0 >> (8 * j)) & 63u;
                mn = (w1 >> (8 * j)) & 63u;
            } else {
                sc = ((w2 >> (8 * j)) & 0xFu) | (((w0 >> (8 * j + 6)) & 3u) << 4);
                mn = ((w2 >> (8 * j + 4)) & 0xFu) | (((w1 >> (8 * j + 6)) & 3u) << 4);
            }
            const float dsc = d * (float)sc, dmn = dmin * (float)mn;
            asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(out + 8u * j), "f"(dsc), "f"(dmn) : "memory");
        }
    }
    template <int U, int BLK, int ROW>
    static __device__ __forceinline__ void block(uint32_t wt, uint32_t, int, uint32_t (&p)[4]) {
        constexpr int S = 2 * U + BLK;                  // sub-block = bit of the fifth-bit bytes
        uint32_t qa = lds32<ROW + 48 + 32 * U>(wt), qb = lds32<ROW + 48 + 32 * U + 16>(wt);
        const uint32_t ha = lds32<ROW + 16>(wt), hb = lds32<ROW + 32>(wt);   // fifth bits of weights 4t.. and 16+4t..
        if (BLK == 1) {
            qa >>= 4;
            qb >>= 4;
        }
        qa = (qa & 0x0F0F0F0Fu) | (((ha >> S) & 0x01010101u) << 4);
        qb = (qb & 0x0F0F0F0Fu) | (((hb >> S) & 0x01010101u) << 4);
        const uint32_t bias = 0x43004300u;              // (128, 128): (128 + q) - 128 = q, exactly
        p[0] = sub_bf16x2(bytes_to_bf16_128_plus<0>(qa), bias);
        p[1] = sub_bf16x2(bytes_to_bf16_128_plus<2>(qa), bias);
        p[2] = sub_bf16x2(bytes_to_bf16_128_plus<0>(qb), bias);
        p[3] = sub_bf16x2(bytes_to_bf16_128_plus<2>(qb), bias);
    }
    template <int U, int BLK, int ROW>
    static __device__ __forceinline__ void scales(uint32_t, uint32_t tabg, float& d, float& m) {
        lds_f32x2<(ROW / kPiece) * kTabRow + 8 * (2 * U + BLK)>(tabg, d, m);
    }
};

// Four bits (0..3 of `x`) spread to bit 4 of four bytes: the fifth bits of four 5-bit codes.
__device__ __forceinline__ uint32_t fifth_bits(uint32_t x) { return ((x & 0xFu) * 0x02040810u) & 0x10101010u; }

// The 32-weight formats with an offset and / or a fifth bit: q4_1 {d, m, 16 bytes of nibbles} = d * q + m, q5_0 {d, 32
// fifth bits, nibbles} = d * (q - 16), q5_1 {d, m, fifth bits, nibbles} = d * q + m; nibble and bit order as in q4_0
// (byte j: weights j and j + 16; bit j: weight j).  Codes 0..31 are exact in bf16.  q5_0 has no offset: E = 0; the
// offsets m of q4_1 / q5_1 go onto fp32 block sums of the activations (extra term E, c = 2^-18).
template <int FMT>
struct MmaLegacy {
    static constexpr bool kFive = FMT != LW_Q4_1;
    static constexpr bool kHasMin = FMT != LW_Q5_0;
    static constexpr int kBlock = FMT == LW_Q4_1 ? 20 : (FMT == LW_Q5_0 ? 22 : 24);
    static constexpr int kStageRows = 256;
    static constexpr bool kF16 = false;
    static constexpr bool kQ6K = false;
    static constexpr bool kQ2K = false;
    // 16 bytes more than a row's 256 columns are fetched for q4_1 and q5_1: their 160- and 192-byte pitches would put
    // the eight rows a warp reads at once into four resp. two banks (176 and 208 spread them over eight)
    static constexpr int kPiece = 8 * kBlock + (FMT == LW_Q5_0 ? 0 : 16);
    static constexpr int kXWords = 8 * kBlock / 4;
    static constexpr int kTableBytes = 0;
    static __device__ __forceinline__ void prepare(uint32_t, uint32_t, int) {}
    // wt = the row's piece + 4 t, row = the row's piece, t = lane % 4
    template <int U, int BLK, int ROW>
    static __device__ __forceinline__ void block(uint32_t wt, uint32_t row, int t, uint32_t (&p)[4]) {
        constexpr int B0 = ROW + 2 * kBlock * U + kBlock * BLK;       // the block, in bytes from the row's piece
        uint32_t q, qh = 0;
        if constexpr (FMT == LW_Q4_1) {
            q = lds32<B0 + 4>(wt);
        } else if constexpr (FMT == LW_Q5_1) {
            q = lds32<B0 + 8>(wt);
            qh = lds32<B0 + 4>(row);
        } else if constexpr (BLK == 0) {                             // q5_0, block at 44 U: fields two bytes off a word
            q = __byte_perm(lds32<B0 + 4>(wt), lds32<B0 + 8>(wt), 0x5432u);         // nibble bytes 6 + 4t ..
            qh = __byte_perm(lds32<B0>(row), lds32<B0 + 4>(row), 0x5432u);          // fifth bits at bytes 2 .. 5
        } else {                                                     // q5_0, block at 44 U + 22: fields on words
            q = lds32<B0 + 6>(wt);
            qh = lds32<B0 + 2>(row);
        }
        uint32_t lo = q & 0x0F0F0F0Fu, hi = (q >> 4) & 0x0F0F0F0Fu;
        if constexpr (kFive) {
            const uint32_t h = qh >> (4 * t);                        // bits 4t .. 4t+3: weights 4t ..; 16 higher: 16+4t ..
            lo |= fifth_bits(h);
            hi |= fifth_bits(h >> 16);
        }
        const uint32_t bias = FMT == LW_Q5_0 ? 0x43104310u : 0x43004300u;     // (128 + q) - 144 = q - 16, resp. - 128 = q
        p[0] = sub_bf16x2(bytes_to_bf16_128_plus<0>(lo), bias);
        p[1] = sub_bf16x2(bytes_to_bf16_128_plus<2>(lo), bias);
        p[2] = sub_bf16x2(bytes_to_bf16_128_plus<0>(hi), bias);
        p[3] = sub_bf16x2(bytes_to_bf16_128_plus<2>(hi), bias);
    }
    // (d, minus the offset: the caller subtracts m times the block's sum of activations)
    template <int U, int BLK, int ROW>
    static __device__ __forceinline__ void scales(uint32_t row, uint32_t, float& d, float& m) {
        constexpr int B0 = ROW + 2 * kBlock * U + kBlock * BLK;
        d = lds_half<B0>(row);
        if constexpr (kHasMin) m = -lds_half<B0 + 2>(row);
        else m = 0.f;
    }
};

// f16 weights: they are the A operand as they lie in memory (mma with f16 operands), nothing is decoded.  A row's
// 256 columns are 512 bytes, fetched as four 128-byte slices (one per 64-column unit) with the 128-byte swizzle of
// the tensor copy, so that the eight rows a warp reads at once fall into different banks: 16-byte chunk c of row r
// of a slice sits at chunk c ^ (r % 8).  A stage is 128 rows; warps 0-7 take units 0 and 1 of their 16 rows, warps
// 8-15 units 2 and 3.  The activations are held as f16 terms of x * s, s a power of two per block of 32 and
// column that brings the block's largest magnitude to 2^14..2^15: the first term is cut off exactly, the second
// rounds what is left (22 significant bits of the element, but nothing below 2^-38 of the block's largest
// magnitude: the extra term E of the accuracy statement with a tiny constant); 1 / s multiplies the block's sum.
struct MmaF16 {
    static constexpr int kStageRows = 128;
    static constexpr bool kF16 = true;
    static constexpr bool kQ6K = false;
    static constexpr bool kQ2K = false;
    static constexpr int kPiece = 512;
    static constexpr bool kHasMin = false;
    static constexpr int kTableBytes = 0;
    static constexpr int kSliceBytes = kStageRows * 128;     // one unit of all the stage's rows
};

__device__ __forceinline__ void mma_f16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_f16_first(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t b0, uint32_t b1) {
    asm("{\n\t.reg .f32 z;\n\tmov.f32 z, 0f00000000;\n\t"
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{z, z, z, z};\n\t}"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// One block of 32 f16 weights of the warp's 16 rows against all columns.  wrow = address of row g's 128 bytes in
// slice 0 of the stage plus 8 (t % 2); sw[h] = byte offset of the lane's swizzled 16-byte chunk for half h of block
// 0 (block 1: sw[2 + h]); sx = the lane's two block scales (1 / s), group nt 32 bytes further.
template <int NT, int U, int BLK>
__device__ __forceinline__ void block_step_f16(uint32_t wrow, const uint32_t (&sw)[4], uint32_t sx,
                                               const uint32_t (&xp)[NT][kTerms], float (&y)[NT][4]) {
    constexpr int kSlice = U * MmaF16::kSliceBytes;
    uint32_t a[4], b[4];
    lds64<kSlice>(wrow + sw[2 * BLK], a[0], a[1]);               // row g: k = 4t .. 4t+3
    lds64<kSlice>(wrow + sw[2 * BLK + 1], a[2], a[3]);           //        k = 16+4t ..
    lds64<kSlice + 8 * 128>(wrow + sw[2 * BLK], b[0], b[1]);     // row g + 8 (same swizzle: (g + 8) % 8 == g)
    lds64<kSlice + 8 * 128>(wrow + sw[2 * BLK + 1], b[2], b[3]);
    constexpr int kX = 2 * (64 * U + 32 * BLK);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        float c[4];
#pragma unroll
        for (int s = 0; s < kTerms; ++s) {
            uint32_t b0, b1, b2, b3;
            lds128<kX>(xp[nt][s], b0, b1, b2, b3);
            if (s == 0)
                mma_f16_first(c, a[0], b[0], a[1], b[1], b0, b1);
            else
                mma_f16(c, a[0], b[0], a[1], b[1], b0, b1);
            mma_f16(c, a[2], b[2], a[3], b[3], b2, b3);
        }
        float s0, s1;                                            // 1 / s of columns 2 t and 2 t + 1 of the group
        if (nt == 0)
            lds_f32x2<kSxBlockBytes * (2 * U + BLK)>(sx, s0, s1);
        else
            lds_f32x2<kSxBlockBytes * (2 * U + BLK) + 32>(sx, s0, s1);
        y[nt][0] = fmaf(s0, c[0], y[nt][0]);
        y[nt][1] = fmaf(s1, c[1], y[nt][1]);
        y[nt][2] = fmaf(s0, c[2], y[nt][2]);
        y[nt][3] = fmaf(s1, c[3], y[nt][3]);
    }
}

// q6_K: 210-byte super-blocks {128 bytes of low nibbles, 64 bytes of upper bit pairs, 16 int8 scales (one per 16
// weights), d}.  210 is not a multiple of 16, so a row's piece of a stage starts anywhere on a 2-byte grid: the
// tensor copy starts at the 16-byte boundary below it and fetches 240 bytes per row, and the kernel indexes from
// the remainder `o` (0, 2, .. 14); where o is 2 modulo 4 every word of the piece straddles two words of shared
// memory (MIS: two loads and a byte permute).  A code is nibble | two upper bits << 4 = 0..63, minus 32: exact in
// bf16, and there is no offset term: E = 0.  The two 16-weight halves of a block have their own scales, so the two
// mma of a term go to separate accumulators.  Unit U = half U / 2 of the super-block, groups {0, 1} (low nibbles of
// bytes l and l + 32) for even U and {2, 3} (high nibbles) for odd U.
struct MmaQ6K {
    static constexpr int kStageRows = 256;
    static constexpr bool kF16 = false;
    static constexpr bool kQ6K = true;
    static constexpr bool kQ2K = false;
    static constexpr int kSuper = 210;                  // bytes of 256 weights
    static constexpr int kPiece = 240;                  // bytes fetched per row and stage: 210 + up to 14 in front, and 16
                                                        // more so that the pitch spreads eight rows over eight banks
    static constexpr bool kHasMin = false;
    static constexpr int kTableBytes = 16 * kTabRow;    // per warp: 16 rows x 16 (d * scale)
    // rows = the warp's first row piece + o; lane: row lane / 2, scales 8 (lane % 2) .. + 7
    static __device__ __forceinline__ void prepare(uint32_t rows, uint32_t tab, int lane) {
        const uint32_t row = rows + (uint32_t)(lane >> 1) * kPiece;
        const float d = lds_half<208>(row);
        const uint32_t sc = row + 192u + 8u * (lane & 1), out = tab + (uint32_t)(lane >> 1) * kTabRow + 32u * (lane & 1);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            int v;
            asm volatile("ld.shared.s8 %0, [%1];" : "=r"(v) : "r"(sc + j));
            asm volatile("st.shared.f32 [%0], %1;" ::"r"(out + 4u * j), "f"(d * (float)v) : "memory");
        }
    }
};

// q2_K: 84-byte super-blocks {16 bytes of 4-bit scale | 4-bit offset (one per 16 weights), 64 bytes of 2-bit codes, d,
// dmin}: weight = d * sc * q - dmin * m.  84 is a multiple of 4 but not of 16: fetched like q6_K from the 16-byte
// boundary below the piece (112 bytes per row), the remainder is a whole number of words.  Group j (0..3) of a half
// of 128 weights is bits 2j, 2j+1 of the half's 32 bytes.  Codes 0..3 are exact in bf16; the offsets go onto fp32
// sums of each 16 activations (extra term E, c = 2^-18).  Unit U = half U / 2, groups {0, 1} or {2, 3}.
struct MmaQ2K {
    static constexpr int kStageRows = 256;
    static constexpr bool kF16 = false;
    static constexpr bool kQ6K = false;
    static constexpr bool kQ2K = true;
    static constexpr int kSuper = 84;
    static constexpr int kPiece = 112;                  // 84 + up to 12 in front + 16 (bank spread, as for q6_K)
    static constexpr bool kHasMin = false;              // (its own block step applies the offsets)
    static constexpr int kTabRow2 = 136;                // 128 bytes of entries + 8 (bank spread as above)
    static constexpr int kTableBytes = 16 * kTabRow2;   // per warp: 16 rows x 16 x (d * sc, dmin * m)
    // rows = the warp's first row piece + o; lane: row lane / 2, sub-blocks 8 (lane % 2) .. + 7
    static __device__ __forceinline__ void prepare(uint32_t rows, uint32_t tab, int lane) {
        const uint32_t row = rows + (uint32_t)(lane >> 1) * kPiece;
        const uint32_t dd = lds32<80>(row);
        const float d = __half2float(__ushort_as_half((unsigned short)(dd & 0xFFFFu)));
        const float dmin = __half2float(__ushort_as_half((unsigned short)(dd >> 16)));
        const uint32_t w0 = lds32<0>(row + 8u * (lane & 1)), w1 = lds32<4>(row + 8u * (lane & 1));
        const uint32_t out = tab + (uint32_t)(lane >> 1) * kTabRow2 + 64u * (lane & 1);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t b = ((j < 4 ? w0 : w1) >> (8 * (j & 3))) & 0xFFu;
            asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(out + 8u * j), "f"(d * (float)(b & 0xFu)),
                         "f"(dmin * (float)(b >> 4))
                         : "memory");
        }
    }
};

// One group of 32 q2_K weights of the warp's 16 rows against all columns.  tabg = the warp's table at row g; sx = the
// lane's sums of 16 activations: [block of 32][half][16 columns], columns 2 t and 2 t + 1, group nt 32 bytes further.
template <int NT, int U, int BLK>
__device__ __forceinline__ void block_step_q2k(uint32_t wt, uint32_t tabg, uint32_t sx, const uint32_t (&xp)[NT][kTerms],
                                               float (&y)[NT][4]) {
    constexpr int kHalf = U / 2, kGroup = 2 * (U & 1) + BLK, kShift = 2 * kGroup;
    constexpr int kQs = 16 + 32 * kHalf, kRow8 = 8 * MmaQ2K::kPiece;
    const uint32_t bias = 0x43004300u;                  // (128 + q) - 128 = q, exactly
    uint32_t a[4], b[4];
    {
        const uint32_t q0 = (lds32<kQs>(wt) >> kShift) & 0x03030303u, q1 = (lds32<kQs + 16>(wt) >> kShift) & 0x03030303u;
        a[0] = sub_bf16x2(bytes_to_bf16_128_plus<0>(q0), bias);
        a[1] = sub_bf16x2(bytes_to_bf16_128_plus<2>(q0), bias);
        a[2] = sub_bf16x2(bytes_to_bf16_128_plus<0>(q1), bias);
        a[3] = sub_bf16x2(bytes_to_bf16_128_plus<2>(q1), bias);
        const uint32_t r0 = (lds32<kRow8 + kQs>(wt) >> kShift) & 0x03030303u,
                       r1 = (lds32<kRow8 + kQs + 16>(wt) >> kShift) & 0x03030303u;
        b[0] = sub_bf16x2(bytes_to_bf16_128_plus<0>(r0), bias);
        b[1] = sub_bf16x2(bytes_to_bf16_128_plus<2>(r0), bias);
        b[2] = sub_bf16x2(bytes_to_bf16_128_plus<0>(r1), bias);
        b[3] = sub_bf16x2(bytes_to_bf16_128_plus<2>(r1), bias);
    }
    // (d * sc, dmin * m) of the group's two halves: row g, then row g + 8
    float d00, m00, d01, m01, d10, m10, d11, m11;
    constexpr int kT = 8 * (8 * kHalf + 2 * kGroup);
    lds_f32x2<kT>(tabg, d00, m00);
    lds_f32x2<kT + 8>(tabg, d01, m01);
    lds_f32x2<8 * MmaQ2K::kTabRow2 + kT>(tabg, d10, m10);
    lds_f32x2<8 * MmaQ2K::kTabRow2 + kT + 8>(tabg, d11, m11);
    constexpr int kX = 2 * (64 * U + 32 * BLK);
    constexpr int kS = 128 * (2 * U + BLK);              // the block's sums of activations
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        float c0[4], c1[4];
#pragma unroll
        for (int s = 0; s < kTerms; ++s) {
            uint32_t b0, b1, b2, b3;
            lds128<kX>(xp[nt][s], b0, b1, b2, b3);
            if (s == 0) {
                mma_bf16_first(c0, a[0], b[0], a[1], b[1], b0, b1);
                mma_bf16_first(c1, a[2], b[2], a[3], b[3], b2, b3);
            } else {
                mma_bf16(c0, a[0], b[0], a[1], b[1], b0, b1);
                mma_bf16(c1, a[2], b[2], a[3], b[3], b2, b3);
            }
        }
        float s00, s01, s10, s11;                        // sums of the first / second 16 activations, columns 2t, 2t+1
        if (nt == 0) {
            lds_f32x2<kS>(sx, s00, s01);
            lds_f32x2<kS + 64>(sx, s10, s11);
        } else {
            lds_f32x2<kS + 32>(sx, s00, s01);
            lds_f32x2<kS + 64 + 32>(sx, s10, s11);
        }
        y[nt][0] = fmaf(-m01, s10, fmaf(-m00, s00, fmaf(d01, c1[0], fmaf(d00, c0[0], y[nt][0]))));
        y[nt][1] = fmaf(-m01, s11, fmaf(-m00, s01, fmaf(d01, c1[1], fmaf(d00, c0[1], y[nt][1]))));
        y[nt][2] = fmaf(-m11, s10, fmaf(-m10, s00, fmaf(d11, c1[2], fmaf(d10, c0[2], y[nt][2]))));
        y[nt][3] = fmaf(-m11, s11, fmaf(-m10, s01, fmaf(d11, c1[3], fmaf(d10, c0[3], y[nt][3]))));
    }
}

// A 32-bit word of the piece at byte OFF from `wt` (word-aligned address below the piece's word + 4 t); MIS: the piece
// is two bytes off the word grid.
template <int OFF, bool MIS>
__device__ __forceinline__ uint32_t q6k_word(uint32_t wt) {
    if (MIS) return __byte_perm(lds32<OFF>(wt), lds32<OFF + 4>(wt), 0x5432u);
    return lds32<OFF>(wt);
}

// One group of 32 q6_K weights of the warp's 16 rows against all columns.  tabg = the warp's table at row g.
template <int NT, int U, int BLK, bool MIS>
__device__ __forceinline__ void block_step_q6k(uint32_t wt, uint32_t tabg, const uint32_t (&xp)[NT][kTerms],
                                               float (&y)[NT][4]) {
    constexpr int kHalf = U / 2, kGroup = 2 * (U & 1) + BLK;
    constexpr int kQl = 64 * kHalf + 32 * BLK, kQh = 128 + 32 * kHalf, kShift = 2 * kGroup;
    constexpr bool kHigh = (U & 1) != 0;
    constexpr int kRow8 = 8 * MmaQ6K::kPiece;
    uint32_t a[4], b[4];
    {
        const uint32_t bias = 0x43204320u;              // (160, 160): (128 + code) - 160 = code - 32, exactly
        uint32_t l0 = q6k_word<kQl, MIS>(wt), l1 = q6k_word<kQl + 16, MIS>(wt);
        uint32_t h0 = q6k_word<kQh, MIS>(wt), h1 = q6k_word<kQh + 16, MIS>(wt);
        if (kHigh) l0 >>= 4, l1 >>= 4;
        l0 = (l0 & 0x0F0F0F0Fu) | (((h0 >> kShift) & 0x03030303u) << 4);
        l1 = (l1 & 0x0F0F0F0Fu) | (((h1 >> kShift) & 0x03030303u) << 4);
        a[0] = sub_bf16x2(bytes_to_bf16_128_plus<0>(l0), bias);
        a[1] = sub_bf16x2(bytes_to_bf16_128_plus<2>(l0), bias);
        a[2] = sub_bf16x2(bytes_to_bf16_128_plus<0>(l1), bias);
        a[3] = sub_bf16x2(bytes_to_bf16_128_plus<2>(l1), bias);
        l0 = q6k_word<kRow8 + kQl, MIS>(wt), l1 = q6k_word<kRow8 + kQl + 16, MIS>(wt);
        h0 = q6k_word<kRow8 + kQh, MIS>(wt), h1 = q6k_word<kRow8 + kQh + 16, MIS>(wt);
        if (kHigh) l0 >>= 4, l1 >>= 4;
        l0 = (l0 & 0x0F0F0F0Fu) | (((h0 >> kShift) & 0x03030303u) << 4);
        l1 = (l1 & 0x0F0F0F0Fu) | (((h1 >> kShift) & 0x03030303u) << 4);
        b[0] = sub_bf16x2(bytes_to_bf16_128_plus<0>(l0), bias);
        b[1] = sub_bf16x2(bytes_to_bf16_128_plus<2>(l0), bias);
        b[2] = sub_bf16x2(bytes_to_bf16_128_plus<0>(l1), bias);
        b[3] = sub_bf16x2(bytes_to_bf16_128_plus<2>(l1), bias);
    }
    float s00, s01, s10, s11;                            // d * scale of (row g, half 0 / 1), (row g + 8, half 0 / 1)
    lds_f32x2<4 * (8 * kHalf + 2 * kGroup)>(tabg, s00, s01);
    lds_f32x2<8 * kTabRow + 4 * (8 * kHalf + 2 * kGroup)>(tabg, s10, s11);
    constexpr int kX = 2 * (64 * U + 32 * BLK);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        float c0[4], c1[4];
#pragma unroll
        for (int s = 0; s < kTerms; ++s) {
            uint32_t b0, b1, b2, b3;
            lds128<kX>(xp[nt][s], b0, b1, b2, b3);
            if (s == 0) {
                mma_bf16_first(c0, a[0], b[0], a[1], b[1], b0, b1);
                mma_bf16_first(c1, a[2], b[2], a[3], b[3], b2, b3);
            } else {
                mma_bf16(c0, a[0], b[0], a[1], b[1], b0, b1);
                mma_bf16(c1, a[2], b[2], a[3], b[3], b2, b3);
            }
        }
        y[nt][0] = fmaf(s01, c1[0], fmaf(s00, c0[0], y[nt][0]));
        y[nt][1] = fmaf(s01, c1[1], fmaf(s00, c0[1], y[nt][1]));
        y[nt][2] = fmaf(s11, c1[2], fmaf(s10, c0[2], y[nt][2]));
        y[nt][3] = fmaf(s11, c1[3], fmaf(s10, c0[3], y[nt][3]));
    }
}

template <int NT, bool MIS>
__device__ __forceinline__ void stage_q6k(uint32_t wt, uint32_t tabg, const uint32_t (&xp)[NT][kTerms], float (&y)[NT][4]) {
    block_step_q6k<NT, 0, 0, MIS>(wt, tabg, xp, y);
    block_step_q6k<NT, 0, 1, MIS>(wt, tabg, xp, y);
    block_step_q6k<NT, 1, 0, MIS>(wt, tabg, xp, y);
    block_step_q6k<NT, 1, 1, MIS>(wt, tabg, xp, y);
    block_step_q6k<NT, 2, 0, MIS>(wt, tabg, xp, y);
    block_step_q6k<NT, 2, 1, MIS>(wt, tabg, xp, y);
    block_step_q6k<NT, 3, 0, MIS>(wt, tabg, xp, y);
    block_step_q6k<NT, 3, 1, MIS>(wt, tabg, xp, y);
}

// One block (32 weights) of the warp's 16 rows against all columns: decode the lane's fragments of rows g and
// g + 8, six products per group of eight columns into one accumulator, then the block scales in fp32.
// U = unit of the stage (0..3), BLK = block of the unit; xp[nt][s] = address of the lane's B fragments of plane s,
// column group nt, at the stage's first column.
// tabg = the warp's scale table at row g (formats with one); sx = address of the lane's two block sums of the
// activations, group nt 32 bytes further (formats with an offset term).
template <class T, int NT, int U, int BLK>
__device__ __forceinline__ void block_step(uint32_t wt, uint32_t row, uint32_t tabg, uint32_t sx,
                                           const uint32_t (&xp)[NT][kTerms], float (&y)[NT][4]) {
    constexpr int kPiece = T::kPiece;
    uint32_t a[4], b[4];
    const int t = (int)((wt - row) >> 2);
    T::template block<U, BLK, 0>(wt, row, t, a);
    T::template block<U, BLK, 8 * kPiece>(wt, row, t, b);
    float d0, d1, m0, m1;
    T::template scales<U, BLK, 0>(row, tabg, d0, m0);
    T::template scales<U, BLK, 8 * kPiece>(row, tabg, d1, m1);
    constexpr int kX = 2 * (64 * U + 32 * BLK);          // bytes into a plane's column
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        float c[4];
#pragma unroll
        for (int s = 0; s < kTerms; ++s) {
            uint32_t b0, b1, b2, b3;
            lds128<kX>(xp[nt][s], b0, b1, b2, b3);      // k = 4t .. 4t+3 and k = 16+4t .. 16+4t+3
            if (s == 0)
                mma_bf16_first(c, a[0], b[0], a[1], b[1], b0, b1);
            else
                mma_bf16(c, a[0], b[0], a[1], b[1], b0, b1);
            mma_bf16(c, a[2], b[2], a[3], b[3], b2, b3);
        }
        y[nt][0] = fmaf(d0, c[0], y[nt][0]);
        y[nt][1] = fmaf(d0, c[1], y[nt][1]);
        y[nt][2] = fmaf(d1, c[2], y[nt][2]);
        y[nt][3] = fmaf(d1, c[3], y[nt][3]);
        if constexpr (T::kHasMin) {
            // minus the block's offset times the sum of its activations (columns 2 t and 2 t + 1 of the group)
            float s0, s1;
            if (nt == 0)
                lds_f32x2<kSxBlockBytes * (2 * U + BLK)>(sx, s0, s1);
            else
                lds_f32x2<kSxBlockBytes * (2 * U + BLK) + 32>(sx, s0, s1);
            y[nt][0] = fmaf(-m0, s0, y[nt][0]);
            y[nt][1] = fmaf(-m0, s1, y[nt][1]);
            y[nt][2] = fmaf(-m1, s0, y[nt][2]);
            y[nt][3] = fmaf(-m1, s1, y[nt][3]);
        }
    }
}

// fp32 -> bf16 terms.  The first is x cut off after eight significant bits (exact difference).  With two terms
// (the default) the second is the rest rounded to nearest: x1 + x2 = x (1 + e), |e| <= 2^-16.  With three
// (-DLW_MMA_TERMS=3) the second is cut off as well and the third holds what is left: x1 + x2 + x3 == x exactly.
// A NaN stays one (in x1, or in x2 when only its low payload bits were set); an Inf gives x2 = NaN.
__device__ __forceinline__ void split3(float x, uint32_t& h1, uint32_t& h2, uint32_t& h3) {
    const uint32_t b1 = __float_as_uint(x) & 0xFFFF0000u;
    const float r1 = x - __uint_as_float(b1);
    h1 = b1 >> 16;
    if (kTerms == 2) {
        unsigned short r;
        asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(r) : "f"(r1));
        h2 = r;
        h3 = 0;
    } else {
        const uint32_t b2 = __float_as_uint(r1) & 0xFFFF0000u;
        const float r2 = r1 - __uint_as_float(b2);
        h2 = b2 >> 16;
        h3 = __float_as_uint(r2) >> 16;                 // at most eight significant bits are left: exact
    }
}

// fp32 -> f16 terms of x (already scaled into the f16 range): cut off (exact differences) except the last, which
// rounds the rest
__device__ __forceinline__ void split3_f16(float x, uint32_t& h1, uint32_t& h2, uint32_t& h3) {
    unsigned short a, b, c;
    asm("cvt.rz.f16.f32 %0, %1;" : "=h"(a) : "f"(x));
    const float r1 = x - __half2float(__ushort_as_half(a));
    if (kTerms == 2) asm("cvt.rn.f16.f32 %0, %1;" : "=h"(b) : "f"(r1));
    else asm("cvt.rz.f16.f32 %0, %1;" : "=h"(b) : "f"(r1));
    const float r2 = r1 - __half2float(__ushort_as_half(b));
    asm("cvt.rn.f16.f32 %0, %1;" : "=h"(c) : "f"(r2));
    h1 = a, h2 = b, h3 = c;
}

// Clears the Y of every matrix of a launch of the kernel below.  Launched like it (see launch_matvec_mma_group): lets
// its successor start its set-up at once and waits for its predecessor before it writes.
struct ZeroList {
    float* y[kMmaMaxItems];
    int64_t n[kMmaMaxItems];      // floats (Y is 16-byte aligned)
    int n_items;
};
__global__ void __launch_bounds__(256) zero_kernel(const __grid_constant__ ZeroList z) {
    grid_launch_dependents();
    grid_dependency_wait();
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int it = 0; it < z.n_items; ++it) {
        const int64_t quads = z.n[it] / 4;
        float4* y4 = reinterpret_cast<float4*>(z.y[it]);
        for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < quads; i += (int64_t)gridDim.x * blockDim.x)
            y4[i] = zero;
        if (blockIdx.x == 0 && (int64_t)threadIdx.x < z.n[it] - 4 * quads) z.y[it][4 * quads + threadIdx.x] = 0.f;
    }
}

// Where a CTA is in its range of stages: chunk c, row stage rs (numbered through all matrices of the launch) of
// matrix `it`, sub-stage j of the chunk, ring slot and the parity of the slot's current use.  Stepped without
// divisions.
struct Cursor {
    int c, rs, j, slot, it;
    uint32_t parity;
    __device__ __forceinline__ void init(const MmaParams& p, int64_t first, int spc) {
        const int64_t pair = first / spc;
        j = (int)(first - pair * spc);
        c = (int)(pair / p.total_rs);
        rs = (int)(pair - (int64_t)c * p.total_rs);
        it = 0;
        while (it + 1 < p.n_items && rs >= p.item[it + 1].rs_begin) ++it;
        slot = 0;
        parity = 0;
    }
    __device__ __forceinline__ void step(const MmaParams& p, int spc, int ring) {
        if (++slot == ring) {
            slot = 0;
            parity ^= 1u;
        }
        if (++j == spc) {
            j = 0;
            if (++rs == p.total_rs) {
                rs = 0;
                it = 0;
                ++c;
            } else if (it + 1 < p.n_items && rs >= p.item[it + 1].rs_begin) {
                ++it;
            }
        }
    }
};

// DROP: a build for lw_debug_drop_copy (the producer requests nothing from stage p.drop_stage on, so the wait for
// that stage runs out); the kernels of ordinary calls carry none of it.
template <class T, int NT, bool DROP = false>
__global__ void __launch_bounds__(kMmaThreads, kCtasPerSm) matvec_mma_kernel(const __grid_constant__ MmaParams p,
                                                                             const __grid_constant__ MmaMaps maps) {
    extern __shared__ __align__(128) uint8_t smem[];
    uint64_t* full = reinterpret_cast<uint64_t*>(smem);               // [kMaxRing]
    uint64_t* empty = full + kMaxRing;                                // [kMaxRing]
    volatile int* stop = reinterpret_cast<volatile int*>(smem + 64);  // set when a wait gave up
    constexpr int NB = 8 * NT;                                        // columns held (beyond the batch: zeros)
    constexpr int kPiece = T::kPiece;                                 // bytes of a row's share of a stage
    constexpr int kStageRows = T::kStageRows;                         // (shadows the 256 of the quantised formats)
    constexpr int kStageBytes = kStageRows * kPiece;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int Kx = p.chunk_cols;
    const uint32_t x_pitch = 2u * Kx + kXPad;                         // bytes between columns of a plane
    const uint32_t plane_pitch = NB * x_pitch;
    const int spc = Kx / kStageCols;                                  // stages per (chunk, row stage)
    const int n_rs = p.total_rs;
    const int n_chunks = (int)(p.cols / Kx);
    const int64_t n_stages = (int64_t)n_chunks * n_rs * spc;
    const int64_t first = n_stages * blockIdx.x / gridDim.x, last = n_stages * (blockIdx.x + 1) / gridDim.x;
    const int ring = p.ring;

    // With programmatic dependent launch this kernel may have been placed while its predecessor on the stream
    // (the kernel that clears Y, and through it everything before) is still running: its successor may be placed
    // from now on, and nothing of X or Y is touched before grid_dependency_wait() returns.  Both are no-ops in
    // an ordinary launch.
    grid_launch_dependents();
    if (tid == 0) {
        for (int s = 0; s < kMaxRing; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], kMmaWarps);
        }
        *stop = 0;
        fence_barrier_init();
    }
    __syncthreads();
    volatile unsigned* gen_seen = reinterpret_cast<volatile unsigned*>(smem + 72);   // generation before this CTA arrived

    if (warp == kMmaWarps) {
        // ------------------------------------------------------------- producer (one thread) ---
        if (lane != 0) return;
        if (!p.early_weights) grid_dependency_wait();
        const uint64_t policy = l2_evict_first_policy();
        const int count = (int)(last - first);
        Cursor cur;
        cur.init(p, first, spc);
        int n = 0;
        for (; n < count; ++n, cur.step(p, spc, ring)) {
            if (*stop) break;
            if constexpr (DROP) {
                if (n >= p.drop_stage) break;
            }
            if (n >= ring && !mbar_wait_bounded(&empty[cur.slot], cur.parity ^ 1u)) {   // the slot's previous use
                atomicExch(p.fault, (int)FAULT_BULK_WAIT_TIMEOUT);
                *stop = 1;
                break;
            }
            mbar_expect_tx(&full[cur.slot], kStageBytes);   // a box always delivers all its bytes (zeros past the end)
            if constexpr (T::kF16) {
                // four swizzled 128-byte slices (one per 64-column unit), each all the stage's rows
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    tensor_load_2d(smem + p.w_off + (size_t)cur.slot * kStageBytes + u * MmaF16::kSliceBytes,
                                   &maps.m[cur.it], ((cur.c * spc + cur.j) * 4 + u) * 32,
                                   (cur.rs - p.item[cur.it].rs_begin) * kStageRows, &full[cur.slot], policy);
            } else if constexpr (T::kQ6K || T::kQ2K) {
                // the piece starts at byte kSuper * (stage's column index) of the row: fetch from the 16-byte boundary below
                tensor_load_2d(smem + p.w_off + (size_t)cur.slot * kStageBytes, &maps.m[cur.it],
                               ((T::kSuper * (cur.c * spc + cur.j)) >> 4) << 2,
                               (cur.rs - p.item[cur.it].rs_begin) * kStageRows, &full[cur.slot], policy);
            } else {
                tensor_load_2d(smem + p.w_off + (size_t)cur.slot * kStageBytes, &maps.m[cur.it],
                               (cur.c * spc + cur.j) * T::kXWords, (cur.rs - p.item[cur.it].rs_begin) * kStageRows,
                               &full[cur.slot], policy);
            }
        }
        if (*stop) {
            // the consumers have stopped waiting: make sure nothing is still landing in shared memory (stage m,
            // the latest armed use of its slot, is the (m / ring)-th use)
            for (int m = n - 1; m >= 0 && m >= n - ring; --m)
                if (!mbar_wait_bounded(&full[m % ring], (uint32_t)(m / ring) & 1u))
                    atomicExch(p.fault, (int)FAULT_DRAIN_TIMEOUT);
        }
        return;
    }

    // ------------------------------------------------------------------- compute warps ---
    grid_dependency_wait();
    if (p.self_clear) {
        // this CTA's share of Y, then its arrival at the grid barrier; nobody adds into Y before the barrier
        // has completed (checked before the first flush, by which time it normally has)
        for (int it = 0; it < p.n_items; ++it) {
            const int64_t n = (int64_t)p.batch * p.item[it].rows, quads = n / 4;
            const int64_t q0 = quads * blockIdx.x / gridDim.x, q1 = quads * (blockIdx.x + 1) / gridDim.x;
            float4* y4 = reinterpret_cast<float4*>(p.item[it].Y);
            for (int64_t i = q0 + tid; i < q1; i += kMmaComputeThreads) y4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (blockIdx.x == 0 && tid < (int)(n - 4 * quads)) p.item[it].Y[4 * quads + tid] = 0.f;
        }
        compute_barrier();
        if (tid == 0) {
            unsigned gen, prev;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(gen) : "l"(p.grid_bar + 1) : "memory");
            *gen_seen = gen;
            // release: the stores above (ordered before this thread by the barrier) become visible device-wide to
            // whoever observes the new generation; acquire: the last CTA to arrive has seen everybody's
            asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(prev) : "l"(p.grid_bar) : "memory");
            if (prev == gridDim.x - 1) {
                asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p.grid_bar), "r"(0u) : "memory");
                asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.grid_bar + 1) : "memory");
            }
        }
    }
    bool cleared = !p.self_clear;       // may this warp add into Y yet?
    const int g = lane >> 2, t = lane & 3;
    const uint32_t xs = smem_u32(smem + p.x_off);
    // this lane's B fragments: column g of each group of eight, slots 8 t .. 8 t + 7 of a block of 32
    const uint32_t xlane = xs + g * x_pitch + 16u * t;
    // the warp's 16 rows of a stage; f16: 128-row stages, warps 0-7 take units 0 and 1, warps 8-15 units 2 and 3
    const int mt = T::kF16 ? (warp & 7) : warp;
    const uint32_t wrow = smem_u32(smem + p.w_off) +
                          (T::kF16 ? (uint32_t)(16 * mt + g) * 128u + 8u * (t & 1) : (uint32_t)(16 * warp + g) * kPiece);
    uint32_t sw[4];                                     // f16: the lane's swizzled chunk offsets (see block_step_f16)
#pragma unroll
    for (int i = 0; i < 4; ++i) sw[i] = (uint32_t)(((2 * i + (t >> 1)) ^ g) << 4);

    float y[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) y[nt][i] = 0.f;
    int cur_c = -1, cur_rs = -1, cur_it = 0;
    const float* cur_x = nullptr;

    auto flush = [&]() {
        // add this warp's sums of (chunk, row stage cur_rs) into Y: rows g and g + 8 of the warp's 16, columns
        // 8 nt + 2 t and 8 nt + 2 t + 1
        if (!cleared) {
            // the grid barrier: every CTA has cleared its share of Y once the generation has moved on
            if (lane == 0 && !*stop) {
                const unsigned gen0 = *gen_seen;       // written before the barriers of the first conversion
                unsigned gen = gen0;
                for (uint32_t i = 0; i < kGridPolls && gen == gen0; ++i)
                    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(gen) : "l"(p.grid_bar + 1) : "memory");
                if (gen == gen0) {
                    atomicExch(p.fault, (int)FAULT_GRID_BARRIER_TIMEOUT);
                    *stop = 1;
                }
            }
            __syncwarp();
            cleared = true;
        }
        const MmaItem& m = p.item[cur_it];
        const int64_t r = (int64_t)(cur_rs - m.rs_begin) * kStageRows + 16 * mt + g;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int b = 8 * nt + 2 * t + (i & 1);
                const int64_t rr = r + (i >> 1) * 8;
                if (b < p.batch && rr < m.rows) atomicAdd(m.Y + (int64_t)b * m.rows + rr, y[nt][i]);
                y[nt][i] = 0.f;
            }
    };

    const int count = (int)(last - first);
    Cursor cur;
    cur.init(p, first, spc);
    for (int n = 0; n < count; ++n, cur.step(p, spc, ring)) {
        const int c = cur.c, rs = cur.rs, j = cur.j, slot = cur.slot;
        const MmaItem& mat = p.item[cur.it];
        if (c != cur_c || rs != cur_rs) {
            if (cur_rs >= 0) flush();
            cur_rs = rs;
            cur_it = cur.it;
        }
        if (c != cur_c || mat.X != cur_x) {
            // the chunk's activations as one bf16 (f16) plane per term: plane s, column b.  Inside a block of 32 the order is
            // the one the fragments want: slots 8 q .. 8 q + 3 hold k = 4 q .. 4 q + 3 and slots 8 q + 4 .. 8 q + 7
            // hold k = 16 + 4 q .., so a lane reads both halves of its B operand with one 16-byte load.
            cur_c = c;
            cur_x = mat.X;
            compute_barrier();                          // every warp is done with the previous chunk
            // Only the 256-column pieces this CTA's stages inside the chunk will read (all of them once it has
            // `spc` or more stages here); a piece is 64 quads of each column: one quad per thread and group of
            // eight columns.  All loads are issued before the first conversion.
            const int64_t in_chunk = (int64_t)(mat.same_x_end - rs) * spc - j;    // stages ahead that read this X
            const int left = count - n;
            const int m = (int)(in_chunk < left ? in_chunk : left);
            float4 v[4][NT * kXR];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int jj = (j + q) % spc;
#pragma unroll
                for (int nt = 0; nt < NT * kXR; ++nt) {
                    const int idx = tid + nt * kMmaComputeThreads;
                    const int b = idx >> 6, k4 = jj * (kStageCols / 4) + (idx & 63);
                    v[q][nt] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (q < spc && q < m && b < p.batch)
                        v[q][nt] = __ldg(reinterpret_cast<const float4*>(mat.X + (int64_t)b * p.cols + (int64_t)c * Kx) + k4);
                }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int jj = (j + q) % spc;
                if (q < spc && q < m) {
#pragma unroll
                    for (int nt = 0; nt < NT * kXR; ++nt) {
                        const int idx = tid + nt * kMmaComputeThreads;
                        const int b = idx >> 6, k4 = jj * (kStageCols / 4) + (idx & 63);
                        uint32_t h[3][4];
                        if constexpr (T::kF16) {
                            // f16 terms of x * s, s = the power of two that brings the block's largest magnitude (eight
                            // consecutive lanes hold a block of 32) to 2^14 .. 2^15; 1 / s goes to [block][column]
                            float mx = fmaxf(fmaxf(fabsf(v[q][nt].x), fabsf(v[q][nt].y)), fmaxf(fabsf(v[q][nt].z), fabsf(v[q][nt].w)));
                            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
                            int se = 268 - (int)((__float_as_uint(mx) >> 23) & 0xFFu);      // biased exponent of s
                            se = se < 1 ? 1 : (se > 253 ? 253 : se);
                            const float sc = __uint_as_float((uint32_t)se << 23);
                            if ((lane & 7) == 0)
                                *reinterpret_cast<float*>(smem + p.sx_off + (size_t)(k4 >> 3) * kSxBlockBytes + 4 * b) =
                                    __uint_as_float((uint32_t)(254 - se) << 23);
                            split3_f16(v[q][nt].x * sc, h[0][0], h[1][0], h[2][0]);
                            split3_f16(v[q][nt].y * sc, h[0][1], h[1][1], h[2][1]);
                            split3_f16(v[q][nt].z * sc, h[0][2], h[1][2], h[2][2]);
                            split3_f16(v[q][nt].w * sc, h[0][3], h[1][3], h[2][3]);
                        } else {
                            split3(v[q][nt].x, h[0][0], h[1][0], h[2][0]);
                            split3(v[q][nt].y, h[0][1], h[1][1], h[2][1]);
                            split3(v[q][nt].z, h[0][2], h[1][2], h[2][2]);
                            split3(v[q][nt].w, h[0][3], h[1][3], h[2][3]);
                        }
                        if constexpr (T::kQ2K) {
                            // sums of each 16 activations (four consecutive lanes hold them): [block][half][column]
                            float sum = (v[q][nt].x + v[q][nt].y) + (v[q][nt].z + v[q][nt].w);
                            sum += __shfl_xor_sync(0xffffffffu, sum, 1);
                            sum += __shfl_xor_sync(0xffffffffu, sum, 2);
                            if ((lane & 3) == 0)
                                *reinterpret_cast<float*>(smem + p.sx_off + (size_t)(k4 >> 3) * 128 + ((k4 >> 2) & 1) * 64 + 4 * b) = sum;
                        }
                        if constexpr (T::kHasMin) {
                            // sum of each block of 32 activations (eight consecutive lanes hold one), for the
                            // formats with a per-block offset: [block of the chunk][column]
                            float sum = (v[q][nt].x + v[q][nt].y) + (v[q][nt].z + v[q][nt].w);
                            sum += __shfl_xor_sync(0xffffffffu, sum, 1);
                            sum += __shfl_xor_sync(0xffffffffu, sum, 2);
                            sum += __shfl_xor_sync(0xffffffffu, sum, 4);
                            if ((lane & 7) == 0)
                                *reinterpret_cast<float*>(smem + p.sx_off + (size_t)(k4 >> 3) * kSxBlockBytes + 4 * b) = sum;
                        }
                        const int slot4 = (k4 & ~7) + 2 * (k4 & 3) + ((k4 >> 2) & 1);    // quad of slots the quad of k goes to
                        const uint32_t dst = xs + b * x_pitch + 8u * slot4;
#pragma unroll
                        for (int s = 0; s < kTerms; ++s)
                            asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(dst + s * plane_pitch),
                                         "r"(h[s][0] | (h[s][1] << 16)), "r"(h[s][2] | (h[s][3] << 16))
                                         : "memory");
                    }
                }
            }
            compute_barrier();
        }
        if (!*stop && !mbar_wait_bounded(&full[slot], cur.parity)) {
            if (lane == 0) {
                atomicExch(p.fault, (int)FAULT_BULK_WAIT_TIMEOUT);
                *stop = 1;
            }
        }
        const int64_t r0 = (int64_t)(rs - mat.rs_begin) * kStageRows;
        if (r0 + 16 * mt < mat.rows) {
            const uint32_t row = wrow + (uint32_t)slot * kStageBytes, wt = row + 4u * t;
            const uint32_t tab = smem_u32(smem + p.tab_off) + (uint32_t)warp * T::kTableBytes, tabg = tab + (uint32_t)kTabRow * g;
            const uint32_t sx = smem_u32(smem + p.sx_off) + (uint32_t)(8 * j) * kSxBlockBytes + 8u * t;
            if constexpr (T::kQ6K || T::kQ2K) {
                const uint32_t o = (uint32_t)(T::kSuper * (c * spc + j)) & 15u;      // the piece's offset in the fetched bytes
                T::prepare(row - (uint32_t)g * kPiece + o, tab, lane);
                __syncwarp();
            } else if constexpr (T::kTableBytes > 0) {
                T::prepare(row - (uint32_t)g * kPiece, tab, lane);
                __syncwarp();
            }
            uint32_t xp[NT][kTerms];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int s = 0; s < kTerms; ++s)
                    xp[nt][s] = xlane + 2u * (uint32_t)(j * kStageCols) + s * plane_pitch + nt * 8 * x_pitch;
            if constexpr (T::kQ2K) {
                const uint32_t wo = wt + ((uint32_t)(84 * (c * spc + j)) & 15u);
                const uint32_t tq = tab + (uint32_t)MmaQ2K::kTabRow2 * g, sq = smem_u32(smem + p.sx_off) + (uint32_t)(8 * j) * 128u + 8u * t;
                block_step_q2k<NT, 0, 0>(wo, tq, sq, xp, y);
                block_step_q2k<NT, 0, 1>(wo, tq, sq, xp, y);
                block_step_q2k<NT, 1, 0>(wo, tq, sq, xp, y);
                block_step_q2k<NT, 1, 1>(wo, tq, sq, xp, y);
                block_step_q2k<NT, 2, 0>(wo, tq, sq, xp, y);
                block_step_q2k<NT, 2, 1>(wo, tq, sq, xp, y);
                block_step_q2k<NT, 3, 0>(wo, tq, sq, xp, y);
                block_step_q2k<NT, 3, 1>(wo, tq, sq, xp, y);
            } else if constexpr (T::kQ6K) {
                const uint32_t o = (uint32_t)(210 * (c * spc + j)) & 15u;
                if (o & 2u)
                    stage_q6k<NT, true>(wt + (o & ~3u), tabg, xp, y);
                else
                    stage_q6k<NT, false>(wt + o, tabg, xp, y);
            } else if constexpr (T::kF16) {
                const uint32_t wr = wrow + (uint32_t)slot * kStageBytes;
                if (warp < 8) {
                    block_step_f16<NT, 0, 0>(wr, sw, sx, xp, y);
                    block_step_f16<NT, 0, 1>(wr, sw, sx, xp, y);
                    block_step_f16<NT, 1, 0>(wr, sw, sx, xp, y);
                    block_step_f16<NT, 1, 1>(wr, sw, sx, xp, y);
                } else {
                    block_step_f16<NT, 2, 0>(wr, sw, sx, xp, y);
                    block_step_f16<NT, 2, 1>(wr, sw, sx, xp, y);
                    block_step_f16<NT, 3, 0>(wr, sw, sx, xp, y);
                    block_step_f16<NT, 3, 1>(wr, sw, sx, xp, y);
                }
            } else {
                block_step<T, NT, 0, 0>(wt, row, tabg, sx, xp, y);
                block_step<T, NT, 0, 1>(wt, row, tabg, sx, xp, y);
                block_step<T, NT, 1, 0>(wt, row, tabg, sx, xp, y);
                block_step<T, NT, 1, 1>(wt, row, tabg, sx, xp, y);
                block_step<T, NT, 2, 0>(wt, row, tabg, sx, xp, y);
                block_step<T, NT, 2, 1>(wt, row, tabg, sx, xp, y);
                block_step<T, NT, 3, 0>(wt, row, tabg, sx, xp, y);
                block_step<T, NT, 3, 1>(wt, row, tabg, sx, xp, y);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[slot]);
    }
    if (cur_rs >= 0) flush();
    // this CTA's share of the next launch's outputs (complete, like everything else here, when this grid completes)
    for (int it = 0; it < p.n_next; ++it) {
        const int64_t quads = p.next_n[it] / 4;
        const int64_t q0 = quads * blockIdx.x / gridDim.x, q1 = quads * (blockIdx.x + 1) / gridDim.x;
        float4* y4 = reinterpret_cast<float4*>(p.next_y[it]);
        for (int64_t i = q0 + tid; i < q1; i += kMmaComputeThreads) y4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (blockIdx.x == 0 && tid < (int)(p.next_n[it] - 4 * quads)) p.next_y[it][4 * quads + tid] = 0.f;
    }
}

template <class T, int NT, bool DROP = false>
int launch_mma(const MmaParams& p, const MmaMaps& maps, int grid, size_t smem_bytes, bool overlap,
               cudaStream_t stream) {
    // self-clearing launches are cooperative (their CTAs wait for one another) and ordinary in stream order
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return (int)e;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        e = cudaFuncSetAttribute(matvec_mma_kernel<T, NT, DROP>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemPerCta);
        if (e != cudaSuccess) return (int)e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kMmaThreads);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    // (a cooperative launch that also carries the programmatic attribute works but measured slower than the
    // clearing-kernel chain: 2.27 against 1.95 ms per 8B q4_0 step at 8 columns)
    cudaLaunchAttribute attr[1];
    if (p.self_clear) {
        attr[0].id = cudaLaunchAttributeCooperative;
        attr[0].val.cooperative = 1;
    } else {
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
    }
    cfg.attrs = attr;
    cfg.numAttrs = (p.self_clear || overlap) ? 1 : 0;
    return (int)cudaLaunchKernelEx(&cfg, matvec_mma_kernel<T, NT, DROP>, p, maps);
}

// cuTensorMapEncodeTiled through the runtime's driver entry point lookup (no link against the driver library)
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            f = nullptr;
        return reinterpret_cast<EncodeTiledFn>(f);
    }();
    return fn;
}

int mma_stage_rows(int fmt) { return fmt == LW_F16 ? MmaF16::kStageRows : kStageRows; }

// The weight matrix as a 2-D tensor of 32-bit words (row_bytes / 4 per row, `rows` rows) with boxes of one stage;
// f16: boxes of one 128-byte slice of a stage's rows, written with the 128-byte swizzle.
bool make_weight_map(CUtensorMap* map, int fmt, const void* W, int64_t rows, int64_t row_bytes, int piece_bytes) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const bool f16 = fmt == LW_F16;
    const cuuint64_t dims[2] = {(cuuint64_t)(row_bytes / 4), (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)(f16 ? 32 : piece_bytes / 4), (cuuint32_t)mma_stage_rows(fmt)};
    const cuuint32_t elem[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void*>(W), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, f16 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int mma_sm_count() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
    return n;
}

// Shared-memory plan of a launch: the largest chunk (1024, 512, 256 columns) that divides cols and leaves room
// for at least two stages.  Returns false if nothing fits.
bool mma_plan(int fmt, int64_t cols, int nt, int& chunk_cols, int& ring, size_t& x_bytes, size_t& stage_bytes,
              size_t& extra_bytes) {
    const int piece = fmt == LW_Q8_0   ? MmaQ80::kPiece
                      : fmt == LW_Q4_0 ? MmaQ40::kPiece
                      : fmt == LW_Q4_K ? MmaQ4K::kPiece
                      : fmt == LW_Q5_K ? MmaQ5K::kPiece
                      : fmt == LW_Q4_1 ? MmaLegacy<LW_Q4_1>::kPiece
                      : fmt == LW_Q5_0 ? MmaLegacy<LW_Q5_0>::kPiece
                      : fmt == LW_Q5_1 ? MmaLegacy<LW_Q5_1>::kPiece
                      : fmt == LW_Q6_K ? MmaQ6K::kPiece
                      : fmt == LW_Q2_K ? MmaQ2K::kPiece
                                       : MmaF16::kPiece;
    stage_bytes = (size_t)mma_stage_rows(fmt) * piece;
    // q4_K: block sums of the activations (64 bytes per block of a chunk of up to 1024 columns) and the warps' tables
    extra_bytes = fmt == LW_Q2_K ? (size_t)(1024 / 32) * 128 + (size_t)kMmaWarps * MmaQ2K::kTableBytes
                  : (fmt == LW_Q4_K || fmt == LW_Q5_K || fmt == LW_Q6_K)
                      ? (size_t)(1024 / 32) * kSxBlockBytes + (size_t)kMmaWarps * MmaQ4K::kTableBytes
                      : ((fmt == LW_F16 || fmt == LW_Q4_1 || fmt == LW_Q5_1) ? (size_t)(1024 / 32) * kSxBlockBytes : 0);
    // (f16: up to 1 KB more goes into aligning the swizzled stages)
    const size_t budget = kSmemPerCta - kMmaHeader - extra_bytes - (fmt == LW_F16 ? 1024 : 0);
    // the largest chunk that leaves room for two stages (q8_0, 458752 x 4096, 8 columns: 0.40 ms with chunks of
    // 1024 columns and two 68 KB stages against 0.49 ms with chunks of 256 and three)
    for (int kx = 1024; kx >= 256; kx /= 2) {
        if (cols % kx != 0) continue;
        x_bytes = (size_t)kTerms * 8 * nt * (2 * kx + kXPad);
        if (x_bytes + 2 * stage_bytes > budget) continue;
        size_t n = (budget - x_bytes) / stage_bytes;
        ring = (int)(n > (size_t)kMaxRing ? kMaxRing : n);
        chunk_cols = kx;
        return true;
    }
    return false;
}

}  // namespace

bool matvec_mma_supported(int fmt, int64_t rows, int64_t cols, int batch) {
    if (fmt != LW_Q4_0 && fmt != LW_Q8_0 && fmt != LW_Q4_K && fmt != LW_Q5_K && fmt != LW_F16 && fmt != LW_Q4_1 &&
        fmt != LW_Q5_0 && fmt != LW_Q5_1 && fmt != LW_Q6_K && fmt != LW_Q2_K)
        return false;
    if (fmt == LW_Q6_K && cols % 2048 != 0) return false;      // 210-byte super-blocks: rows must be whole 16-byte units
    if (fmt == LW_Q2_K && cols % 1024 != 0) return false;      // 84-byte super-blocks likewise
    if (batch < 2 || batch > 16) return false;
    if (cols % kStageCols != 0) return false;
    return rows >= 1 && rows <= (int64_t)1 << 30;
}

bool matvec_mma_group_supported(int fmt, int64_t cols, int n_items, const int64_t* rows, int batch) {
    if (n_items < 1 || n_items > kMmaMaxItems) return false;
    int64_t total_rs = 0;
    for (int i = 0; i < n_items; ++i) {
        if (!matvec_mma_supported(fmt, rows[i], cols, batch)) return false;
        total_rs += (rows[i] + mma_stage_rows(fmt) - 1) / mma_stage_rows(fmt);
    }
    return total_rs * (cols / kStageCols) < ((int64_t)1 << 31);
}

// Up to kMmaMaxItems matrices of one format and width in one launch, each with its own X and Y (matrices that
// share an X pointer and follow one another share its converted copy).  Arguments are validated by the caller;
// returns a cudaError_t as int.
// overlap: 0 ordinary launches; 1 programmatic dependent launch (set-up overlaps the previous kernel's end);
// 2 the same, and the weight copies start before the previous kernel has completed.  self_clear: one cooperative
// launch whose CTAs clear Y themselves (no clearing kernel, no programmatic launch).
// pre_cleared: the launch before this one on the stream has cleared these outputs (no clearing of any kind here);
// n_next / next_y / next_n: outputs of the launch after this one, to be cleared by this one at its end.
int launch_matvec_mma_group(int fmt, int64_t cols, int n_items, const void* const* W, const int64_t* rows,
                            const float* const* X, float* const* Y, int batch, int overlap, bool self_clear,
                            cudaStream_t stream, bool pre_cleared, int n_next, float* const* next_y,
                            const int64_t* next_n) {
    int* fault = device_fault_word();
    if (!fault) return (int)cudaErrorInvalidValue;
    if (pre_cleared) self_clear = false;
    {
        // The grid barrier of the self-clearing form is one pair of words per device: it relies on two such
        // launches never running at the same time, which holds because each needs every SM to itself (cooperative
        // launch, one CTA per SM, more than half an SM's shared memory per CTA).  Should a plan ever need less, take
        // the clearing kernel instead.
        int cc = 0, rg = 0;
        size_t xb = 0, sb = 0, eb = 0;
        if (!mma_plan(fmt, cols, batch > 8 ? 2 : 1, cc, rg, xb, sb, eb)) return (int)cudaErrorInvalidValue;
        if (2 * ((kMmaHeader + xb + eb + 127) / 128 * 128 + (size_t)rg * sb + 1024) <= 228 * 1024 || kCtasPerSm != 1)   // (f16's alignment slack only adds)
            self_clear = false;
    }
    unsigned* grid_bar = nullptr;
    if (self_clear && cudaGetSymbolAddress(reinterpret_cast<void**>(&grid_bar), g_mma_grid_barrier) != cudaSuccess)
        return (int)cudaErrorInvalidValue;
    // the kernel adds every (chunk, row stage) share into Y: clear it first (Y is 16-byte aligned)
    if (!self_clear && !pre_cleared) {
        ZeroList z{};
        int64_t most = 0;
        for (int i = 0; i < n_items; ++i) {
            z.y[i] = Y[i];
            z.n[i] = (int64_t)batch * rows[i];
            if (z.n[i] > most) most = z.n[i];
        }
        z.n_items = n_items;
        int64_t blocks = (most / 4 + 255) / 256;
        if (blocks < 1) blocks = 1;
        if (blocks > 4 * mma_sm_count()) blocks = 4 * mma_sm_count();
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)blocks);
        cfg.blockDim = dim3(256);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = overlap ? 1 : 0;
        const cudaError_t e = cudaLaunchKernelEx(&cfg, zero_kernel, z);
        if (e != cudaSuccess) return (int)e;
    }
    const int nt = batch > 8 ? 2 : 1;
    MmaParams p{};
    size_t x_bytes = 0, stage_bytes = 0, extra_bytes = 0;
    if (!mma_plan(fmt, cols, nt, p.chunk_cols, p.ring, x_bytes, stage_bytes, extra_bytes)) return (int)cudaErrorInvalidValue;
    alignas(64) MmaMaps maps;
    const int64_t row_bytes = (int64_t)lw_row_bytes(fmt, cols);
    int rs = 0;
    for (int i = 0; i < n_items; ++i) {
        p.item[i].X = X[i];
        p.item[i].Y = Y[i];
        p.item[i].rows = rows[i];
        p.item[i].rs_begin = rs;
        rs += (int)((rows[i] + mma_stage_rows(fmt) - 1) / mma_stage_rows(fmt));
        if (!make_weight_map(&maps.m[i], fmt, W[i], rows[i], row_bytes, (int)(stage_bytes / mma_stage_rows(fmt))))
            return (int)cudaErrorInvalidValue;
    }
    for (int i = n_items - 1; i >= 0; --i)          // end of the run of matrices that read the same X
        p.item[i].same_x_end = (i + 1 < n_items && X[i + 1] == X[i]) ? p.item[i + 1].same_x_end : (i + 1 < n_items ? p.item[i + 1].rs_begin : rs);
    for (int i = n_items; i < kMmaMaxItems; ++i) maps.m[i] = maps.m[0];
    p.n_items = n_items;
    p.total_rs = rs;
    p.fault = fault;
    p.cols = cols;
    p.batch = batch;
    p.early_weights = overlap >= 2 && !self_clear;
    p.self_clear = self_clear ? 1 : 0;
    p.grid_bar = grid_bar;
    p.x_off = kMmaHeader;
    p.sx_off = (uint32_t)(kMmaHeader + x_bytes);
    p.tab_off = p.sx_off + (uint32_t)(fmt == LW_Q2_K ? (1024 / 32) * 128
                                      : (fmt == LW_Q4_K || fmt == LW_Q5_K || fmt == LW_Q6_K) ? (1024 / 32) * kSxBlockBytes : 0);
    // the stages: 128-byte aligned; f16's swizzle pattern is one of address bits, so its stages start on 1 KB
    const size_t w_align = fmt == LW_F16 ? 1024 : 128;
    p.w_off = (uint32_t)((kMmaHeader + x_bytes + extra_bytes + w_align - 1) / w_align * w_align);
    const size_t smem_bytes = p.w_off + (size_t)p.ring * stage_bytes;
    const int64_t n_stages = (cols / kStageCols) * (int64_t)rs;
    int grid = kCtasPerSm * mma_sm_count();
    if ((int64_t)grid > n_stages && !self_clear) grid = (int)n_stages;   // self-clearing: every SM, so launches never overlap
    p.drop_stage = -1;
    p.n_next = n_next;
    for (int i = 0; i < n_next; ++i) {
        p.next_y[i] = next_y[i];
        p.next_n[i] = next_n[i];
    }
    if (fmt == LW_Q4_0 && nt == 1) {
        // testing aid: a pending lw_debug_drop_copy request is consumed by this launch
        const int drop = take_drop_unit();
        if (drop >= 0) {
            p.drop_stage = drop;
            return launch_mma<MmaQ40, 1, true>(p, maps, grid, smem_bytes, overlap != 0, stream);
        }
    }
    if (fmt == LW_Q4_0)
        return nt == 1 ? launch_mma<MmaQ40, 1>(p, maps, grid, smem_bytes, overlap != 0, stream)
                       : launch_mma<MmaQ40, 2>(p, maps, grid, smem_bytes, overlap != 0, stream);
    if (fmt == LW_Q4_K)
        return nt == 1 ? launch_mma<MmaQ4K, 1>(p, maps, grid, smem_bytes, overlap != 0, stream)
                       : launch_mma<MmaQ4K, 2>(p, maps, grid, smem_bytes, overlap != 0, stream);
    if (fmt == LW_Q5_K)
        return nt == 1 ? launch_mma<MmaQ5K, 1>(p, maps, grid, smem_bytes, overlap != 0, stream)
                       : launch_mma<MmaQ5K, 2>(p, maps, grid, smem_bytes, overlap != 0, stream);
    if (fmt == LW_F16)
        return nt == 1 ? launch_mma<MmaF16, 1>(p, maps, grid, smem_bytes, overlap != 0, stream)
                       : launch_mma<MmaF16, 2>(p, maps, grid, smem_bytes, overlap != 0, stream);
    if (fmt == LW_Q2_K)
        return nt == 1 ? launch_mma<MmaQ2K, 1>(p, maps, grid, smem_bytes, overlap != 0, stream)
                       : launch_mma<MmaQ2K, 2>(p, maps, grid, smem_bytes, overlap != 0, stream);
    if (fmt == LW_Q6_K)
        return nt == 1 ? launch_mma<MmaQ6K, 1>(p, maps, grid, smem_bytes, overlap != 0, stream)
                       : launch_mma<MmaQ6K, 2>(p, maps, grid, smem_bytes, overlap != 0, stream);
    if (fmt == LW_Q4_1)
        return nt == 1 ? launch_mma<MmaLegacy<LW_Q4_1>, 1>(p, maps, grid, smem_bytes, overlap != 0, stream)
                       : launch_mma<MmaLegacy<LW_Q4_1>, 2>(p, maps, grid, smem_bytes, overlap != 0, stream);
    if (fmt == LW_Q5_0)
        return nt == 1 ? launch_mma<MmaLegacy<LW_Q5_0>, 1>(p, maps, grid, smem_bytes, overlap != 0, stream)
                       : launch_mma<MmaLegacy<LW_Q5_0>, 2>(p, maps, grid, smem_bytes, overlap != 0, stream);
    if (fmt == LW_Q5_1)
        return nt == 1 ? launch_mma<MmaLegacy<LW_Q5_1>, 1>(p, maps, grid, smem_bytes, overlap != 0, stream)
                       : launch_mma<MmaLegacy<LW_Q5_1>, 2>(p, maps, grid, smem_bytes, overlap != 0, stream);
    return nt == 1 ? launch_mma<MmaQ80, 1>(p, maps, grid, smem_bytes, overlap != 0, stream)
                   : launch_mma<MmaQ80, 2>(p, maps, grid, smem_bytes, overlap != 0, stream);
}

int launch_matvec_mma(int fmt, const void* W, int64_t rows, int64_t cols, const float* X, float* Y, int batch,
                      int overlap, bool self_clear, cudaStream_t stream) {
    return launch_matvec_mma_group(fmt, cols, 1, &W, &rows, &X, &Y, batch, overlap, self_clear, stream, false, 0, nullptr,
                                   nullptr);
}

}  // namespace lw
