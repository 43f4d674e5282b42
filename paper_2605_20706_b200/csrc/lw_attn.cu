// Decode attention of one query token over a block-quantised KV cache: the cache's blocks are
// decoded in registers by the same per-format routines the mat-vec kernels use (the paper notes that
// its decode routines serve the KV cache in attention too, Sec 3.3), the scores never
// leave the chip (online softmax, paper Sec 3.2 "FlashAttention": one running maximum, exponential sum
// and output accumulator per query row while the cached K/V rows stream by).
//
// The cached positions are split over the grid (the cache is read exactly once, every SM busy);
// each part leaves an unnormalised partial (running maximum, exponential sum, accumulator) in the
// caller's workspace and a second small kernel merges the parts.
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>

#include "lw_formats.cuh"
#include "lw_internal.h"

namespace lw {
namespace {

constexpr int kAttnThreads = 128;
constexpr int kAttnWarps = kAttnThreads / 32;
constexpr int kMaxParts = 256;          // upper bound of partial results per head
constexpr float kNegInf = -INFINITY;

// Number of parts the positions are cut into by the general kernel: at least 64 positions per part,
// about four CTAs per SM over all KV heads and head batches.
int general_parts(int64_t n_kv_head, int64_t head_batches, int64_t n_pos, int sm_count) {
    const int64_t by_len = (n_pos + 63) / 64;
    const int64_t by_grid = (4LL * sm_count + n_kv_head * head_batches - 1) / (n_kv_head * head_batches);
    int64_t parts = by_len < by_grid ? by_len : by_grid;
    if (parts < 1) parts = 1;
    if (parts > kMaxParts) parts = kMaxParts;
    return (int)parts;
}

struct AttnParams {
    const uint8_t* K;
    const uint8_t* V;
    const float* q;       // [n_head][head_dim]
    float* out;           // [n_head][head_dim]
    float* ws;            // [n_head][parts][head_dim + 2]: accumulator, then maximum, then sum
    int n_head, n_kv_head, n_rep, head_dim;
    int n_pos, parts;
    int64_t row_bytes;    // bytes of one cached position (all KV heads)
    float scale;
};

// Merge of two online-softmax states (m, l, acc) of the same query row.
template <int N>
__device__ __forceinline__ void merge_state(float& m, float& l, float (&acc)[N], float m2, float l2, const float (&acc2)[N]) {
    const float mn = fmaxf(m, m2);
    const float a = (m == kNegInf) ? 0.f : __expf(m - mn);
    const float b = (m2 == kNegInf) ? 0.f : __expf(m2 - mn);
    l = l * a + l2 * b;
#pragma unroll
    for (int i = 0; i < N; ++i) acc[i] = acc[i] * a + acc2[i] * b;
    m = mn;
}

// General kernel: any n_rep (in batches of NREP query heads), head_dim in {32, 64, 128, 256}.
// grid = (parts, n_kv_head, head batches).  A lane owns 8 consecutive dims of a row; head_dim / 8
// lanes cover one cached position, so a warp takes 32 / (head_dim / 8) positions at a time.
template <class Fmt, int NREP>
__global__ void __launch_bounds__(kAttnThreads) attn_decode_general_kernel(const AttnParams p) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the merge kernel may become resident and wait
    const int L = p.head_dim >> 3;                 // lanes per position
    const int sub = lane / L, j = lane - sub * L;  // which of the warp's positions, which 8 dims
    const int per_warp = 32 / L;
    const int g = blockIdx.y;
    const int h0 = g * p.n_rep + blockIdx.z * NREP;                 // first query head of this batch
    const int heads = min(NREP, p.n_rep - (int)blockIdx.z * NREP);  // heads of this batch
    const int chunk = (p.n_pos + p.parts - 1) / p.parts;
    const int t_begin = blockIdx.x * chunk;
    const int t_end = min(p.n_pos, t_begin + chunk);

    float qr[NREP][8];
#pragma unroll
    for (int r = 0; r < NREP; ++r) {
        const int h = h0 + (r < heads ? r : 0);
        const float4 a = __ldg(reinterpret_cast<const float4*>(p.q + (int64_t)h * p.head_dim + 8 * j));
        const float4 b = __ldg(reinterpret_cast<const float4*>(p.q + (int64_t)h * p.head_dim + 8 * j + 4));
        const float s = (r < heads) ? p.scale : 0.f;
        qr[r][0] = a.x * s, qr[r][1] = a.y * s, qr[r][2] = a.z * s, qr[r][3] = a.w * s;
        qr[r][4] = b.x * s, qr[r][5] = b.y * s, qr[r][6] = b.z * s, qr[r][7] = b.w * s;
    }
    float m[NREP], l[NREP], acc[NREP][8];
#pragma unroll
    for (int r = 0; r < NREP; ++r) {
        m[r] = kNegInf, l[r] = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[r][i] = 0.f;
    }
    const int64_t k0 = (int64_t)g * p.head_dim + 8 * j;
    // the trip count is the same for every lane of a warp (the shuffles below are warp-wide); a lane whose
    // position falls past the end decodes the last valid row and drops the result
    for (int tb = t_begin + warp * per_warp; tb < t_end; tb += kAttnWarps * per_warp) {
        const bool valid = tb + sub < t_end;
        const int t = valid ? tb + sub : t_end - 1;
        float kf[8], vf[8];
        Fmt::decode8(p.K + (int64_t)t * p.row_bytes, k0, kf);
        Fmt::decode8(p.V + (int64_t)t * p.row_bytes, k0, vf);
#pragma unroll
        for (int r = 0; r < NREP; ++r) {
            float s = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) s = fmaf(qr[r][i], kf[i], s);
            for (int o = 1; o < L; o <<= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (valid) {
                const float mn = fmaxf(m[r], s);
                const float corr = __expf(m[r] - mn);          // exp(-inf) = 0 on the first position
                const float pr = __expf(s - mn);
                l[r] = l[r] * corr + pr;
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[r][i] = fmaf(pr, vf[i], acc[r][i] * corr);
                m[r] = mn;
            }
        }
    }
    // merge the warp's position slots (lanes with equal j), then the warps through shared memory
#pragma unroll
    for (int r = 0; r < NREP; ++r) {
        for (int o = L; o < 32; o <<= 1) {
            const float m2 = __shfl_xor_sync(0xffffffffu, m[r], o);
            const float l2 = __shfl_xor_sync(0xffffffffu, l[r], o);
            float a2[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) a2[i] = __shfl_xor_sync(0xffffffffu, acc[r][i], o);
            merge_state(m[r], l[r], acc[r], m2, l2, a2);
        }
    }
    __shared__ float sm_acc[kAttnWarps][NREP][256];
    __shared__ float sm_ml[kAttnWarps][NREP][2];
    if (sub == 0) {
#pragma unroll
        for (int r = 0; r < NREP; ++r) {
#pragma unroll
            for (int i = 0; i < 8; ++i) sm_acc[warp][r][8 * j + i] = acc[r][i];
            if (j == 0) sm_ml[warp][r][0] = m[r], sm_ml[warp][r][1] = l[r];
        }
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < heads * p.head_dim; idx += kAttnThreads) {
        const int r = idx / p.head_dim, d = idx - r * p.head_dim;
        float mm = kNegInf;
        for (int w = 0; w < kAttnWarps; ++w) mm = fmaxf(mm, sm_ml[w][r][0]);
        float a = 0.f, ll = 0.f;
        for (int w = 0; w < kAttnWarps; ++w) {
            const float f = (sm_ml[w][r][0] == kNegInf) ? 0.f : __expf(sm_ml[w][r][0] - mm);
            a = fmaf(sm_acc[w][r][d], f, a);
            ll = fmaf(sm_ml[w][r][1], f, ll);
        }
        float* dst = p.ws + ((int64_t)(h0 + r) * p.parts + blockIdx.x) * (p.head_dim + 2);
        dst[d] = a;
        if (d == 0) dst[p.head_dim] = mm, dst[p.head_dim + 1] = ll;
    }
}

// Merge of the parts: grid = (n_head, head_dim / 32); a CTA owns 32 dims of one head.  Thread s first
// turns part s's maximum into its weight exp(m_s - max) (kept in shared memory, with the weighted
// exponential sums added up on the way); then 16 lanes of two dims each x 16 groups share out the
// parts, every load independent of the others, and the groups' sums meet in shared memory.
__global__ void __launch_bounds__(256) attn_merge_kernel(const float* __restrict__ ws, float* __restrict__ out, int parts,
                                                          int head_dim) {
    __shared__ float weight[kMaxParts];
    __shared__ float red[8], red_l[8];
    __shared__ float2 sums[256];
    const int h = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int stride = head_dim + 2;
    const float* base = ws + (int64_t)h * parts * stride;
    const int x = tid & 15, y = tid >> 4;
    const float* col = base + 32 * blockIdx.y + 2 * x;
    // launched early (programmatic dependent launch): wait here until the kernel that writes the parts is done
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // every load of this thread is issued before anything is computed: one trip to L2 for all of them
    constexpr int kPerThread = kMaxParts / 16;
    float2 v[kPerThread];
#pragma unroll
    for (int k = 0; k < kPerThread; ++k) {
        const int s = y + 16 * k;
        v[k] = s < parts ? *reinterpret_cast<const float2*>(col + (int64_t)s * stride) : make_float2(0.f, 0.f);
    }
    const float ms = tid < parts ? base[(int64_t)tid * stride + head_dim] : kNegInf;
    const float ls = tid < parts ? base[(int64_t)tid * stride + head_dim + 1] : 0.f;
    float mm = ms;
    for (int o = 16; o > 0; o >>= 1) mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, o));
    if (lane == 0) red[warp] = mm;
    __syncthreads();
    mm = red[0];
    for (int w = 1; w < 8; ++w) mm = fmaxf(mm, red[w]);
    const float f = (ms == kNegInf) ? 0.f : __expf(ms - mm);
    weight[tid] = f;
    float ll = ls * f;
    for (int o = 16; o > 0; o >>= 1) ll += __shfl_xor_sync(0xffffffffu, ll, o);
    if (lane == 0) red_l[warp] = ll;
    __syncthreads();
    float a0 = 0.f, a1 = 0.f;
#pragma unroll
    for (int k = 0; k < kPerThread; ++k) {
        const float fs = weight[y + 16 * k];
        a0 = fmaf(v[k].x, fs, a0), a1 = fmaf(v[k].y, fs, a1);
    }
    sums[tid] = make_float2(a0, a1);
    __syncthreads();
    if (y == 0) {
        for (int g = 1; g < 16; ++g) a0 += sums[16 * g + x].x, a1 += sums[16 * g + x].y;
        float total = 0.f;
        for (int w = 0; w < 8; ++w) total += red_l[w];
        const float inv = 1.f / total;
        *reinterpret_cast<float2*>(out + (int64_t)h * head_dim + 32 * blockIdx.y + 2 * x) = make_float2(a0 * inv, a1 * inv);
    }
}

// The merge is launched with the programmatic-serialisation attribute: its CTAs may become resident while
// the kernel before it on the stream is finishing, and wait for that kernel's results at griddepcontrol.wait.
cudaError_t launch_merge(const float* ws, float* out, int n_head, int parts, int head_dim, cudaStream_t stream) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(n_head, head_dim / 32);
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, attn_merge_kernel, ws, out, parts, head_dim);
}

// ---------------------------------------------------------------------------------------------
// Tensor-core kernel (grouped-query shapes: head_dim 64 or 128, 1, 2, 4 or 8 KV heads, cache rows a whole number
// of 16-byte pieces; four query heads of a KV head per CTA row, further heads in further CTA rows).
//
// With four query heads sharing every cached row, the fp32 multiply-adds per cached byte exceed what the
// FMA pipes deliver at HBM speed, so both contractions run as m16n8k16 f16 MMAs with fp32 accumulation:
//   scores   S^T[t][n]  = sum_d K[t][d] * Q^T[d][n]      A = 16 cached positions x 16 dims, B = query
//   output   O[n][dim]  = sum_t P[n][t] * V[t][dim]      A = probabilities,                B = values
// where the n index is (query head, high | low part): the query and the probabilities are split into
// two f16 numbers (value = high + low) so that their rounding to f16 costs 2^-22, not 2^-11, and the
// integer codes of the cache are exact in f16; the block scales d are applied in fp32 -- to the score
// sums per 32-dim block, and to the probabilities (per position and block) before the second product.
// One CTA per SM takes a contiguous range of positions for all KV heads; a producer warp copies each stage
// as groups of rows (bulk copies on mbarriers) with padding chosen so that the K and V fragment loads are
// free of bank conflicts (host-side simulation, attn_bank_conflicts; the conflicts a profiler still counts,
// about 15 % of the shared-memory wavefronts at 32768 positions, belong to the other shared-memory traffic);
// compute warp w serves KV head w mod n_kv_head and the tiles TPW * (w / n_kv_head) ... of the stage.
//
// Why mma.sync and not tcgen05.  The M of both products is 8 (four query heads x high | low part) per KV
// head.  tcgen05.mma needs M = 64 or 128 with A read through a shared-memory descriptor in its canonical
// (swizzled core-matrix) layout and D in TMEM.  For the code-valued caches (q8_0, q4_0) A would first have to
// be decoded into that layout -- a second pass over every byte through shared memory, which is what the
// register decode avoids.  For the f16 cache the scores could take a K tile as A as stored (a tensor-map
// copy can produce the layout), but the second product has the cached positions as its K dimension and
// the probabilities as the operand that changes every tile: they would have to go register -> shared memory ->
// tensor core each tile, with the accumulator read back from TMEM for every rescale, and M padded from 8
// to 64.  The f16 kernel as it stands is bound by its copies (its time with the arithmetic switched off is
// within 2 % of the full kernel), so there is nothing for a faster contraction to win there.
struct AttnMmaParams {
    const uint8_t* K;
    const uint8_t* V;
    const float* q;
    float* ws;
    int n_kv_head, n_rep, n_pos;
    int chunk;            // positions per CTA, a multiple of the stage's positions
    int parts;            // CTAs
    int row_bytes, gs_k, gs_v;   // bytes of a cached row in HBM; of a group of rows (one copy) of K / V in shared memory
    int stages;
    float scale;
    int* fault;           // device word that records a bounded wait giving up
};

__device__ __forceinline__ void mma_m16n8k16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                             uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Same product when only rows 0-7 of A are in use (rows 8-15 are zero): two live accumulators.
__device__ __forceinline__ void mma_m16n8k16_top(float& d0, float& d1, uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
    float t2, t3;
    asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%5}, {%7,%8}, {%0,%1,%9,%9};"
        : "+f"(d0), "+f"(d1), "=f"(t2), "=f"(t3)
        : "r"(a0), "r"(0u), "r"(a2), "r"(b0), "r"(b1), "f"(0.f));
}

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
    uint32_t y;
    asm("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}

constexpr uint32_t kAttnWaitTries = 1u << 16;          // each try may sleep up to kAttnWaitNs: about 0.1 s in all
constexpr uint32_t kAttnWaitNs = 2000;

__device__ __forceinline__ void attn_mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void attn_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait on an mbarrier phase; false when the limit ran out.
__device__ __forceinline__ bool attn_mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kAttnWaitTries; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity), "r"(kAttnWaitNs)
            : "memory");
        if (ok) return true;
    }
    return false;
}
// 1-D bulk copy global -> shared, completion counted in bytes on the mbarrier; all three 16-byte granular.
__device__ __forceinline__ void attn_bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

// Loads from shared-memory byte addresses (32-bit shared window addresses keep the pointers in one register).
__device__ __forceinline__ uint32_t lds32(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t a) {
    uint2 v;
    asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
    return v;
}
__device__ __forceinline__ float lds_half(uint32_t a) {
    unsigned short h;
    asm volatile("ld.shared.b16 %0, [%1];" : "=h"(h) : "r"(a));
    return __half2float(__ushort_as_half(h));
}

// 32-bit word at a 2-byte-aligned shared address: one load when the address is a multiple of four,
// else the two aligned words around it and a byte permute.
template <bool MISALIGNED>
__device__ __forceinline__ uint32_t lds_word(uint32_t a) {
    if constexpr (!MISALIGNED) {
        return lds32(a);
    } else {
        return __byte_perm(lds32(a - 2), lds32(a + 2), 0x5432);
    }
}

// Bytes (b0, b1) resp. (b2, b3) of a word of small unsigned integers -> two f16 numbers minus `bias`:
// 0x64 above a byte u is the f16 number 1024 + u, and the subtraction is exact.
__device__ __forceinline__ uint32_t bytes01_to_h2(uint32_t w, uint32_t bias_h2) {
    const uint32_t m = __byte_perm(w, 0x64646464u, 0x4140);
    __half2 r = __hsub2(*reinterpret_cast<const __half2*>(&m), *reinterpret_cast<const __half2*>(&bias_h2));
    return *reinterpret_cast<uint32_t*>(&r);
}
__device__ __forceinline__ uint32_t bytes23_to_h2(uint32_t w, uint32_t bias_h2) {
    const uint32_t m = __byte_perm(w, 0x64646464u, 0x4342);
    __half2 r = __hsub2(*reinterpret_cast<const __half2*>(&m), *reinterpret_cast<const __half2*>(&bias_h2));
    return *reinterpret_cast<uint32_t*>(&r);
}

// (high, low) f16 pair of an fp32 number: x = high + low up to 2^-22 |x|.
__device__ __forceinline__ uint32_t split_hi_lo(float x) {
    const __half hi = __float2half_rn(x);
    const __half lo = __float2half_rn(x - __half2float(hi));
    return (uint32_t)__half_as_ushort(hi) | ((uint32_t)__half_as_ushort(lo) << 16);
}

// The same split for two numbers at once, with the two-wide conversions: xa = (high, low) of a, xb of b.
__device__ __forceinline__ void split_hi_lo2(float a, float b, uint32_t& xa, uint32_t& xb) {
    uint32_t hi, lo;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(hi) : "f"(b), "f"(a));        // upper half from the first operand
    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&hi));
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(lo) : "f"(b - f.y), "f"(a - f.x));
    xa = __byte_perm(hi, lo, 0x5410), xb = __byte_perm(hi, lo, 0x7632);
}

__device__ __forceinline__ float fast_exp2(float x) {      // 2^x, 2^-inf = 0; relative error about 2^-22
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

constexpr int kFmtF16 = 0, kFmtQ8 = 1, kFmtQ4 = 2;

// A stage lands in shared memory as groups of consecutive cached rows, one bulk copy per group (a copy costs
// about 60 ns whatever its size, so rows of 1-2 KB are moved four resp. two at a time), each group followed
// by a few bytes of padding.  Which position of a 16-position tile plays which row of the MMA tile is free;
// it is chosen so that the rows a fragment load touches at once come from different groups (or from rows of
// a group that sit in different banks), which together with the padding keeps the loads free of bank conflicts.
__host__ __device__ constexpr int attn_group_rows(int fmt) { return fmt == kFmtF16 ? 2 : 4; }
// Position (0..15) within its tile of MMA tile row m.
__host__ __device__ constexpr int attn_sigma(int fmt, int m) {
    return fmt == kFmtF16 ? 2 * (m & 7) + (m >> 3) : 4 * ((m & 7) >> 1) + 2 * (m >> 3) + (m & 1);
}
// Byte offset of stage row `row` in a region whose groups of `group_rows` rows are `group_stride` bytes apart.
__host__ __device__ constexpr int attn_row_offset(int row, int group_rows, int group_stride, int row_bytes) {
    return (row / group_rows) * group_stride + (row % group_rows) * row_bytes;
}
constexpr float kPdScale = 256.f;       // probabilities x value scale are kept 2^8 up, clear of f16 subnormals

template <int FMT, int HD, int TPW>      // TPW: 16-position tiles a warp takes per stage (their work interleaves)
__global__ void __launch_bounds__(288, 1) attn_decode_mma_kernel(const AttnMmaParams p) {
    extern __shared__ __align__(16) uint8_t smem[];          // 128 bytes of mbarriers and flags, then the ring of stages
    constexpr int kRing = 128;
    constexpr int kBlocks = HD / 32;                       // 32-dim blocks per head
    constexpr int kBlk = FMT == kFmtQ8 ? 34 : FMT == kFmtQ4 ? 18 : 64;   // bytes per block (f16: 32 values)
    constexpr int kHeadBytes = kBlocks * kBlk;
    constexpr uint32_t kBias = FMT == kFmtQ8 ? 0x64806480u : 0x64086408u;  // 1024 + 128 | 1024 + 8
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nthreads = blockDim.x - 32;                  // the last warp only moves data; the others compute
    const bool producer = warp == (nthreads >> 5);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the merge kernel may become resident and wait
    const int r = lane >> 2, c = lane & 3;
    const int n_kv = p.n_kv_head;
    const int g = warp % n_kv, j = warp / n_kv;
    const int tiles = TPW * (nthreads >> 5) / n_kv;        // 16-position tiles per stage and KV head
    const int P = 16 * tiles;
    constexpr int kG = attn_group_rows(FMT);
    const int groups = P / kG;                             // copies per stage and tensor
    const int slot_bytes = groups * (p.gs_k + p.gs_v);
    const int t_begin = blockIdx.x * p.chunk;
    const int t_end = min(p.n_pos, t_begin + p.chunk);
    const int n_iter = t_end > t_begin ? (t_end - t_begin + P - 1) / P : 0;
    // more than four query heads per KV head: blockIdx.y picks a batch of four (the cache is read once per batch)
    const int h_first = 4 * blockIdx.y;
    const int heads_here = min(4, p.n_rep - h_first);

    // ---- copies: the producer warp moves a stage with one bulk copy per group of rows; rows past the end of
    // the range are zeroed with plain stores instead (only the last stage can have such rows).  Per ring slot
    // a "full" barrier counts the bytes that land and an "empty" barrier the compute warps that are done with it.
    const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem);
    const uint32_t ring = smem_base + kRing;
    const uint32_t full_bar = smem_base, empty_bar = smem_base + 32;
    volatile int* ctl = reinterpret_cast<volatile int*>(smem + 64);   // [0] a wait gave up, [1] stages issued so far
    const int NS = p.stages;
    if (tid == 0) {
        for (int s = 0; s < NS; ++s) {
            attn_mbar_init(full_bar + 8 * s, 1);
            attn_mbar_init(empty_bar + 8 * s, nthreads >> 5);
        }
        ctl[0] = 0, ctl[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    auto issue = [&](int it, int slot) {                   // producer warp only
        const uint32_t ks = ring + slot * slot_bytes, vs = ks + groups * p.gs_k;
        const int t0 = t_begin + it * P;
        const int valid = min(P, t_end - t0);
        for (int grp = lane; grp < groups; grp += 32) {    // rows past the end: zeros, with plain stores
            for (int e = max(min(kG, valid - grp * kG), 0); e < kG; ++e) {
                uint8_t* kz = smem + kRing + slot * slot_bytes + grp * p.gs_k + e * p.row_bytes;
                uint8_t* vz = smem + kRing + slot * slot_bytes + groups * p.gs_k + grp * p.gs_v + e * p.row_bytes;
                for (int b = 0; b < p.row_bytes; b += 16) {
                    *reinterpret_cast<uint4*>(kz + b) = make_uint4(0, 0, 0, 0);
                    *reinterpret_cast<uint4*>(vz + b) = make_uint4(0, 0, 0, 0);
                }
            }
        }
        __syncwarp();                                      // the stores above are ordered before lane 0's arrive
        if (lane == 0) attn_mbar_expect_tx(full_bar + 8 * slot, 2u * (uint32_t)valid * (uint32_t)p.row_bytes);
        __syncwarp();
        for (int grp = lane; grp < groups; grp += 32) {
            const int rows = min(kG, valid - grp * kG);    // rows of this group inside the range
            if (rows > 0) {
                const int64_t off = (int64_t)(t0 + grp * kG) * p.row_bytes;
                attn_bulk_load(ks + grp * p.gs_k, p.K + off, (uint32_t)(rows * p.row_bytes), full_bar + 8 * slot);
                attn_bulk_load(vs + grp * p.gs_v, p.V + off, (uint32_t)(rows * p.row_bytes), full_bar + 8 * slot);
            }
        }
    };
    float m_run = kNegInf, l_run = 0.f;
    float o[HD / 8][2];
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) o[i][0] = 0.f, o[i][1] = 0.f;

    if (producer) {
        int slot = 0, round = 0;
        for (int it = 0; it < n_iter; ++it) {
            if (round > 0) {
                // the slot's previous stage must have been released by every compute warp
                if (ctl[0] != 0) break;
                if (!attn_mbar_wait(empty_bar + 8 * slot, (uint32_t)(round - 1) & 1u)) {
                    if (lane == 0 && ctl[0] == 0) atomicExch(p.fault, (int)FAULT_BULK_WAIT_TIMEOUT);
                    ctl[0] = 1;
                    break;
                }
            }
            issue(it, slot);
            __syncwarp();
            if (lane == 0) ctl[1] = it + 1;
            if (++slot == NS) slot = 0, ++round;
        }
    } else {
    // ---- query fragments: B operand of the score product, n = lane / 4 = (head, high | low)
    uint32_t bq[HD / 16][2];
    float fk;                                              // factor of the scores of head (lane & 3)
    {
        const int hq = r >> 1;
        const bool live = h_first + hq < p.n_rep;
        const float* qh = p.q + (int64_t)(g * p.n_rep + (live ? h_first + hq : 0)) * HD;
        float4 v[HD / 16];
        float amax = 0.f;
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk) {
            v[kk] = live ? __ldg(reinterpret_cast<const float4*>(qh + 16 * kk + 4 * c)) : make_float4(0.f, 0.f, 0.f, 0.f);
            amax = fmaxf(amax, fmaxf(fmaxf(fabsf(v[kk].x), fabsf(v[kk].y)), fmaxf(fabsf(v[kk].z), fabsf(v[kk].w))));
        }
        amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
        amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
        int e = 0;
        if (amax > 0.f) (void)frexpf(amax, &e);           // amax = f * 2^e, f in [0.5, 1)
        const float down = ldexpf(1.f, -e);                // the head's query scaled into (-1, 1), exactly
        const bool low = r & 1;
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk) {
            const uint32_t x = split_hi_lo(v[kk].x * down), y = split_hi_lo(v[kk].y * down);
            const uint32_t z = split_hi_lo(v[kk].z * down), w = split_hi_lo(v[kk].w * down);
            bq[kk][0] = low ? __byte_perm(x, y, 0x7632) : __byte_perm(x, y, 0x5410);
            bq[kk][1] = low ? __byte_perm(z, w, 0x7632) : __byte_perm(z, w, 0x5410);
        }
        const float fk_own = p.scale * 1.4426950408889634f * ldexpf(1.f, e);
        fk = __shfl_sync(0xffffffffu, fk_own, 8 * c);      // from a lane whose n index belongs to head c
    }

    int slot = 0;
    uint32_t parity = 0;
    for (int it = 0; it < n_iter; ++it) {
        if (it > 0) {
            __syncwarp();                                  // every lane is done with the previous stage's slot
            if (lane == 0)
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(empty_bar + 8 * (slot == 0 ? NS - 1 : slot - 1))
                             : "memory");
        }
        if (ctl[0] != 0) break;
        if (!attn_mbar_wait(full_bar + 8 * slot, parity)) {
            if (lane == 0 && ctl[0] == 0) atomicExch(p.fault, (int)FAULT_BULK_WAIT_TIMEOUT);
            ctl[0] = 1;                                    // every warp stops at its next stage boundary
            break;
        }
        const int t_tile = t_begin + it * P + 16 * TPW * j;
        // a tile is a whole number of groups: its rows start (16 / kG) * tile groups into the region
        const uint32_t Ks = ring + slot * slot_bytes + (16 / kG) * TPW * j * p.gs_k + g * kHeadBytes;
        const uint32_t Vs = ring + slot * slot_bytes + groups * p.gs_k + (16 / kG) * TPW * j * p.gs_v + g * kHeadBytes;
        if (++slot == NS) slot = 0, parity ^= 1u;
        if (t_tile >= t_end) continue;                     // the same for the whole warp

        // ---- scores of positions r and r + 8 of each of the warp's tiles, for head c
        float sc[TPW][2];
#pragma unroll
        for (int u = 0; u < TPW; ++u) {
            float s0 = 0.f, s1 = 0.f;
            const uint32_t k0 = Ks + attn_row_offset(16 * u + attn_sigma(FMT, r), kG, p.gs_k, p.row_bytes);
            const uint32_t k8 = Ks + attn_row_offset(16 * u + attn_sigma(FMT, r + 8), kG, p.gs_k, p.row_bytes);
            if constexpr (FMT == kFmtF16) {
                float c4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {
                    const uint2 x = lds64(k0 + 32 * kk + 8 * c);
                    const uint2 y = lds64(k8 + 32 * kk + 8 * c);
                    mma_m16n8k16(c4, x.x, y.x, x.y, y.y, bq[kk][0], bq[kk][1]);
                }
                s0 = c4[0] + c4[1], s1 = c4[2] + c4[3];
            } else {
#pragma unroll
                for (int b = 0; b < kBlocks; ++b) {
                    float c4[4] = {0.f, 0.f, 0.f, 0.f};
                    const bool mis = (b & 1) == 0;         // kBlk * b + 2 is 2 mod 4 for even b
                    if constexpr (FMT == kFmtQ8) {
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const uint32_t a = k0 + kBlk * b + 2 + 16 * h + 4 * c;
                            const uint32_t a8 = k8 + kBlk * b + 2 + 16 * h + 4 * c;
                            const uint32_t w = (mis ? lds_word<true>(a) : lds_word<false>(a)) ^ 0x80808080u;
                            const uint32_t w8 = (mis ? lds_word<true>(a8) : lds_word<false>(a8)) ^ 0x80808080u;
                            mma_m16n8k16(c4, bytes01_to_h2(w, kBias), bytes01_to_h2(w8, kBias), bytes23_to_h2(w, kBias),
                                         bytes23_to_h2(w8, kBias), bq[2 * b + h][0], bq[2 * b + h][1]);
                        }
                    } else {
                        const uint32_t a = k0 + kBlk * b + 2 + 4 * c;
                        const uint32_t a8 = k8 + kBlk * b + 2 + 4 * c;
                        const uint32_t w = mis ? lds_word<true>(a) : lds_word<false>(a);
                        const uint32_t w8 = mis ? lds_word<true>(a8) : lds_word<false>(a8);
                        const uint32_t lo = w & 0x0F0F0F0Fu, hi = (w >> 4) & 0x0F0F0F0Fu;
                        const uint32_t lo8 = w8 & 0x0F0F0F0Fu, hi8 = (w8 >> 4) & 0x0F0F0F0Fu;
                        mma_m16n8k16(c4, bytes01_to_h2(lo, kBias), bytes01_to_h2(lo8, kBias), bytes23_to_h2(lo, kBias),
                                     bytes23_to_h2(lo8, kBias), bq[2 * b][0], bq[2 * b][1]);
                        mma_m16n8k16(c4, bytes01_to_h2(hi, kBias), bytes01_to_h2(hi8, kBias), bytes23_to_h2(hi, kBias),
                                     bytes23_to_h2(hi8, kBias), bq[2 * b + 1][0], bq[2 * b + 1][1]);
                    }
                    s0 = fmaf(lds_half(k0 + kBlk * b), c4[0] + c4[1], s0);
                    s1 = fmaf(lds_half(k8 + kBlk * b), c4[2] + c4[3], s1);
                }
            }
            sc[u][0] = (t_tile + 16 * u + attn_sigma(FMT, r) < t_end) ? s0 * fk : kNegInf;
            sc[u][1] = (t_tile + 16 * u + attn_sigma(FMT, r + 8) < t_end) ? s1 * fk : kNegInf;
        }

        // ---- online softmax (base 2): the eight lanes with equal c share the head's running maximum
        float mt = fmaxf(sc[0][0], sc[0][1]);
#pragma unroll
        for (int u = 1; u < TPW; ++u) mt = fmaxf(mt, fmaxf(sc[u][0], sc[u][1]));
        mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 4));
        mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 8));
        mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 16));
        const float m_new = fmaxf(m_run, mt);              // finite: the first position of the first tile is valid
        const float corr = fast_exp2(m_run - m_new);
        float ps[TPW][2], psum = 0.f;
#pragma unroll
        for (int u = 0; u < TPW; ++u) {
            const float p0 = fast_exp2(sc[u][0] - m_new), p1 = fast_exp2(sc[u][1] - m_new);
            psum += p0 + p1;
            ps[u][0] = p0 * kPdScale, ps[u][1] = p1 * kPdScale;
        }
        l_run = fmaf(l_run, corr, psum);                   // this lane's share of the head's exponential sum
        m_run = m_new;
        const float corr_o = __shfl_sync(0xffffffffu, corr, r >> 1);   // the accumulators of row r belong to head r / 2
        if (__any_sync(0xffffffffu, corr_o != 1.f)) {
#pragma unroll
            for (int i = 0; i < HD / 8; ++i) o[i][0] *= corr_o, o[i][1] *= corr_o;
        }

        // ---- output: per 32-dim block, A = (p * d_V * 2^8 as high | low) transposed into place, B = V codes
        uint32_t a0[TPW], a2[TPW];
        if constexpr (FMT == kFmtF16) {
#pragma unroll
            for (int u = 0; u < TPW; ++u) {
                uint32_t xa, xb;
                split_hi_lo2(ps[u][0], ps[u][1], xa, xb);
                a0[u] = movmatrix_trans(xa), a2[u] = movmatrix_trans(xb);
            }
        }
#pragma unroll
        for (int b = 0; b < kBlocks; ++b) {
#pragma unroll
            for (int u = 0; u < TPW; ++u) {
                // tile rows 2c, 2c + 1, 2c + 8, 2c + 9: the contraction index of the probabilities
                const uint32_t v0 = Vs + attn_row_offset(16 * u + attn_sigma(FMT, 2 * c), kG, p.gs_v, p.row_bytes);
                const uint32_t v1 = Vs + attn_row_offset(16 * u + attn_sigma(FMT, 2 * c + 1), kG, p.gs_v, p.row_bytes);
                const uint32_t v8 = Vs + attn_row_offset(16 * u + attn_sigma(FMT, 2 * c + 8), kG, p.gs_v, p.row_bytes);
                const uint32_t v9 = Vs + attn_row_offset(16 * u + attn_sigma(FMT, 2 * c + 9), kG, p.gs_v, p.row_bytes);
                if constexpr (FMT == kFmtF16) {
                    const uint2 x0 = lds64(v0 + 64 * b + 8 * r);
                    const uint2 x1 = lds64(v1 + 64 * b + 8 * r);
                    const uint2 x8 = lds64(v8 + 64 * b + 8 * r);
                    const uint2 x9 = lds64(v9 + 64 * b + 8 * r);
                    mma_m16n8k16_top(o[4 * b + 0][0], o[4 * b + 0][1], a0[u], a2[u], __byte_perm(x0.x, x1.x, 0x5410),
                                     __byte_perm(x8.x, x9.x, 0x5410));
                    mma_m16n8k16_top(o[4 * b + 1][0], o[4 * b + 1][1], a0[u], a2[u], __byte_perm(x0.x, x1.x, 0x7632),
                                     __byte_perm(x8.x, x9.x, 0x7632));
                    mma_m16n8k16_top(o[4 * b + 2][0], o[4 * b + 2][1], a0[u], a2[u], __byte_perm(x0.y, x1.y, 0x5410),
                                     __byte_perm(x8.y, x9.y, 0x5410));
                    mma_m16n8k16_top(o[4 * b + 3][0], o[4 * b + 3][1], a0[u], a2[u], __byte_perm(x0.y, x1.y, 0x7632),
                                     __byte_perm(x8.y, x9.y, 0x7632));
                } else {
                    const float dv0 =
                        lds_half(Vs + attn_row_offset(16 * u + attn_sigma(FMT, r), kG, p.gs_v, p.row_bytes) + kBlk * b);
                    const float dv8 =
                        lds_half(Vs + attn_row_offset(16 * u + attn_sigma(FMT, r + 8), kG, p.gs_v, p.row_bytes) + kBlk * b);
                    uint32_t xa, xb;
                    split_hi_lo2(ps[u][0] * dv0, ps[u][1] * dv8, xa, xb);
                    a0[u] = movmatrix_trans(xa), a2[u] = movmatrix_trans(xb);
                    const bool mis = (b & 1) == 0;
                    uint32_t w0, w1, w8, w9;
                    if constexpr (FMT == kFmtQ8) {
                        const int off = kBlk * b + 2 + 4 * r;
                        w0 = (mis ? lds_word<true>(v0 + off) : lds_word<false>(v0 + off)) ^ 0x80808080u;
                        w1 = (mis ? lds_word<true>(v1 + off) : lds_word<false>(v1 + off)) ^ 0x80808080u;
                        w8 = (mis ? lds_word<true>(v8 + off) : lds_word<false>(v8 + off)) ^ 0x80808080u;
                        w9 = (mis ? lds_word<true>(v9 + off) : lds_word<false>(v9 + off)) ^ 0x80808080u;
                    } else {
                        const int off = kBlk * b + 2 + 4 * (r & 3);
                        const int sh = 4 * (r >> 2);       // dims 16..31 of a block sit in the high nibbles
                        w0 = ((mis ? lds_word<true>(v0 + off) : lds_word<false>(v0 + off)) >> sh) & 0x0F0F0F0Fu;
                        w1 = ((mis ? lds_word<true>(v1 + off) : lds_word<false>(v1 + off)) >> sh) & 0x0F0F0F0Fu;
                        w8 = ((mis ? lds_word<true>(v8 + off) : lds_word<false>(v8 + off)) >> sh) & 0x0F0F0F0Fu;
                        w9 = ((mis ? lds_word<true>(v9 + off) : lds_word<false>(v9 + off)) >> sh) & 0x0F0F0F0Fu;
                    }
                    // byte i of the four words = dim 4r + i of the block at the four positions
                    const uint32_t lo01 = __byte_perm(w0, w1, 0x5140), hi01 = __byte_perm(w0, w1, 0x7362);
                    const uint32_t lo89 = __byte_perm(w8, w9, 0x5140), hi89 = __byte_perm(w8, w9, 0x7362);
                    mma_m16n8k16_top(o[4 * b + 0][0], o[4 * b + 0][1], a0[u], a2[u], bytes01_to_h2(lo01, kBias),
                                     bytes01_to_h2(lo89, kBias));
                    mma_m16n8k16_top(o[4 * b + 1][0], o[4 * b + 1][1], a0[u], a2[u], bytes23_to_h2(lo01, kBias),
                                     bytes23_to_h2(lo89, kBias));
                    mma_m16n8k16_top(o[4 * b + 2][0], o[4 * b + 2][1], a0[u], a2[u], bytes01_to_h2(hi01, kBias),
                                     bytes01_to_h2(hi89, kBias));
                    mma_m16n8k16_top(o[4 * b + 3][0], o[4 * b + 3][1], a0[u], a2[u], bytes23_to_h2(hi01, kBias),
                                     bytes23_to_h2(hi89, kBias));
                }
            }
        }
    }
    }   // compute warps
    __syncthreads();
    if (ctl[0] != 0) {
        // a wait gave up: let the copies still in flight land before the CTA leaves -- the last stages issued,
        // one per ring slot, each with one more bounded wait
        const int issued = ctl[1];
        for (int s = max(0, issued - NS); s < issued; ++s)
            if (!attn_mbar_wait(full_bar + 8 * (s % NS), (uint32_t)(s / NS) & 1u)) atomicExch(p.fault, (int)FAULT_DRAIN_TIMEOUT);
        __syncthreads();
    }                                                      // the ring is free: it now holds the warps' results
    if (producer && tiles == TPW) return;

    // ---- per warp: high + low rows, the head's exponential sum; then the tiles of a KV head are merged
    float* acc_sm = reinterpret_cast<float*>(smem + kRing);   // [warp][4 heads][HD]
    float* ml_sm = acc_sm + (nthreads >> 5) * 4 * HD;      // [warp][4 heads][2]
    float l_head = l_run;
    l_head += __shfl_xor_sync(0xffffffffu, l_head, 4);
    l_head += __shfl_xor_sync(0xffffffffu, l_head, 8);
    l_head += __shfl_xor_sync(0xffffffffu, l_head, 16);
    if (r == 0 && !producer) ml_sm[(warp * 4 + c) * 2] = m_run, ml_sm[(warp * 4 + c) * 2 + 1] = l_head;
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) {
        const float x = o[i][0] + __shfl_xor_sync(0xffffffffu, o[i][0], 4);
        const float y = o[i][1] + __shfl_xor_sync(0xffffffffu, o[i][1], 4);
        if ((r & 1) == 0 && !producer) {
            float* dst = acc_sm + (warp * 4 + (r >> 1)) * HD + 32 * (i >> 2) + (i & 3);
            dst[8 * c] = x, dst[8 * c + 4] = y;            // accumulator columns 2c, 2c + 1 = dims 8c + i, 8c + 4 + i
        }
    }
    if (tiles == TPW) {
        // one warp per KV head: the warp hands its own result over, no merge within the CTA
        __syncwarp();
        for (int hh = 0; hh < heads_here; ++hh) {
            float* dst = p.ws + ((int64_t)(g * p.n_rep + h_first + hh) * p.parts + blockIdx.x) * (HD + 2);
            const float* src = acc_sm + (warp * 4 + hh) * HD;
#pragma unroll
            for (int d = lane; d < HD; d += 32) dst[d] = src[d] * (1.f / kPdScale);
            if (lane < 2) dst[HD + lane] = lane == 0 ? ml_sm[(warp * 4 + hh) * 2] * 0.6931471805599453f : ml_sm[(warp * 4 + hh) * 2 + 1];
        }
        return;
    }
    __syncthreads();
    if (producer) return;
    const int per_g = heads_here * HD;
    for (int idx = tid; idx < n_kv * per_g; idx += nthreads) {
        const int gg = idx / per_g, rest = idx - gg * per_g;
        const int hh = rest / HD, d = rest - hh * HD;
        float mm = kNegInf;
        const int wpg = tiles / TPW;                       // warps per KV head
        for (int t = 0; t < wpg; ++t) mm = fmaxf(mm, ml_sm[((gg + n_kv * t) * 4 + hh) * 2]);
        float a = 0.f, ll = 0.f;
        for (int t = 0; t < wpg; ++t) {
            const int w = gg + n_kv * t;
            const float ms = ml_sm[(w * 4 + hh) * 2];
            const float f = (ms == kNegInf) ? 0.f : exp2f(ms - mm);
            a = fmaf(acc_sm[(w * 4 + hh) * HD + d], f, a);
            ll = fmaf(ml_sm[(w * 4 + hh) * 2 + 1], f, ll);
        }
        float* dst = p.ws + ((int64_t)(gg * p.n_rep + h_first + hh) * p.parts + blockIdx.x) * (HD + 2);
        dst[d] = a * (1.f / kPdScale);
        if (d == 0) dst[HD] = mm * 0.6931471805599453f, dst[HD + 1] = ll;   // the merge works in natural logarithms
    }
}

int sm_count_of_current_device() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

template <class Fmt>
cudaError_t launch_general(const AttnParams& p, cudaStream_t stream) {
    const int nrep_t = p.n_rep <= 1 ? 1 : p.n_rep <= 2 ? 2 : 4;
    const int batches = (p.n_rep + nrep_t - 1) / nrep_t;
    const dim3 grid(p.parts, p.n_kv_head, batches);
    if (nrep_t == 1) attn_decode_general_kernel<Fmt, 1><<<grid, kAttnThreads, 0, stream>>>(p);
    else if (nrep_t == 2) attn_decode_general_kernel<Fmt, 2><<<grid, kAttnThreads, 0, stream>>>(p);
    else attn_decode_general_kernel<Fmt, 4><<<grid, kAttnThreads, 0, stream>>>(p);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    return launch_merge(p.ws, p.out, p.n_head, p.parts, p.head_dim, stream);
}

// Geometry of the tensor-core kernel for a shape, or ok = false when the shape goes to the general kernel.
struct MmaPlan {
    bool ok;
    int threads, stages, smem_bytes, grid, tpw;
    AttnMmaParams p;
};

constexpr int kMmaSmemLimit = 227 * 1024;

// Worst number of distinct 32-bit words that fall into one bank for one fragment-load instruction of the
// tensor-core kernel, over its K loads (keys = true) or V loads, for a group stride; 1 = conflict-free.
int attn_bank_conflicts(int kfmt, bool keys, int row_bytes, int group_stride) {
    const int G = attn_group_rows(kfmt);
    int worst = 1;
    const int kinds[4] = {0, 1, 8, 9};
    for (int inst = 0; inst < (keys ? 2 : 4); ++inst) {
        const int halves = kfmt == kFmtF16 ? 2 : 1;        // 64-bit loads are served half a warp at a time
        for (int hw = 0; hw < halves; ++hw) {
            int words[64], n = 0;
            for (int lane = hw * (32 / halves); lane < (hw + 1) * (32 / halves); ++lane) {
                const int r = lane >> 2, c = lane & 3;
                const int m = keys ? r + 8 * inst : 2 * c + kinds[inst];
                const int base = attn_row_offset(attn_sigma(kfmt, m), G, group_stride, row_bytes) / 4;
                if (kfmt == kFmtF16) {
                    const int w = base + 2 * (keys ? c : r);
                    words[n++] = w, words[n++] = w + 1;
                } else {
                    words[n++] = base + (keys ? c : (kfmt == kFmtQ4 ? (r & 3) : r));
                }
            }
            for (int bank = 0; bank < 32; ++bank) {
                int distinct = 0;
                for (int i = 0; i < n; ++i) {
                    if ((words[i] & 31) != bank) continue;
                    bool seen = false;
                    for (int k = 0; k < i; ++k) seen = seen || words[k] == words[i];
                    if (!seen) ++distinct;
                }
                if (distinct > worst) worst = distinct;
            }
        }
    }
    return worst;
}

// Group stride (bytes) with the fewest bank conflicts: the group's rows plus 0..7 pieces of 16 bytes.
int attn_group_stride(int kfmt, bool keys, int row_bytes) {
    const int G = attn_group_rows(kfmt);
    int best = G * row_bytes, best_cost = 1 << 30;
    for (int pad = 0; pad < 8; ++pad) {
        const int cost = attn_bank_conflicts(kfmt, keys, row_bytes, G * row_bytes + 16 * pad);
        if (cost < best_cost) best_cost = cost, best = G * row_bytes + 16 * pad;
    }
    return best;
}

MmaPlan make_mma_plan(int fmt, int64_t n_head, int64_t n_kv_head, int64_t head_dim, int64_t n_pos, int sm_count) {
    MmaPlan pl{};
    pl.ok = false;
    const int64_t n_rep = n_head / n_kv_head;
    if (n_rep > 64 || (head_dim != 64 && head_dim != 128)) return pl;
    if (n_kv_head != 1 && n_kv_head != 2 && n_kv_head != 4 && n_kv_head != 8) return pl;
    const int64_t rb = (int64_t)lw_row_bytes(fmt, n_kv_head * head_dim);
    if (rb == 0 || rb % 16 != 0 || rb > 8192) return pl;
    AttnMmaParams& p = pl.p;
    p.row_bytes = (int)rb;
    const int kfmt = fmt == LW_F16 ? kFmtF16 : fmt == LW_Q8_0 ? kFmtQ8 : kFmtQ4;
    const int G = attn_group_rows(kfmt);
    p.gs_k = attn_group_stride(kfmt, true, (int)rb);
    p.gs_v = attn_group_stride(kfmt, false, (int)rb);
    // eight compute warps (plus the warp that moves the data) with two tiles each per stage where two stages of
    // that size fit, else one tile each
    for (int tpw = 2; tpw >= 1; --tpw) {
        const int warps = 8;
        const int tiles = tpw * warps / (int)n_kv_head;
        const int P = 16 * tiles;
        const int slot = P / G * (p.gs_k + p.gs_v);
        int stages = (kMmaSmemLimit - 128 - 16) / slot;
        if (stages > 4) stages = 4;
        const int results = warps * (4 * (int)head_dim + 8) * 4;      // the warps' results reuse the ring
        if (stages < 2 || stages * slot < results) continue;
        int grid = sm_count < kMaxParts ? sm_count : kMaxParts;
        const int64_t stages_total = (n_pos + P - 1) / P;
        if (stages_total < grid) grid = (int)stages_total;
        int64_t chunk = (n_pos + grid - 1) / grid;
        chunk = (chunk + P - 1) / P * P;
        grid = (int)((n_pos + chunk - 1) / chunk);
        pl.threads = 32 * (warps + 1), pl.stages = stages, pl.smem_bytes = stages * slot + 128 + 16, pl.grid = grid;
        pl.tpw = tpw;
        p.chunk = (int)chunk, p.parts = grid, p.stages = stages;
        p.n_kv_head = (int)n_kv_head, p.n_rep = (int)n_rep, p.n_pos = (int)n_pos;
        pl.ok = true;
        return pl;
    }
    return pl;
}

template <int FMT, int HD, int TPW>
cudaError_t launch_mma_one(const MmaPlan& pl, cudaStream_t stream) {
    static bool configured[64] = {false};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        err = cudaFuncSetAttribute(attn_decode_mma_kernel<FMT, HD, TPW>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   kMmaSmemLimit);
        if (err != cudaSuccess) return err;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    attn_decode_mma_kernel<FMT, HD, TPW><<<dim3(pl.grid, (pl.p.n_rep + 3) / 4), pl.threads, pl.smem_bytes, stream>>>(pl.p);
    return cudaGetLastError();
}

template <int FMT, int HD>
cudaError_t launch_mma_tpw(const MmaPlan& pl, cudaStream_t stream) {
    return pl.tpw == 2 ? launch_mma_one<FMT, HD, 2>(pl, stream) : launch_mma_one<FMT, HD, 1>(pl, stream);
}

cudaError_t launch_mma(int fmt, int head_dim, const MmaPlan& pl, cudaStream_t stream) {
    if (head_dim == 128) {
        if (fmt == LW_F16) return launch_mma_tpw<kFmtF16, 128>(pl, stream);
        if (fmt == LW_Q8_0) return launch_mma_tpw<kFmtQ8, 128>(pl, stream);
        return launch_mma_tpw<kFmtQ4, 128>(pl, stream);
    }
    if (fmt == LW_F16) return launch_mma_tpw<kFmtF16, 64>(pl, stream);
    if (fmt == LW_Q8_0) return launch_mma_tpw<kFmtQ8, 64>(pl, stream);
    return launch_mma_tpw<kFmtQ4, 64>(pl, stream);
}

int& attn_variant_storage() {
    static int v = 0;
    return v;
}

}  // namespace

bool attn_shape_supported(int fmt, int64_t n_head, int64_t n_kv_head, int64_t head_dim, int64_t n_pos) {
    if (fmt != LW_F16 && fmt != LW_Q8_0 && fmt != LW_Q4_0) return false;
    if (n_kv_head < 1 || n_head < 1 || n_head % n_kv_head != 0 || n_head > 1024) return false;
    if (head_dim != 32 && head_dim != 64 && head_dim != 128 && head_dim != 256) return false;
    return n_pos >= 1 && n_pos <= (int64_t)1 << 30;
}

int attn_parts(int64_t n_head, int64_t n_kv_head, int64_t head_dim, int64_t n_pos) {
    const int64_t n_rep = n_head / n_kv_head;
    const int nrep_t = n_rep <= 1 ? 1 : n_rep <= 2 ? 2 : 4;
    (void)head_dim;
    return general_parts(n_kv_head, (n_rep + nrep_t - 1) / nrep_t, n_pos, sm_count_of_current_device());
}

int64_t attn_workspace_bytes(int64_t n_head, int64_t n_kv_head, int64_t head_dim, int64_t n_pos) {
    (void)n_kv_head, (void)n_pos;
    return n_head * (int64_t)kMaxParts * (head_dim + 2) * (int64_t)sizeof(float);
}

void set_attn_variant(int variant) { attn_variant_storage() = variant; }

int attn_variant_of(int fmt, int64_t n_head, int64_t n_kv_head, int64_t head_dim, int64_t n_pos) {
    if (attn_variant_storage() == 1) return 1;
    return make_mma_plan(fmt, n_head, n_kv_head, head_dim, n_pos, sm_count_of_current_device()).ok ? 2 : 1;
}

int launch_attn_decode(int fmt, const void* K, const void* V, const float* q, float* out, int64_t n_head,
                       int64_t n_kv_head, int64_t head_dim, int64_t n_pos, float scale, void* workspace,
                       cudaStream_t stream) {
    if (attn_variant_storage() != 1) {
        MmaPlan pl = make_mma_plan(fmt, n_head, n_kv_head, head_dim, n_pos, sm_count_of_current_device());
        if (pl.ok) {
            pl.p.K = static_cast<const uint8_t*>(K);
            pl.p.V = static_cast<const uint8_t*>(V);
            pl.p.q = q, pl.p.ws = static_cast<float*>(workspace), pl.p.scale = scale;
            pl.p.fault = device_fault_word();
            if (!pl.p.fault) return (int)cudaErrorInvalidValue;
            cudaError_t err = launch_mma(fmt, (int)head_dim, pl, stream);
            if (err != cudaSuccess) return (int)err;
            return (int)launch_merge(pl.p.ws, out, (int)n_head, pl.p.parts, (int)head_dim, stream);
        }
    }
    AttnParams p;
    p.K = static_cast<const uint8_t*>(K);
    p.V = static_cast<const uint8_t*>(V);
    p.q = q, p.out = out, p.ws = static_cast<float*>(workspace);
    p.n_head = (int)n_head, p.n_kv_head = (int)n_kv_head, p.n_rep = (int)(n_head / n_kv_head), p.head_dim = (int)head_dim;
    p.n_pos = (int)n_pos;
    p.parts = attn_parts(n_head, n_kv_head, head_dim, n_pos);
    p.row_bytes = lw_row_bytes(fmt, n_kv_head * head_dim);
    p.scale = scale;
    cudaError_t err;
    switch (fmt) {
        case LW_F16: err = launch_general<FmtF16>(p, stream); break;
        case LW_Q8_0: err = launch_general<FmtQ8_0>(p, stream); break;
        default: err = launch_general<FmtQ4_0>(p, stream); break;
    }
    return (int)err;
}

}  // namespace lw

// ---------------------------------------------------------------------------------------------
// lw_attn_decode_static: the same attention for callers that have no device allocator to take a
// workspace from.  The partial results go to one fixed array that is part of the library's image.

namespace lw {
namespace {

// 4 Mi floats = 16 MiB, resident on every GPU that loads the library until the process exits.  With up to
// 256 partial results per head this covers n_head * (head_dim + 2) <= 16384: 64 heads of 128, 32 heads of 256.
constexpr int64_t kStaticScratchFloats = (int64_t)1 << 22;
static __device__ __align__(256) float g_attn_static_scratch[kStaticScratchFloats];

// Device address of the array on the current device, looked up once per device.  In host code the
// array's name is only a handle for the runtime; the kernels need the address the runtime maps it to.
float* static_scratch_of_current_device(cudaError_t* err) {
    constexpr int kMaxDevices = 64;
    static float* cached[kMaxDevices] = {nullptr};
    int dev = 0;
    *err = cudaGetDevice(&dev);
    if (*err != cudaSuccess) return nullptr;
    if (dev >= 0 && dev < kMaxDevices && cached[dev]) return cached[dev];
    float* ptr = nullptr;
    *err = cudaGetSymbolAddress((void**)&ptr, g_attn_static_scratch);
    if (*err != cudaSuccess) return nullptr;
    if (dev >= 0 && dev < kMaxDevices) cached[dev] = ptr;
    return ptr;
}

}  // namespace
}  // namespace lw

extern "C" int lw_attn_decode_static(int kv_fmt, const void* K_blocks, const void* V_blocks, const float* q, float* out,
                                     int64_t n_head, int64_t n_kv_head, int64_t head_dim, int64_t n_pos, float scale,
                                     void* stream) {
    using namespace lw;
    if (kv_fmt != LW_F16 && kv_fmt != LW_Q8_0 && kv_fmt != LW_Q4_0) return LW_ERR_FORMAT;
    if (!attn_shape_supported(kv_fmt, n_head, n_kv_head, head_dim, n_pos) || !std::isfinite(scale)) return LW_ERR_SHAPE;
    if (!K_blocks || !V_blocks || !q || !out) return LW_ERR_NULL;
    const uintptr_t any = reinterpret_cast<uintptr_t>(K_blocks) | reinterpret_cast<uintptr_t>(V_blocks) |
                          reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out);
    if (any & 15u) return LW_ERR_ALIGN;
    if (attn_workspace_bytes(n_head, n_kv_head, head_dim, n_pos) > kStaticScratchFloats * (int64_t)sizeof(float))
        return LW_ERR_WORKSPACE;                        // shape beyond the built-in scratch
    cudaError_t err = cudaSuccess;
    float* scratch = static_scratch_of_current_device(&err);
    if (!scratch) return LW_ERR_CUDA;
    return launch_attn_decode(kv_fmt, K_blocks, V_blocks, q, out, n_head, n_kv_head, head_dim, n_pos, scale, scratch,
                              static_cast<cudaStream_t>(stream)) == 0 ? LW_OK : LW_ERR_CUDA;
}
