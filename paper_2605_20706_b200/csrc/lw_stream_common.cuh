// Shared by the streaming mat-vec kernels (one launch per mat-vec, and the persistent sequence kernel):
// PTX helpers, the activation state a thread keeps in registers, and the per-format decode routines
// ("traits") [paper Sec 3.3: one decode routine per block format, spliced into a common kernel skeleton].
#ifndef LW_STREAM_COMMON_CUH_
#define LW_STREAM_COMMON_CUH_

#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <type_traits>

#include "lw_internal.h"

namespace lw {
namespace {

constexpr int kThreads = 256;
constexpr int kMaxStages = 4;
constexpr int kMaxGroup = 8;        // matrices per grouped launch
constexpr int kSmemHeader = 384;    // barriers, flags and unit records in front of the partial tables
constexpr int kUnitRecords = 8;     // per worker group, used in turn (more than ring slots + 2)
constexpr uint32_t kWaitSpinLimit = 1u << 16;    // tries; each may sleep up to kWaitSuspendNs (~0.1 s in all)
#ifndef LW_WAIT_NS
#define LW_WAIT_NS 2000
#endif
constexpr uint32_t kWaitSuspendNs = LW_WAIT_NS;

// ------------------------------------------------------------------ PTX helpers ---

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar_addr, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar_addr), "r"(parity), "r"(kWaitSuspendNs)
        : "memory");
    return ok != 0;
}

// Bounded wait on the barrier at shared-memory address bar_addr; returns false if the limit ran out.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar_addr, uint32_t parity) {
    for (uint32_t i = 0; i < kWaitSpinLimit; ++i)
        if (mbar_try_wait(bar_addr, parity)) return true;
    return false;
}
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
    return mbar_wait_bounded(smem_u32(bar), parity);
}

__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

// 1-D bulk copy global -> this CTA's shared memory, completion counted in bytes on `bar`.
// dst, src and bytes are multiples of 16.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar,
                                          uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1], %2, [%3], %4;" ::"r"(smem_u32(dst)),
        "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}

__device__ __forceinline__ void bulk_load_default(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            smem_u32(dst)),
        "l"(src), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}

__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Packed pair of floats in one 64-bit register, operand type of the two-wide FP32 instructions.
typedef unsigned long long f2;

__device__ __forceinline__ f2 pack2(float lo, float hi) {
    f2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ f2 pack2u(uint32_t lo, uint32_t hi) {
    f2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(f2 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f2 fma2(f2 a, f2 b, f2 c) {
    f2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ f2 mul2(f2 a, f2 b) {
    f2 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f2 add2(f2 a, f2 b) {
    f2 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float hsum2(f2 v) {
    float a, b;
    unpack2(v, a, b);
    return a + b;
}

// A small unsigned integer v < 128 placed in byte `I` of `src` becomes the float 128 + v: the byte
// lands in mantissa bits 16..22 of the constant 128.0f (0x43000000).
template <int I>
__device__ __forceinline__ uint32_t byte_to_128_plus(uint32_t src) {
    return __byte_perm(src, 0x43000000u, 0x7044u | (I << 8));
}
// A biased byte b (0..255) in byte `I` of `src` becomes the float 2^23 + b (0x4B000000 | b).
template <int I>
__device__ __forceinline__ uint32_t byte_to_2p23_plus(uint32_t src) {
    return __byte_perm(src, 0x4B000000u, 0x7440u | I);
}

__device__ __forceinline__ float half_lo_to_float(uint32_t w) {
    return __half2float(__ushort_as_half((unsigned short)(w & 0xFFFFu)));
}
__device__ __forceinline__ float half_hi_to_float(uint32_t w) {
    return __half2float(__ushort_as_half((unsigned short)(w >> 16)));
}

// Four masked nibbles (one per byte of `m`) times the activation pairs xa, xb, accumulated into
// the two chains p0, p1.  Values are 128 + q; the offset is removed once per block by the caller.
__device__ __forceinline__ void nibbles4_fma(uint32_t m, f2 xa, f2 xb, f2& p0, f2& p1) {
    p0 = fma2(pack2u(byte_to_128_plus<0>(m), byte_to_128_plus<1>(m)), xa, p0);
    p1 = fma2(pack2u(byte_to_128_plus<2>(m), byte_to_128_plus<3>(m)), xb, p1);
}

__device__ __forceinline__ int dp4a_uu(uint32_t a, uint32_t b, int c) {
    int r;
    asm("dp4a.u32.u32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    return r;
}
__device__ __forceinline__ int dp4a_us(uint32_t a, uint32_t b, int c) {
    int r;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    return r;
}
__device__ __forceinline__ int dp4a_su(uint32_t a, uint32_t b, int c) {
    int r;
    asm("dp4a.s32.u32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    return r;
}
__device__ __forceinline__ int dp4a_ss(uint32_t a, uint32_t b, int c) {
    int r;
    asm("dp4a.s32.s32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    return r;
}
// Exact int -> float for |s| < 2^22 without a conversion instruction (1.5 * 2^23 magic).
__device__ __forceinline__ float small_int_to_float(int s) {
    return __uint_as_float(0x4B400000u + (uint32_t)s) - 12582912.f;
}
// sum q * xq from the three byte-plane sums: (s2 * 256 + s1) * 256 + s0
__device__ __forceinline__ float combine_planes(int s0, int s1, int s2) {
    const float t = fmaf(small_int_to_float(s2), 256.f, small_int_to_float(s1));
    return fmaf(t, 256.f, small_int_to_float(s0));
}
// The same for two sums at once, in packed two-wide arithmetic (half the issue slots).  The six
// plane sums must have been accumulated on top of kIntMagic (the dp4a chains start from it instead of
// zero), so that each one already is the bit pattern of the float 1.5 * 2^23 + sum.
constexpr int kIntMagic = 0x4B400000;
__device__ __forceinline__ f2 combine_planes2(int a0, int a1, int a2, int b0, int b1, int b2) {
    const f2 bias = pack2(-12582912.f, -12582912.f);
    const f2 c256 = pack2(256.f, 256.f);
    const f2 f0 = add2(pack2u((uint32_t)a0, (uint32_t)b0), bias);
    const f2 f1 = add2(pack2u((uint32_t)a1, (uint32_t)b1), bias);
    const f2 f2v = add2(pack2u((uint32_t)a2, (uint32_t)b2), bias);
    return fma2(fma2(f2v, c256, f1), c256, f0);
}

// The six-bit (scale, min) pairs of sub-blocks 2g and 2g+1 of a q4_K super-block header, as bytes
// [scA, scB, mA, mB].  Branch-free: g only picks byte selectors and masks, which are loop-invariant
// per thread.  For g < 2 the fields are the low six bits of header bytes 2g, 2g+1 (scales) and
// 4+2g, 5+2g (mins); for g >= 2 the low nibbles of bytes 8+2(g-2).. carry bits 0-3 (scales low
// nibble, mins high nibble) and the top two bits of bytes 2(g-2).. and 4+2(g-2).. carry bits 4-5.
// SEL says what is known at compile time: 0 -> g < 2, 1 -> g >= 2, -1 -> decided at run time.  The
// kernels split their main loop by SEL (g is uniform per warp), so that no selector or mask has
// to be recomputed or kept in registers per product.
template <int SEL>
__device__ __forceinline__ uint32_t q4k_fields(const uint4& hdr, int g) {
    const uint32_t sel_pair = (g & 1) ? 0x7632u : 0x5410u;          // bytes (j, j+1) of hdr.y and of hdr.z
    const uint32_t pair = __byte_perm(hdr.y, hdr.z, sel_pair);
    if (SEL == 0) return pair & 0x3F3F3F3Fu;
    const uint32_t sel_nib = (g & 1) ? 0x3232u : 0x1010u;           // bytes (j, j+1) of hdr.w, twice
    const uint32_t nib = __byte_perm(hdr.w, hdr.w, sel_nib);
    const uint32_t high = ((pair >> 2) & 0x30303030u) | (nib & 0x00000F0Fu) | ((nib >> 4) & 0x0F0F0000u);
    if (SEL == 1) return high;
    return g < 2 ? (pair & 0x3F3F3F3Fu) : high;
}

// d*sc and dmin*m of sub-blocks 2g, 2g+1 as packed pairs: (128 + v) * d - 128 d = v * d exactly.
template <int SEL>
__device__ __forceinline__ void q4k_scales(const uint4& hdr, int g, f2& dsc, f2& dmn) {
    const uint32_t fields = q4k_fields<SEL>(hdr, g);
    const float d = half_lo_to_float(hdr.x), dmin = half_hi_to_float(hdr.x);
    dsc = fma2(pack2u(byte_to_128_plus<0>(fields), byte_to_128_plus<1>(fields)), pack2(d, d),
               pack2(-128.f * d, -128.f * d));
    dmn = fma2(pack2u(byte_to_128_plus<2>(fields), byte_to_128_plus<3>(fields)), pack2(dmin, dmin),
               pack2(-128.f * dmin, -128.f * dmin));
}

// ------------------------------------------------------------ activation state ---

// Traits without a kAnyStageRows member keep the first form of the stage completion.
template <class T, class = void>
struct any_stage_rows : std::false_type {};
template <class T>
struct any_stage_rows<T, std::void_t<decltype(T::kAnyStageRows)>> : std::bool_constant<T::kAnyStageRows> {};

struct Mapping {
    int row_slot;      // which of the wave's rows this thread works on
    int col_slot;      // index of this thread among the threads of that row (0..units-1)
    bool active;
};

// Activations owned by a thread, floating-point form: 32 packed pairs plus the sums over the two
// 32-weight halves.  `rd(i)` returns the thread's activations i..i+3 (i a multiple of 4).
struct XRegs {
    f2 x[32];
    float sum_a, sum_b;

    template <class Reader>
    __device__ __forceinline__ void load(Reader rd, bool active) {
#pragma unroll
        for (int i = 0; i < 64; i += 4) {
            const float4 v = active ? rd(i) : make_float4(0.f, 0.f, 0.f, 0.f);
            x[i / 2] = pack2(v.x, v.y);
            x[i / 2 + 1] = pack2(v.z, v.w);
        }
        f2 sa = 0, sb = 0;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            sa = add2(sa, x[i]);
            sb = add2(sb, x[16 + i]);
        }
        sum_a = hsum2(sa);
        sum_b = hsum2(sb);
    }
};

// Activations owned by a thread, block fixed-point form for the integer-dot variants: every group of
// GROUP consecutive activations shares one fp32 scale d = amax/4194303 and each value is the integer
// xq = rint(x/d) (|xq| <= 2^22), stored as three byte planes (p[0] low, p[1] middle: unsigned; p[2]
// high: signed), four elements per word so that one dp4a consumes four weights.  The representation
// error |x - d*xq| <= amax * 2^-23 per element is of the order of fp32 rounding itself.
// The conversion is done once per CTA, cooperatively, into shared memory (quantize_activations);
// each thread then copies the 48 plane words and the scales of its own 64-value unit.
constexpr int kXqUnitWords = 60;   // 48 plane words + 8 scale/sum words + 4 words of padding

template <bool Q4K_LAYOUT>
__device__ __forceinline__ int xq_unit_offset(int unit) {
    // q4_K threads of a warp read units 4 apart: one more 4-word pad per super-block keeps their
    // 16-byte loads on distinct banks; the other formats read consecutive units.
    return unit * kXqUnitWords + (Q4K_LAYOUT ? (unit >> 2) * 4 : 0);
}

// Converts the activation vector X[0..cols) to block fixed point in shared memory.  Each thread
// converts runs of 16 consecutive values (coalesced 64-byte reads); with GROUP == 32 two adjacent
// lanes share one scale.  `xq` is laid out per 64-value unit: words [16c + 4j, 16c + 4j + 4) hold
// byte plane c of the j-th run, words 48 + 2j and 49 + 2j its scale d and the sum d * sum(xq).
// `after_first_loads()` is called once, right after the first run's loads have been issued and before
// their values are needed: the caller uses it to request the weights behind the activations.
// COHERENT: read X past the L1 cache (it may have been written by other SMs earlier in the same launch).
template <int GROUP, bool Q4K_LAYOUT, int NTHREADS, int DEPTH = 4, bool COHERENT = false, class AfterLoads>
__device__ __forceinline__ void quantize_activations(const float* __restrict__ X, int cols, uint32_t* xq,
                                                     int tid, AfterLoads after_first_loads) {
    const int runs = cols >> 4;          // cols is a multiple of 256: runs is a multiple of 16
    constexpr int kDepth = DEPTH;        // runs whose loads are in flight together (one latency, not four)
    const int padded = (runs + 31) & ~31;
    bool first = true;
    for (int run0 = tid; run0 < padded; run0 += kDepth * NTHREADS) {
        float v[kDepth][16];
#pragma unroll
        for (int j = 0; j < kDepth; ++j) {
            const int run = run0 + j * NTHREADS;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
                if (run < runs)
                    t = COHERENT ? __ldcg(reinterpret_cast<const float4*>(X) + run * 4 + i)
                                 : __ldg(reinterpret_cast<const float4*>(X) + run * 4 + i);
                v[j][4 * i] = t.x;
                v[j][4 * i + 1] = t.y;
                v[j][4 * i + 2] = t.z;
                v[j][4 * i + 3] = t.w;
            }
        }
        if (first) {
            after_first_loads();
            first = false;
        }
#pragma unroll
        for (int j = 0; j < kDepth; ++j) {
            if (run0 + j * NTHREADS >= padded) break;      // warp-uniform: whole warps drop out together
            const int run = run0 + j * NTHREADS;
            const bool valid = run < runs;
            float amax = 0.f;
#pragma unroll
            for (int i = 0; i < 16; ++i) amax = fmaxf(amax, fabsf(v[j][i]));
            if (GROUP == 32) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
            const bool nonzero = amax > 1e-30f;
            float d = nonzero ? amax / 4194303.f : 0.f;
            const float inv = nonzero && amax <= 3.0e38f ? 4194303.f / amax : 0.f;
            int q[16];
            int total = 0;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                // round to nearest integer through the 1.5 * 2^23 magic constant (no conversion unit)
                q[i] = __float_as_int(fmaf(v[j][i], inv, 12582912.f)) - 0x4B400000;
                total += q[i];
            }
            // A NaN or Inf activation must reach every output it touches (as in fp32 arithmetic), but the
            // maximum above drops NaNs.  A non-finite value (or a finite one times inv = 0 of an infinite
            // maximum) leaves a NaN pattern in its code, more than 2^29 away from any sum of 16 proper codes
            // (|code| <= 2^22), whatever the number of such values: the run's sum gives it away, off the
            // critical path of the conversion, and the group's scale becomes NaN.
            int nonfinite = (total > 16 * 4194303 || total < -16 * 4194303) ? 1 : 0;
            if (GROUP == 32) nonfinite |= __shfl_xor_sync(0xFFFFFFFFu, nonfinite, 1);      // every lane takes part
            if (nonfinite) d = __int_as_float(0x7FC00000);
            if (valid) {
                uint32_t* u = xq + xq_unit_offset<Q4K_LAYOUT>(run >> 2);
                const int jj = run & 3;
                uint32_t pl[3][4];
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    const uint32_t lo01 = __byte_perm(q[4 * w], q[4 * w + 1], 0x5140);      // b0 b0 b1 b1
                    const uint32_t lo23 = __byte_perm(q[4 * w + 2], q[4 * w + 3], 0x5140);
                    const uint32_t hi01 = __byte_perm(q[4 * w], q[4 * w + 1], 0x6262);      // b2 b2 . .
                    const uint32_t hi23 = __byte_perm(q[4 * w + 2], q[4 * w + 3], 0x6262);
                    pl[0][w] = __byte_perm(lo01, lo23, 0x5410);
                    pl[1][w] = __byte_perm(lo01, lo23, 0x7632);
                    pl[2][w] = __byte_perm(hi01, hi23, 0x5410);
                }
#pragma unroll
                for (int c = 0; c < 3; ++c)
                    *reinterpret_cast<uint4*>(u + 16 * c + 4 * jj) =
                        make_uint4(pl[c][0], pl[c][1], pl[c][2], pl[c][3]);
                *reinterpret_cast<float2*>(u + 48 + 2 * jj) = make_float2(d, d * (float)total);
            }
        }
    }
}

// The same conversion with 8 values per thread (two lanes share a run of 16, four a group of 32): half the
// loads and arithmetic per thread and twice the threads at work for vectors of up to 8 * NTHREADS columns,
// which is what matters when the conversion sits on the critical path between two dependent mat-vecs.
// COHERENT reads X past the L1 cache (it may have been written by other SMs earlier in the same launch).
// `after_first_loads()` is called once per thread that has a piece, right after its first loads are issued.
// cols is a multiple of 256, NTHREADS a multiple of 32: whole warps take part or drop out together.
template <int GROUP, bool Q4K_LAYOUT, int NTHREADS, bool COHERENT = true, class AfterLoads>
__device__ __forceinline__ void quantize_activations8(const float* __restrict__ X, int cols, uint32_t* xq, int tid,
                                                      AfterLoads after_first_loads) {
    const int pieces = cols >> 3;
    constexpr int kDepth = 2;            // pieces whose loads are in flight together
    for (int p0 = tid; p0 < pieces; p0 += kDepth * NTHREADS) {
        float4 lo[kDepth], hi[kDepth];
#pragma unroll
        for (int j = 0; j < kDepth; ++j) {
            const int piece = p0 + j * NTHREADS;
            if (piece < pieces) {
                const float4* src = reinterpret_cast<const float4*>(X) + 2 * piece;
                lo[j] = COHERENT ? __ldcg(src) : __ldg(src);
                hi[j] = COHERENT ? __ldcg(src + 1) : __ldg(src + 1);
            }
        }
        if (p0 == tid) after_first_loads();
#pragma unroll
        for (int j = 0; j < kDepth; ++j) {
            const int piece = p0 + j * NTHREADS;
            if (piece >= pieces) break;
            const float v[8] = {lo[j].x, lo[j].y, lo[j].z, lo[j].w, hi[j].x, hi[j].y, hi[j].z, hi[j].w};
            float amax = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(v[i]));
            amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
            if (GROUP == 32) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 2));
            // scale and its reciprocal without divisions (this sits on a critical path): d * inv may differ from
            // 1 by a few 2^-23, which scales the whole group alike and is far inside the tolerance
            const bool nonzero = amax > 1e-30f;
            float d = nonzero ? amax * (1.f / 4194303.f) : 0.f;
            const float inv = nonzero && amax <= 3.0e38f ? 4194303.f * __frcp_rn(amax) : 0.f;
            int q[8];
            int total = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                q[i] = __float_as_int(fmaf(v[i], inv, 12582912.f)) - 0x4B400000;
                total += q[i];
            }
            // non-finite values leave NaN patterns as codes (see quantize_activations): the sum of the thread's
            // eight codes gives them away; the flag goes to all lanes of the group, whose scale becomes NaN
            int nonfinite = (total > 8 * 4194303 || total < -8 * 4194303) ? 1 : 0;
            nonfinite |= __shfl_xor_sync(0xFFFFFFFFu, nonfinite, 1);                       // every lane takes part
            if (GROUP == 32) nonfinite |= __shfl_xor_sync(0xFFFFFFFFu, nonfinite, 2);
            if (nonfinite) d = __int_as_float(0x7FC00000);
            total += __shfl_xor_sync(0xFFFFFFFFu, total, 1);      // sum over the run of 16
            const int run = piece >> 1, half = piece & 1;
            uint32_t* u = xq + xq_unit_offset<Q4K_LAYOUT>(run >> 2);
            const int jj = run & 3;
            uint32_t pl[3][2];
#pragma unroll
            for (int w = 0; w < 2; ++w) {
                const uint32_t lo01 = __byte_perm(q[4 * w], q[4 * w + 1], 0x5140);      // b0 b0 b1 b1
                const uint32_t lo23 = __byte_perm(q[4 * w + 2], q[4 * w + 3], 0x5140);
                const uint32_t hi01 = __byte_perm(q[4 * w], q[4 * w + 1], 0x6262);      // b2 b2 . .
                const uint32_t hi23 = __byte_perm(q[4 * w + 2], q[4 * w + 3], 0x6262);
                pl[0][w] = __byte_perm(lo01, lo23, 0x5410);
                pl[1][w] = __byte_perm(lo01, lo23, 0x7632);
                pl[2][w] = __byte_perm(hi01, hi23, 0x5410);
            }
#pragma unroll
            for (int c = 0; c < 3; ++c)
                *reinterpret_cast<uint2*>(u + 16 * c + 4 * jj + 2 * half) = make_uint2(pl[c][0], pl[c][1]);
            if (half == 0) *reinterpret_cast<float2*>(u + 48 + 2 * jj) = make_float2(d, d * (float)total);
        }
    }
}

template <int GROUP>
struct XInt {
    static constexpr int kGroups = 64 / GROUP;
    uint32_t p[3][16];
    float d[kGroups];     // scale of each group
    float sx[2];          // sum of d*xq over each 32-element half (block offset terms need it)

    __device__ __forceinline__ void load(const uint32_t* unit, bool active) {
        if (!active) {
#pragma unroll
            for (int c = 0; c < 3; ++c)
#pragma unroll
                for (int w = 0; w < 16; ++w) p[c][w] = 0;
#pragma unroll
            for (int g = 0; g < kGroups; ++g) d[g] = 0.f;
            sx[0] = sx[1] = 0.f;
            return;
        }
#pragma unroll
        for (int c = 0; c < 3; ++c)
#pragma unroll
            for (int w = 0; w < 16; w += 4) {
                const uint4 t = *reinterpret_cast<const uint4*>(unit + 16 * c + w);
                p[c][w] = t.x;
                p[c][w + 1] = t.y;
                p[c][w + 2] = t.z;
                p[c][w + 3] = t.w;
            }
        const float4 m0 = *reinterpret_cast<const float4*>(unit + 48);   // d0 s0 d1 s1
        const float4 m1 = *reinterpret_cast<const float4*>(unit + 52);   // d2 s2 d3 s3
        if (GROUP == 32) {
            d[0] = m0.x;
            d[1] = m1.x;
        } else {
            d[0] = m0.x;
            d[1 % kGroups] = m0.z;
            d[2 % kGroups] = m1.x;
            d[3 % kGroups] = m1.z;
        }
        sx[0] = m0.y + m0.w;
        sx[1] = m1.y + m1.w;
    }
};

// ------------------------------------------------------------------ format traits ---
//
// A trait describes how one thread consumes one row:
//   X           : the register-resident activation state (XRegs or XInt<>)
//   kXChunk     : activations are staged in shared memory in chunks of this many floats, each followed
//                 by 4 floats of padding, so that the threads' 16-byte reads are conflict-free (0: none)
//   map()       : thread id -> (row slot within a wave, column slot within the row)
//   x_index()   : column of the i-th of the 64 activations of a column slot
//   dot()       : raw bytes of the unit (in shared memory) x activations -> partial sum of the row

// ---- q4_K ----------------------------------------------------------------------------------
// Unit = one 32-byte nibble group of a super-block: weights 64g..64g+63 of the super-block
// (sub-blocks 2g and 2g+1).  All lanes of a warp share g (so the scale unpacking does not diverge)
// and walk consecutive super-blocks (144-byte stride: conflict-free 16-byte shared loads).
struct MapQ4K {
    static constexpr int kFmt = LW_Q4_K;
    static constexpr bool kSplitByGroup = true;     // the main loop is compiled once per half of g
    static constexpr bool kPairRows = true;         // two rows per loop iteration
    static constexpr int kXChunk = 256;
    static __device__ __forceinline__ Mapping map(int tid, int units_per_row, int rows_per_wave) {
        const int wrp = tid >> 5, ln = tid & 31;
        const int g = wrp & 3;
        const int sb_per_row = units_per_row >> 2;
        const int slot = ((wrp >> 2) << 5) + ln;            // super-block slot within the wave
        Mapping m;
        m.row_slot = slot / sb_per_row;
        const int sb = slot - m.row_slot * sb_per_row;
        m.col_slot = sb * 4 + g;
        m.active = m.row_slot < rows_per_wave;
        return m;
    }
    static __device__ __forceinline__ int64_t x_index(int col_slot, int, int i) { return (int64_t)col_slot * 64 + i; }
    // Per-thread constants of the row walk, computed once: byte offsets of the super-block header
    // and of the thread's 32-byte nibble group inside a row, and the group index.
    struct Ctx {
        int hdr_off, q_off, g;
    };
    static __device__ __forceinline__ Ctx make_ctx(int col_slot, int) {
        Ctx c;
        c.g = col_slot & 3;
        c.hdr_off = (col_slot >> 2) * 144;
        c.q_off = c.hdr_off + 16 + 32 * c.g;
        return c;
    }
    static __device__ __forceinline__ int split_sel(const Ctx& c) { return c.g >> 1; }
};

struct StreamQ4K : MapQ4K {
    static constexpr int kMinCtas = 2;
    static constexpr bool kIntegerDot = false;
    using X = XRegs;
    static __device__ __forceinline__ void finish_x(X&) {}
    template <int SEL = -1>
    static __device__ __forceinline__ float dot(const uint8_t* row, const Ctx& c, const X& xr) {
        const int g = c.g;
        const uint4 hdr = *reinterpret_cast<const uint4*>(row + c.hdr_off);
        const uint4 qa = *reinterpret_cast<const uint4*>(row + c.q_off);
        const uint4 qb = *reinterpret_cast<const uint4*>(row + c.q_off + 16);
        f2 dsc, dmn;
        q4k_scales<SEL>(hdr, g, dsc, dmn);
        const f2 corr = fma2(dsc, pack2(128.f, 128.f), dmn);   // 128*d*sc + dmin*m per sub-block
        f2 a0 = 0, a1 = 0, b0 = 0, b1 = 0;                      // sub-block 2g (low) / 2g+1 (high)
        const uint32_t q[8] = {qa.x, qa.y, qa.z, qa.w, qb.x, qb.y, qb.z, qb.w};
#pragma unroll
        for (int w = 0; w < 8; ++w) {
            const uint32_t lo = q[w] & 0x0F0F0F0Fu;
            const uint32_t hi = (q[w] >> 4) & 0x0F0F0F0Fu;
            nibbles4_fma(lo, xr.x[2 * w], xr.x[2 * w + 1], a0, a1);
            nibbles4_fma(hi, xr.x[16 + 2 * w], xr.x[16 + 2 * w + 1], b0, b1);
        }
        const float pa = hsum2(add2(a0, a1)), pb = hsum2(add2(b0, b1));
        f2 t = mul2(dsc, pack2(pa, pb));
        t = fma2(corr, pack2(-xr.sum_a, -xr.sum_b), t);
        return hsum2(t);
    }
};

struct IdotQ4K : MapQ4K {
    static constexpr int kMinCtas = 2;
    static constexpr bool kIntegerDot = true;
    static constexpr bool kXqQ4KLayout = true;
    using X = XInt<32>;
    // sub-block 2g+1 is accumulated from 16*q, so its activation scale absorbs the 1/16
    static __device__ __forceinline__ void finish_x(X& x) { x.d[1] *= 0.0625f; }
    template <int SEL = -1>
    static __device__ __forceinline__ float dot(const uint8_t* row, const Ctx& c, const X& x) {
        const uint4 hdr = *reinterpret_cast<const uint4*>(row + c.hdr_off);
        const uint4 qa = *reinterpret_cast<const uint4*>(row + c.q_off);
        const uint4 qb = *reinterpret_cast<const uint4*>(row + c.q_off + 16);
        // block scales in scalar arithmetic (packing their operands would cost more moves than the
        // packed instructions save): (128 + v) * d - 128 d = v * d exactly
        const uint32_t fields = q4k_fields<SEL>(hdr, c.g);
        const float d = half_lo_to_float(hdr.x), dmin = half_hi_to_float(hdr.x);
        const float nd = -128.f * d, ndmin = -128.f * dmin;
        const float dsc_a = fmaf(__uint_as_float(byte_to_128_plus<0>(fields)), d, nd);
        const float dsc_b = fmaf(__uint_as_float(byte_to_128_plus<1>(fields)), d, nd);
        const float dmn_a = fmaf(__uint_as_float(byte_to_128_plus<2>(fields)), dmin, ndmin);
        const float dmn_b = fmaf(__uint_as_float(byte_to_128_plus<3>(fields)), dmin, ndmin);
        const uint32_t q[8] = {qa.x, qa.y, qa.z, qa.w, qb.x, qb.y, qb.z, qb.w};
        int a0 = kIntMagic, a1 = kIntMagic, a2 = kIntMagic, b0 = kIntMagic, b1 = kIntMagic, b2 = kIntMagic;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t lo = q[i] & 0x0F0F0F0Fu;
            const uint32_t hi16 = q[i] - lo;                    // high nibbles as 16*q, no shift
            a0 = dp4a_uu(lo, x.p[0][i], a0);
            a1 = dp4a_uu(lo, x.p[1][i], a1);
            a2 = dp4a_us(lo, x.p[2][i], a2);
            b0 = dp4a_uu(hi16, x.p[0][8 + i], b0);
            b1 = dp4a_uu(hi16, x.p[1][8 + i], b1);
            b2 = dp4a_us(hi16, x.p[2][8 + i], b2);
        }
        float ta, tb;
        unpack2(combine_planes2(a0, a1, a2, b0, b1, b2), ta, tb);
        float r = dsc_a * (ta * x.d[0]);
        r = fmaf(dsc_b, tb * x.d[1], r);
        r = fmaf(-dmn_a, x.sx[0], r);
        return fmaf(-dmn_b, x.sx[1], r);
    }
};

// ---- q5_K ----------------------------------------------------------------------------------
// q4_K's super-block with 32 bytes qh between the header and the nibbles (176 bytes, 16-byte
// aligned).  A unit is the same 32 nibble bytes as in q4_K plus bits 2g and 2g+1 of all 32 qh bytes:
// code = nibble | bit << 4 (0..31), so both halves go through dp4a as plain bytes.
struct IdotQ5K {
    static constexpr bool kAnyStageRows = true;     // stage rows need not fill a warp evenly (see the stage completion)
    static constexpr int kFmt = LW_Q5_K;
    static constexpr int kMinCtas = 2;
    static constexpr bool kIntegerDot = true;
    static constexpr bool kXqQ4KLayout = true;
    static constexpr bool kSplitByGroup = true;     // compiled once per half of g, as q4_K
    static constexpr bool kPairRows = false;        // 20 raw words per row are live
    static constexpr int kXChunk = 256;
    using X = XInt<32>;
    static __device__ __forceinline__ void finish_x(X&) {}
    static __device__ __forceinline__ Mapping map(int tid, int units_per_row, int rows_per_wave) {
        return MapQ4K::map(tid, units_per_row, rows_per_wave);
    }
    static __device__ __forceinline__ int64_t x_index(int col_slot, int, int i) { return (int64_t)col_slot * 64 + i; }
    struct Ctx {
        int hdr_off, q_off, g;
    };
    static __device__ __forceinline__ Ctx make_ctx(int col_slot, int) {
        Ctx c;
        c.g = col_slot & 3;
        c.hdr_off = (col_slot >> 2) * 176;
        c.q_off = c.hdr_off + 48 + 32 * c.g;
        return c;
    }
    static __device__ __forceinline__ int split_sel(const Ctx& c) { return c.g >> 1; }
    template <int SEL = -1>
    static __device__ __forceinline__ float dot(const uint8_t* row, const Ctx& c, const X& x) {
        const uint4 hdr = *reinterpret_cast<const uint4*>(row + c.hdr_off);
        const uint4 ha = *reinterpret_cast<const uint4*>(row + c.hdr_off + 16);
        const uint4 hb = *reinterpret_cast<const uint4*>(row + c.hdr_off + 32);
        const uint4 qa = *reinterpret_cast<const uint4*>(row + c.q_off);
        const uint4 qb = *reinterpret_cast<const uint4*>(row + c.q_off + 16);
        const uint32_t fields = q4k_fields<SEL>(hdr, c.g);
        const float d = half_lo_to_float(hdr.x), dmin = half_hi_to_float(hdr.x);
        const float nd = -128.f * d, ndmin = -128.f * dmin;
        const float dsc_a = fmaf(__uint_as_float(byte_to_128_plus<0>(fields)), d, nd);
        const float dsc_b = fmaf(__uint_as_float(byte_to_128_plus<1>(fields)), d, nd);
        const float dmn_a = fmaf(__uint_as_float(byte_to_128_plus<2>(fields)), dmin, ndmin);
        const float dmn_b = fmaf(__uint_as_float(byte_to_128_plus<3>(fields)), dmin, ndmin);
        const uint32_t q[8] = {qa.x, qa.y, qa.z, qa.w, qb.x, qb.y, qb.z, qb.w};
        const uint32_t h[8] = {ha.x, ha.y, ha.z, ha.w, hb.x, hb.y, hb.z, hb.w};
        const int hs = 2 * c.g;
        int a0 = kIntMagic, a1 = kIntMagic, a2 = kIntMagic, b0 = kIntMagic, b1 = kIntMagic, b2 = kIntMagic;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t t = h[i] >> hs;                       // bit 0 of each byte: low half, bit 1: high half
            const uint32_t lo = (q[i] & 0x0F0F0F0Fu) | ((t << 4) & 0x10101010u);
            const uint32_t hi = ((q[i] >> 4) & 0x0F0F0F0Fu) | ((t << 3) & 0x10101010u);
            a0 = dp4a_uu(lo, x.p[0][i], a0);
            a1 = dp4a_uu(lo, x.p[1][i], a1);
            a2 = dp4a_us(lo, x.p[2][i], a2);
            b0 = dp4a_uu(hi, x.p[0][8 + i], b0);
            b1 = dp4a_uu(hi, x.p[1][8 + i], b1);
            b2 = dp4a_us(hi, x.p[2][8 + i], b2);
        }
        float ta, tb;
        unpack2(combine_planes2(a0, a1, a2, b0, b1, b2), ta, tb);
        float r = dsc_a * (ta * x.d[0]);
        r = fmaf(dsc_b, tb * x.d[1], r);
        r = fmaf(-dmn_a, x.sx[0], r);
        return fmaf(-dmn_b, x.sx[1], r);
    }
};

// ---- q6_K ----------------------------------------------------------------------------------
// Activations of a unit for q6_K: the three byte planes as above, one scale per run of 16 (the
// weight scales are per 16 too) and, per run, -32 times the sum of its activations (the codes are
// stored with an offset of 32).
struct XInt16R {
    static constexpr int kGroups = 4;
    uint32_t p[3][16];
    float d[4];
    float s[4];
    __device__ __forceinline__ void load(const uint32_t* unit, bool active) {
#pragma unroll
        for (int c = 0; c < 3; ++c)
#pragma unroll
            for (int w = 0; w < 16; w += 4) {
                const uint4 t = active ? *reinterpret_cast<const uint4*>(unit + 16 * c + w) : make_uint4(0, 0, 0, 0);
                p[c][w] = t.x;
                p[c][w + 1] = t.y;
                p[c][w + 2] = t.z;
                p[c][w + 3] = t.w;
            }
        const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
        const float4 m0 = active ? *reinterpret_cast<const float4*>(unit + 48) : z;   // d0 s0 d1 s1
        const float4 m1 = active ? *reinterpret_cast<const float4*>(unit + 52) : z;   // d2 s2 d3 s3
        d[0] = m0.x; s[0] = m0.y; d[1] = m0.z; s[1] = m0.w;
        d[2] = m1.x; s[2] = m1.y; d[3] = m1.z; s[3] = m1.w;
    }
};

// ---- q2_K (uses the activation form above) ---------------------------------------------------
// 84-byte super-blocks (4-byte aligned).  Unit g = half h = g/2, quarter pair p = g mod 2: the 32 code
// bytes of the half, shifted by 4p (quarter 2p: the unit's weights 0..31) and 4p + 2 (quarter 2p+1:
// weights 32..63), and the four (scale | min << 4) pairs 8h + 4p .. +3, one per run of 16.
struct IdotQ2K {
    static constexpr bool kAnyStageRows = true;     // stage rows need not fill a warp evenly (see the stage completion)
    static constexpr int kFmt = LW_Q2_K;
    static constexpr int kMinCtas = 2;
    static constexpr bool kIntegerDot = true;
    static constexpr bool kXqQ4KLayout = true;
    static constexpr bool kSplitByGroup = true;     // compiled once per p
    static constexpr bool kPairRows = true;
    static constexpr int kXChunk = 256;
    using X = XInt16R;
    static __device__ __forceinline__ void finish_x(X&) {}
    static __device__ __forceinline__ Mapping map(int tid, int units_per_row, int rows_per_wave) {
        return MapQ4K::map(tid, units_per_row, rows_per_wave);
    }
    static __device__ __forceinline__ int64_t x_index(int col_slot, int, int i) { return (int64_t)col_slot * 64 + i; }
    struct Ctx {
        int q_word, pair_word, d_word, g;     // 32-bit word indices inside the row
    };
    static __device__ __forceinline__ Ctx make_ctx(int col_slot, int) {
        Ctx c;
        const int base = (col_slot >> 2) * 21;          // 84 bytes = 21 words per super-block
        c.g = col_slot & 3;
        c.q_word = base + 4 + 8 * (c.g >> 1);
        c.pair_word = base + 2 * (c.g >> 1) + (c.g & 1);
        c.d_word = base + 20;
        return c;
    }
    static __device__ __forceinline__ int split_sel(const Ctx& c) { return c.g & 1; }
    template <int SEL = -1>
    static __device__ __forceinline__ float dot(const uint8_t* row, const Ctx& c, const X& x) {
        const uint32_t* w = reinterpret_cast<const uint32_t*>(row);
        uint32_t q[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) q[i] = w[c.q_word + i];
        const uint32_t pairs = w[c.pair_word];
        const uint32_t dd = w[c.d_word];
        const int sh = SEL < 0 ? 4 * (c.g & 1) : 4 * SEL;
        int acc[4][3];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int k = 0; k < 3; ++k) acc[r][k] = kIntMagic;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t ca = (q[i] >> sh) & 0x03030303u;          // weights 4i .. 4i+3
            const uint32_t cb = (q[i] >> (sh + 2)) & 0x03030303u;    // weights 32+4i ..
            const int r = i >> 2;
            acc[r][0] = dp4a_uu(ca, x.p[0][i], acc[r][0]);
            acc[r][1] = dp4a_uu(ca, x.p[1][i], acc[r][1]);
            acc[r][2] = dp4a_us(ca, x.p[2][i], acc[r][2]);
            acc[2 + r][0] = dp4a_uu(cb, x.p[0][8 + i], acc[2 + r][0]);
            acc[2 + r][1] = dp4a_uu(cb, x.p[1][8 + i], acc[2 + r][1]);
            acc[2 + r][2] = dp4a_us(cb, x.p[2][8 + i], acc[2 + r][2]);
        }
        float t[4];
        unpack2(combine_planes2(acc[0][0], acc[0][1], acc[0][2], acc[1][0], acc[1][1], acc[1][2]), t[0], t[1]);
        unpack2(combine_planes2(acc[2][0], acc[2][1], acc[2][2], acc[3][0], acc[3][1], acc[3][2]), t[2], t[3]);
        const float d = half_lo_to_float(dd), dmin = half_hi_to_float(dd);
        const float nd = -128.f * d, ndmin = -128.f * dmin;
        const uint32_t scs = pairs & 0x0F0F0F0Fu, mns = (pairs >> 4) & 0x0F0F0F0Fu;
        // (128 + v) * d - 128 d = v * d exactly
        const float s0 = fmaf(__uint_as_float(byte_to_128_plus<0>(scs)), d, nd);
        const float s1 = fmaf(__uint_as_float(byte_to_128_plus<1>(scs)), d, nd);
        const float s2 = fmaf(__uint_as_float(byte_to_128_plus<2>(scs)), d, nd);
        const float s3 = fmaf(__uint_as_float(byte_to_128_plus<3>(scs)), d, nd);
        const float m0 = fmaf(__uint_as_float(byte_to_128_plus<0>(mns)), dmin, ndmin);
        const float m1 = fmaf(__uint_as_float(byte_to_128_plus<1>(mns)), dmin, ndmin);
        const float m2 = fmaf(__uint_as_float(byte_to_128_plus<2>(mns)), dmin, ndmin);
        const float m3 = fmaf(__uint_as_float(byte_to_128_plus<3>(mns)), dmin, ndmin);
        float v = s0 * (t[0] * x.d[0]);
        v = fmaf(s1, t[1] * x.d[1], v);
        v = fmaf(s2, t[2] * x.d[2], v);
        v = fmaf(s3, t[3] * x.d[3], v);
        v = fmaf(-m0, x.s[0], v);
        v = fmaf(-m1, x.s[1], v);
        v = fmaf(-m2, x.s[2], v);
        return fmaf(-m3, x.s[3], v);
    }
};

// Unit g of a super-block = its weights 64g..64g+63 = half h = g/2, quarter pair p = g mod 2: the
// 64 ql bytes of the half (low nibbles for p = 0, high for p = 1), bits 4p..4p+3 of its 32 qh bytes,
// scales 8h + 4p .. +3.  Super-blocks are only 2-byte aligned in the row (210 bytes each), so every
// word is assembled from two aligned words with a funnel shift.
struct IdotQ6K {
    static constexpr bool kAnyStageRows = true;     // stage rows need not fill a warp evenly (see the stage completion)
    static constexpr int kFmt = LW_Q6_K;
    static constexpr int kMinCtas = 2;
    static constexpr bool kIntegerDot = true;
    static constexpr bool kXqQ4KLayout = true;
    static constexpr bool kSplitByGroup = true;     // compiled once per p
    static constexpr bool kPairRows = false;        // one row at a time: 27 raw words and 12 sums are live
    static constexpr int kXChunk = 256;
    using X = XInt16R;
    static __device__ __forceinline__ void finish_x(X& x) {
#pragma unroll
        for (int r = 0; r < 4; ++r) x.s[r] *= -32.f;
    }
    static __device__ __forceinline__ Mapping map(int tid, int units_per_row, int rows_per_wave) {
        return MapQ4K::map(tid, units_per_row, rows_per_wave);
    }
    static __device__ __forceinline__ int64_t x_index(int col_slot, int, int i) { return (int64_t)col_slot * 64 + i; }
    struct Ctx {
        int word0;      // index of the aligned 32-bit word that holds the super-block's first byte
        int shift;      // 0 or 16: bit offset of that byte inside the word
        int h, g;
    };
    static __device__ __forceinline__ Ctx make_ctx(int col_slot, int) {
        Ctx c;
        const int base = (col_slot >> 2) * 210;
        c.g = col_slot & 3;
        c.h = c.g >> 1;
        c.word0 = base >> 2;
        c.shift = (base & 2) * 8;
        return c;
    }
    static __device__ __forceinline__ int split_sel(const Ctx& c) { return c.g & 1; }
    // eight consecutive words starting `first` words into the super-block
    static __device__ __forceinline__ void load8(const uint32_t* w, int first, int shift, uint32_t (&out)[8]) {
        uint32_t raw[9];
#pragma unroll
        for (int i = 0; i < 9; ++i) raw[i] = w[first + i];
#pragma unroll
        for (int i = 0; i < 8; ++i) out[i] = __funnelshift_r(raw[i], raw[i + 1], shift);
    }
    template <int SEL = -1>
    static __device__ __forceinline__ float dot(const uint8_t* row, const Ctx& c, const X& x) {
        const uint32_t* w = reinterpret_cast<const uint32_t*>(row) + c.word0;
        uint32_t qa[8], qb[8], qh[8];
        load8(w, 16 * c.h, c.shift, qa);            // ql bytes 64h .. 64h+31
        load8(w, 16 * c.h + 8, c.shift, qb);        // ql bytes 64h+32 .. 64h+63
        load8(w, 32 + 8 * c.h, c.shift, qh);        // qh bytes 32h .. 32h+31
        const bool high = SEL < 0 ? (c.g & 1) : (SEL == 1);
        int acc[4][3];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int k = 0; k < 3; ++k) acc[r][k] = kIntMagic;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            // codes of weights 4i..4i+3 (quarter 2p, runs 0-1) and 32+4i.. (quarter 2p+1, runs 2-3)
            const uint32_t la = high ? (qa[i] >> 4) : qa[i];
            const uint32_t lb = high ? (qb[i] >> 4) : qb[i];
            const uint32_t ha = high ? qh[i] : (qh[i] << 4);
            const uint32_t hb = high ? (qh[i] >> 2) : (qh[i] << 2);
            const uint32_t ca = (la & 0x0F0F0F0Fu) | (ha & 0x30303030u);
            const uint32_t cb = (lb & 0x0F0F0F0Fu) | (hb & 0x30303030u);
            const int r = i >> 2;
            acc[r][0] = dp4a_uu(ca, x.p[0][i], acc[r][0]);
            acc[r][1] = dp4a_uu(ca, x.p[1][i], acc[r][1]);
            acc[r][2] = dp4a_us(ca, x.p[2][i], acc[r][2]);
            acc[2 + r][0] = dp4a_uu(cb, x.p[0][8 + i], acc[2 + r][0]);
            acc[2 + r][1] = dp4a_uu(cb, x.p[1][8 + i], acc[2 + r][1]);
            acc[2 + r][2] = dp4a_us(cb, x.p[2][8 + i], acc[2 + r][2]);
        }
        float t[4];
        unpack2(combine_planes2(acc[0][0], acc[0][1], acc[0][2], acc[1][0], acc[1][1], acc[1][2]), t[0], t[1]);
        unpack2(combine_planes2(acc[2][0], acc[2][1], acc[2][2], acc[3][0], acc[3][1], acc[3][2]), t[2], t[3]);
        // the unit's four int8 scales are bytes 192 + 8h + 4p .. +3 of the super-block: one word
        const int sw = 48 + 2 * c.h + (high ? 1 : 0);
        // (the second word is only needed, and only read, when the super-block sits 2 bytes into a word:
        // nothing is read beyond the super-block's 210 bytes)
        const uint32_t biased = __funnelshift_r(w[sw], w[sw + (c.shift >> 4)], c.shift) ^ 0x80808080u;   // scale + 128
        const float d = half_lo_to_float(c.shift ? (w[52] >> 16) : w[52]);                       // fp16 d at byte 208
        const float bias = -(8388608.f + 128.f);
        const float s0 = __uint_as_float(byte_to_2p23_plus<0>(biased)) + bias;
        const float s1 = __uint_as_float(byte_to_2p23_plus<1>(biased)) + bias;
        const float s2 = __uint_as_float(byte_to_2p23_plus<2>(biased)) + bias;
        const float s3 = __uint_as_float(byte_to_2p23_plus<3>(biased)) + bias;
        // sum over the run of (q - 32) * x = dx * sum(q * xq) - 32 * sum(x)
        float v = s0 * fmaf(t[0], x.d[0], x.s[0]);
        v = fmaf(s1, fmaf(t[1], x.d[1], x.s[1]), v);
        v = fmaf(s2, fmaf(t[2], x.d[2], x.s[2]), v);
        v = fmaf(s3, fmaf(t[3], x.d[3], x.s[3]), v);
        return d * v;
    }
};

// ---- q4_0 ----------------------------------------------------------------------------------
// Unit = two consecutive 18-byte blocks (36 bytes = 9 words, 4-byte aligned).  The first block's
// nibbles start 2 bytes into a word and are realigned with byte permutes.
struct MapLinear64 {
    static constexpr int kXChunk = 64;
    static constexpr bool kSplitByGroup = false;
    static constexpr bool kPairRows = true;
    static __device__ __forceinline__ Mapping map(int tid, int units_per_row, int rows_per_wave) {
        Mapping m;
        m.row_slot = tid / units_per_row;
        m.col_slot = tid - m.row_slot * units_per_row;
        m.active = m.row_slot < rows_per_wave;
        return m;
    }
    static __device__ __forceinline__ int64_t x_index(int col_slot, int, int i) { return (int64_t)col_slot * 64 + i; }
    struct Ctx {
        int col_slot;
    };
    static __device__ __forceinline__ Ctx make_ctx(int col_slot, int) { return Ctx{col_slot}; }
};

__device__ __forceinline__ void load_q4_0_unit(const uint8_t* row, int col_slot, uint32_t (&qa)[4],
                                               uint32_t (&qb)[4], float& da, float& db) {
    const uint32_t* p = reinterpret_cast<const uint32_t*>(row + col_slot * 36);
    uint32_t w[9];
#pragma unroll
    for (int i = 0; i < 9; ++i) w[i] = p[i];
    da = half_lo_to_float(w[0]);
    db = half_hi_to_float(w[4]);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        qa[i] = __byte_perm(w[i], w[i + 1], 0x5432u);
        qb[i] = w[5 + i];
    }
}

struct StreamQ40 : MapLinear64 {
    static constexpr int kFmt = LW_Q4_0;
    static constexpr int kMinCtas = 2;
    static constexpr bool kIntegerDot = false;
    using X = XRegs;
    static __device__ __forceinline__ void finish_x(X&) {}
    // one block: 4 words of nibbles; byte j = element j (low) | element j+16 (high)
    static __device__ __forceinline__ float block_sum(const uint32_t (&q)[4], const f2* x) {
        f2 p0 = 0, p1 = 0, p2 = 0, p3 = 0;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const uint32_t lo = q[w] & 0x0F0F0F0Fu;
            const uint32_t hi = (q[w] >> 4) & 0x0F0F0F0Fu;
            nibbles4_fma(lo, x[2 * w], x[2 * w + 1], p0, p1);
            nibbles4_fma(hi, x[8 + 2 * w], x[8 + 2 * w + 1], p2, p3);
        }
        return hsum2(add2(add2(p0, p1), add2(p2, p3)));
    }
    template <int SEL = -1>
    static __device__ __forceinline__ float dot(const uint8_t* row, const Ctx& c, const X& xr) {
        uint32_t qa[4], qb[4];
        float da, db;
        load_q4_0_unit(row, c.col_slot, qa, qb, da, db);
        const float pa = block_sum(qa, xr.x), pb = block_sum(qb, xr.x + 16);
        // sum (128 + q) x  -  136 sum x  =  sum (q - 8) x
        const float ta = fmaf(-136.f, xr.sum_a, pa), tb = fmaf(-136.f, xr.sum_b, pb);
        return fmaf(da, ta, db * tb);
    }
};

struct IdotQ40 : MapLinear64 {
    static constexpr int kFmt = LW_Q4_0;
    static constexpr int kMinCtas = 2;
    static constexpr bool kIntegerDot = true;
    static constexpr bool kXqQ4KLayout = false;
    using X = XInt<16>;       // the low-nibble and high-nibble halves of a block get their own scales
    static __device__ __forceinline__ void finish_x(X& x) {
        x.d[1] *= 0.0625f;    // elements 16..31 of each block are accumulated from 16*q
        x.d[3] *= 0.0625f;
    }
    static __device__ __forceinline__ float block(const uint32_t (&q)[4], float dw, const X& x, int b) {
        int l0 = kIntMagic, l1 = kIntMagic, l2 = kIntMagic, h0 = kIntMagic, h1 = kIntMagic, h2 = kIntMagic;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t lo = q[i] & 0x0F0F0F0Fu;
            const uint32_t hi16 = q[i] - lo;
            l0 = dp4a_uu(lo, x.p[0][8 * b + i], l0);
            l1 = dp4a_uu(lo, x.p[1][8 * b + i], l1);
            l2 = dp4a_us(lo, x.p[2][8 * b + i], l2);
            h0 = dp4a_uu(hi16, x.p[0][8 * b + 4 + i], h0);
            h1 = dp4a_uu(hi16, x.p[1][8 * b + 4 + i], h1);
            h2 = dp4a_us(hi16, x.p[2][8 * b + 4 + i], h2);
        }
        const float t = hsum2(mul2(combine_planes2(l0, l1, l2, h0, h1, h2), pack2(x.d[2 * b], x.d[2 * b + 1])));
        return dw * fmaf(-8.f, x.sx[b], t);          // sum (q - 8) x
    }
    template <int SEL = -1>
    static __device__ __forceinline__ float dot(const uint8_t* row, const Ctx& c, const X& x) {
        uint32_t qa[4], qb[4];
        float da, db;
        load_q4_0_unit(row, c.col_slot, qa, qb, da, db);
        return block(qa, da, x, 0) + block(qb, db, x, 1);
    }
};

// ---- q4_1, q5_0, q5_1 -----------------------------------------------------------------------
// The 32-weight blocks with an fp16 offset and / or a fifth code bit.  A unit is two consecutive
// blocks (40, 44 or 48 bytes: word aligned); fields that start two bytes into a word (q5_0's first
// block) are realigned with byte permutes.  Four fifth bits become bit 4 of four bytes with one
// multiply: ((t & 15) * 0x02040810) & 0x10101010.
template <bool FIVE, bool OFFSET>
struct IdotLegacy : MapLinear64 {
    static constexpr bool kAnyStageRows = true;
    static constexpr int kFmt = FIVE ? (OFFSET ? LW_Q5_1 : LW_Q5_0) : LW_Q4_1;
    static constexpr int kMinCtas = 2;
    static constexpr bool kIntegerDot = true;
    static constexpr bool kXqQ4KLayout = false;
    static constexpr bool kPairRows = !FIVE;
    static constexpr int kBlockBytes = 2 + (OFFSET ? 2 : 0) + (FIVE ? 4 : 0) + 16;
    static constexpr int kUnitWords = 2 * kBlockBytes / 4;
    using X = XInt<16>;       // the low-nibble and high-nibble halves of a block get their own scales
    static __device__ __forceinline__ void finish_x(X& x) {
        if (!FIVE) {          // q4_1 accumulates elements 16..31 of each block from 16*q
            x.d[1] *= 0.0625f;
            x.d[3] *= 0.0625f;
        }
    }
    // word `i` of the field that starts `byte` bytes into the unit (byte is even)
    template <int BYTE>
    static __device__ __forceinline__ uint32_t field_word(const uint32_t (&w)[kUnitWords], int i) {
        if (BYTE % 4 == 0) return w[BYTE / 4 + i];
        return __byte_perm(w[BYTE / 4 + i], w[BYTE / 4 + i + 1], 0x5432u);
    }
    static __device__ __forceinline__ uint32_t spread4(uint32_t t) {
        return ((t & 15u) * 0x02040810u) & 0x10101010u;
    }
    template <int B>
    static __device__ __forceinline__ float block(const uint32_t (&w)[kUnitWords], const X& x) {
        constexpr int kBase = B * kBlockBytes;
        constexpr int kHigh = kBase + 2 + (OFFSET ? 2 : 0);             // qh (if any)
        constexpr int kNib = kHigh + (FIVE ? 4 : 0);
        const uint32_t head = w[kBase / 4];
        const float dw = (kBase % 4 == 0) ? half_lo_to_float(head) : half_hi_to_float(head);
        const uint32_t qh = FIVE ? field_word<kHigh>(w, 0) : 0u;
        int l0 = kIntMagic, l1 = kIntMagic, l2 = kIntMagic, h0 = kIntMagic, h1 = kIntMagic, h2 = kIntMagic;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t q = field_word<kNib>(w, i);
            uint32_t lo = q & 0x0F0F0F0Fu, hi;
            if (FIVE) {
                lo |= spread4(qh >> (4 * i));
                hi = ((q >> 4) & 0x0F0F0F0Fu) | spread4(qh >> (16 + 4 * i));
            } else {
                hi = q - lo;                                            // 16 * high nibble
            }
            l0 = dp4a_uu(lo, x.p[0][8 * B + i], l0);
            l1 = dp4a_uu(lo, x.p[1][8 * B + i], l1);
            l2 = dp4a_us(lo, x.p[2][8 * B + i], l2);
            h0 = dp4a_uu(hi, x.p[0][8 * B + 4 + i], h0);
            h1 = dp4a_uu(hi, x.p[1][8 * B + 4 + i], h1);
            h2 = dp4a_us(hi, x.p[2][8 * B + 4 + i], h2);
        }
        const float t = hsum2(mul2(combine_planes2(l0, l1, l2, h0, h1, h2), pack2(x.d[2 * B], x.d[2 * B + 1])));
        if (OFFSET) return fmaf(dw, t, half_hi_to_float(head) * x.sx[B]);    // d * sum(q x) + m * sum(x)
        return dw * fmaf(-16.f, x.sx[B], t);                                   // d * sum((q - 16) x)
    }
    template <int SEL = -1>
    static __device__ __forceinline__ float dot(const uint8_t* row, const Ctx& c, const X& x) {
        const uint32_t* p = reinterpret_cast<const uint32_t*>(row) + c.col_slot * kUnitWords;
        uint32_t w[kUnitWords];
#pragma unroll
        for (int i = 0; i < kUnitWords; ++i) w[i] = p[i];
        return block<0>(w, x) + block<1>(w, x);
    }
};
using IdotQ41 = IdotLegacy<false, true>;
using IdotQ50 = IdotLegacy<true, false>;
using IdotQ51 = IdotLegacy<true, true>;

// ---- q8_0 ----------------------------------------------------------------------------------
// Unit = two consecutive 34-byte blocks (68 bytes = 17 words).
__device__ __forceinline__ void load_q8_0_unit(const uint8_t* row, int col_slot, uint32_t (&qa)[8],
                                               uint32_t (&qb)[8], float& da, float& db) {
    const uint32_t* p = reinterpret_cast<const uint32_t*>(row + col_slot * 68);
    uint32_t w[17];
#pragma unroll
    for (int i = 0; i < 17; ++i) w[i] = p[i];
    da = half_lo_to_float(w[0]);
    db = half_hi_to_float(w[8]);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        qa[i] = __byte_perm(w[i], w[i + 1], 0x5432u);
        qb[i] = w[9 + i];
    }
}

struct StreamQ80 : MapLinear64 {
    static constexpr int kFmt = LW_Q8_0;
    static constexpr int kMinCtas = 2;
    static constexpr bool kIntegerDot = false;
    using X = XRegs;
    static __device__ __forceinline__ void finish_x(X&) {}
    // int8 -> float without conversion instructions: q ^ 0x80 is dropped into the mantissa of 2^23,
    // and 2^23 + 128 is subtracted exactly with a packed add.
    static __device__ __forceinline__ float block_sum(const uint32_t (&q)[8], const f2* x) {
        const f2 bias = pack2(-8388736.f, -8388736.f);       // -(2^23 + 128)
        f2 p0 = 0, p1 = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) {
            const uint32_t b = q[w] ^ 0x80808080u;
            const f2 v0 = add2(pack2u(byte_to_2p23_plus<0>(b), byte_to_2p23_plus<1>(b)), bias);
            const f2 v1 = add2(pack2u(byte_to_2p23_plus<2>(b), byte_to_2p23_plus<3>(b)), bias);
            p0 = fma2(v0, x[2 * w], p0);
            p1 = fma2(v1, x[2 * w + 1], p1);
        }
        return hsum2(add2(p0, p1));
    }
    template <int SEL = -1>
    static __device__ __forceinline__ float dot(const uint8_t* row, const Ctx& c, const X& xr) {
        uint32_t qa[8], qb[8];
        float da, db;
        load_q8_0_unit(row, c.col_slot, qa, qb, da, db);
        const float pa = block_sum(qa, xr.x), pb = block_sum(qb, xr.x + 16);
        return fmaf(da, pa, db * pb);
    }
};

struct IdotQ80 : MapLinear64 {
    static constexpr int kFmt = LW_Q8_0;
    static constexpr int kMinCtas = 2;
    static constexpr bool kIntegerDot = true;
    static constexpr bool kXqQ4KLayout = false;
    using X = XInt<32>;
    static __device__ __forceinline__ void finish_x(X&) {}
    static __device__ __forceinline__ float block(const uint32_t (&q)[8], float dw, const X& x, int b) {
        int s0 = 0, s1 = 0, s2 = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            s0 = dp4a_su(q[i], x.p[0][8 * b + i], s0);
            s1 = dp4a_su(q[i], x.p[1][8 * b + i], s1);
            s2 = dp4a_ss(q[i], x.p[2][8 * b + i], s2);
        }
        return dw * (combine_planes(s0, s1, s2) * x.d[b]);
    }
    template <int SEL = -1>
    static __device__ __forceinline__ float dot(const uint8_t* row, const Ctx& c, const X& x) {
        uint32_t qa[8], qb[8];
        float da, db;
        load_q8_0_unit(row, c.col_slot, qa, qb, da, db);
        return block(qa, da, x, 0) + block(qb, db, x, 1);
    }
};

// ---- f16 -----------------------------------------------------------------------------------
// Unit = eight 16-byte pieces (8 halves each), piece j of column slot u at byte 16*(u + units*j),
// so a warp's 16-byte shared loads are contiguous.
struct StreamF16 {
    static constexpr int kFmt = LW_F16;
    static constexpr bool kSplitByGroup = false;
    static constexpr bool kPairRows = true;
    static constexpr int kMinCtas = 2;
    static constexpr bool kIntegerDot = false;
    static constexpr int kXChunk = 0;     // one unpadded copy
    using X = XRegs;
    static __device__ __forceinline__ void finish_x(X&) {}
    static __device__ __forceinline__ Mapping map(int tid, int units_per_row, int rows_per_wave) {
        return MapLinear64::map(tid, units_per_row, rows_per_wave);
    }
    static __device__ __forceinline__ int64_t x_index(int col_slot, int units_per_row, int i) {
        return (int64_t)8 * (col_slot + (int64_t)units_per_row * (i >> 3)) + (i & 7);
    }
    struct Ctx {
        int off, stride;      // byte offset of the first piece, bytes between pieces
    };
    static __device__ __forceinline__ Ctx make_ctx(int col_slot, int units_per_row) {
        return Ctx{16 * col_slot, 16 * units_per_row};
    }
    template <int SEL = -1>
    static __device__ __forceinline__ float dot(const uint8_t* row, const Ctx& c, const X& xr) {
        f2 p0 = 0, p1 = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint4 v = *reinterpret_cast<const uint4*>(row + c.off + c.stride * j);
            const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&u[i]));
                if (i & 1) p1 = fma2(pack2(f.x, f.y), xr.x[4 * j + i], p1);
                else p0 = fma2(pack2(f.x, f.y), xr.x[4 * j + i], p0);
            }
        }
        return hsum2(add2(p0, p1));
    }
};

// ------------------------------------------------ pieces of the kernel skeletons ---

// Shared-memory float index of activation k after padding (4 floats after every kXChunk).
template <class T>
__device__ __forceinline__ int x_padded_index(int64_t k) {
    if constexpr (T::kXChunk == 0) return (int)k;
    else return (int)(k + 4 * (k / T::kXChunk));
}

// Completes the rows of one ring stage from its partial table: y[r] = sum over c of part[r*units + c].
// Run by the whole CTA.  When a row's partials are a power-of-two number (<= 32) of 16-byte vectors,
// each thread loads one vector and the row is folded with a few shuffles inside a warp, all rows at
// once; otherwise one warp takes one row at a time.
struct FinishShape {
    int units;          // partials per row
    int vec_shift;      // log2 of the 16-byte vectors per row when the shuffle path applies, else -1
};
__device__ __forceinline__ FinishShape finish_shape(int units) {
    const int vec_per_row = units >> 2;
    const bool fast = vec_per_row >= 1 && vec_per_row <= 32 && (vec_per_row & (vec_per_row - 1)) == 0 &&
                      (units & 3) == 0;
    return FinishShape{units, fast ? 31 - __clz(vec_per_row) : -1};
}
__device__ __forceinline__ void finish_stage(const float* part, int rows_in_stage, const FinishShape& fs, float* y,
                                             int tid) {
    const int units = fs.units;
    if (fs.vec_shift >= 0) {
        const int vec_per_row = 1 << fs.vec_shift;
        const float4* pv = reinterpret_cast<const float4*>(part);
        const int total = rows_in_stage << fs.vec_shift;
        for (int base = 0; base < total; base += kThreads) {        // uniform trip count for the shuffles
            const int i = base + tid;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (i < total) v = pv[i];
            float s = (v.x + v.y) + (v.z + v.w);
            for (int off = vec_per_row >> 1; off > 0; off >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
            if (i < total && (i & (vec_per_row - 1)) == 0) y[i >> fs.vec_shift] = s;
        }
    } else {
        const int warp_id = tid >> 5, lane_id = tid & 31;
        for (int r = warp_id; r < rows_in_stage; r += kThreads / 32) {
            float s = 0.f;
            for (int c = lane_id; c < units; c += 32) s += part[r * units + c];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
            if (lane_id == 0) y[r] = s;
        }
    }
}

// Barrier over one worker group (kThreads threads); groups of a CTA use distinct hardware barriers.
template <int NG>
__device__ __forceinline__ void group_barrier(int wg) {
    if constexpr (NG == 1) {
        __syncthreads();
    } else {
        asm volatile("bar.sync %0, %1;" ::"r"(wg + 1), "n"(kThreads) : "memory");
    }
}

}  // namespace
}  // namespace lw
#endif
