// Stand-alone dequantisation kernels: blocks -> fp32, bit-exact [paper Sec 3.3 decode routines].
// Write-bound (4 bytes out per weight): each thread decodes 8 consecutive weights and issues two
// 16-byte stores; consecutive threads write consecutive 32-byte pieces, a warp consecutive KB.
#include <cuda_runtime.h>

#include "lw_formats.cuh"
#include "lw_internal.h"

namespace lw {

// A warp takes UNROLL consecutive groups of 256 weights per trip (lane l the weights 8l .. 8l+7 of each group: two
// 16-byte streaming stores, consecutive lanes write consecutive 32-byte sectors), so a warp writes UNROLL KB of
// consecutive output; all loads of a trip are issued before the first decode.  (Runs a grid-width apart instead,
// the first form of this kernel, reached 0.73-0.82 of the copy peak for the quantised formats where this one
// reaches 0.82-0.93.)
template <class Fmt, int UNROLL>
__global__ void __launch_bounds__(256) dequant_warp_kernel(const uint8_t* __restrict__ W, int64_t n8,
                                                           float* __restrict__ out) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t g0 = UNROLL * warp; 32 * g0 < n8; g0 += UNROLL * n_warps) {
        float w[UNROLL][8];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int64_t t = 32 * (g0 + u) + lane;
            if (t < n8) Fmt::decode8(W, 8 * t, w[u]);
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int64_t t = 32 * (g0 + u) + lane;
            if (t < n8) {
                float4* o = reinterpret_cast<float4*>(out + 8 * t);
                __stcs(o, make_float4(w[u][0], w[u][1], w[u][2], w[u][3]));
                __stcs(o + 1, make_float4(w[u][4], w[u][5], w[u][6], w[u][7]));
            }
        }
    }
}

// q4_K and q5_K, a warp per group of four super-blocks and trip: lane l unpacks the (scale, min) pair of ONE
// sub-block (super-block l / 8 of the group, sub-block l mod 8) and the lanes that decode that sub-block's
// weights fetch the two factors with shuffles, so the header work is done once per 32 weights instead of once per
// 8.  Lane l then decodes weights 8l .. 8l+7 of each of the four super-blocks (consecutive lanes write
// consecutive 32-byte pieces).  Same arithmetic as FmtQ4_K / FmtQ5_K: fl(fl(d*sc) * q) - fl(dmin*m).
template <bool FIVE>
__global__ void __launch_bounds__(256) dequant_q45k_kernel(const uint8_t* __restrict__ W, int64_t n_sb,
                                                           float* __restrict__ out) {
    constexpr int kBytes = FIVE ? 176 : 144, kQs = FIVE ? 48 : 16;
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int s = lane >> 2;                                   // sub-block of this lane's weights
    const int shift = (s & 1) ? 4 : 0;                         // odd sub-blocks live in the high nibbles
    const int q_off = kQs + 32 * (lane >> 3) + 8 * (lane & 3);
    for (int64_t sb0 = 4 * warp; sb0 < n_sb; sb0 += 4 * n_warps) {
        uint2 qv[4], hv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint8_t* sb = W + (sb0 + u) * kBytes;
            qv[u] = make_uint2(0u, 0u);
            hv[u] = make_uint2(0u, 0u);
            if (sb0 + u < n_sb) {
                qv[u] = __ldg(reinterpret_cast<const uint2*>(sb + q_off));
                if (FIVE) hv[u] = __ldg(reinterpret_cast<const uint2*>(sb + 16 + 8 * (lane & 3)));
            }
        }
        float dl = 0.f, ml = 0.f;
        if (sb0 + (lane >> 3) < n_sb) {
            const uint4 hdr = __ldg(reinterpret_cast<const uint4*>(W + (sb0 + (lane >> 3)) * kBytes));
            uint32_t sc, mn;
            q4k_scale_min(hdr.y, hdr.z, hdr.w, lane & 7, sc, mn);
            dl = __fmul_rn(half_bits_to_float(hdr.x & 0xFFFFu), (float)sc);
            ml = __fmul_rn(half_bits_to_float(hdr.x >> 16), (float)mn);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float dlu = __shfl_sync(0xffffffffu, dl, 8 * u + s);
            const float mlu = __shfl_sync(0xffffffffu, ml, 8 * u + s);
            uint32_t a[2] = {(qv[u].x >> shift) & 0x0F0F0F0Fu, (qv[u].y >> shift) & 0x0F0F0F0Fu};
            if (FIVE) {
                a[0] |= ((hv[u].x >> s) & 0x01010101u) << 4;
                a[1] |= ((hv[u].y >> s) & 0x01010101u) << 4;
            }
            float w[8];
#pragma unroll
            for (int j = 0; j < 8; ++j)
                w[j] = __fsub_rn(__fmul_rn(dlu, (float)((a[j >> 2] >> (8 * (j & 3))) & 0xFFu)), mlu);
            if (sb0 + u < n_sb) {
                float4* o = reinterpret_cast<float4*>(out + (sb0 + u) * 256 + 8 * lane);
                __stcs(o, make_float4(w[0], w[1], w[2], w[3]));
                __stcs(o + 1, make_float4(w[4], w[5], w[6], w[7]));
            }
        }
    }
}

template <bool FIVE>
static int launch_q45k(const void* W, int64_t n, float* out, cudaStream_t stream) {
    const int64_t n_sb = n / 256;
    int64_t blocks = (n_sb + 31) / 32;               // 8 warps of 4 super-blocks each per block and trip
    const int64_t cap = 148 * 256;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    dequant_q45k_kernel<FIVE><<<(unsigned)blocks, 256, 0, stream>>>(static_cast<const uint8_t*>(W), n_sb, out);
    return (int)cudaGetLastError();
}

// Launch shape from sweeps on B200 over 2^28 weights (GB/s of block bytes + 4 bytes per weight): at most
// PER_SM blocks per SM (more trips per warp beyond that), four groups per trip for f16, two for the rest.
template <class Fmt, int UNROLL, int PER_SM>
static int launch(const void* W, int64_t n, float* out, cudaStream_t stream) {
    const int64_t n8 = n / 8;
    int64_t blocks = (n8 + 256 * UNROLL - 1) / (256 * UNROLL);
    const int64_t cap = 148 * PER_SM;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    dequant_warp_kernel<Fmt, UNROLL><<<(unsigned)blocks, 256, 0, stream>>>(static_cast<const uint8_t*>(W), n8, out);
    return (int)cudaGetLastError();
}

int launch_dequant(int fmt, const void* W, int64_t n, float* out, cudaStream_t stream) {
    switch (fmt) {
        case LW_F16: return launch<FmtF16, 4, 256>(W, n, out, stream);
        case LW_Q8_0: return launch<FmtQ8_0, 2, 192>(W, n, out, stream);
        case LW_Q4_0: return launch<FmtQ4_0, 2, 192>(W, n, out, stream);
        case LW_Q4_K: return launch_q45k<false>(W, n, out, stream);
        case LW_Q6_K: return launch<FmtQ6_K, 2, 256>(W, n, out, stream);
        case LW_Q5_K: return launch_q45k<true>(W, n, out, stream);
        case LW_Q2_K: return launch<FmtQ2_K, 2, 512>(W, n, out, stream);
        case LW_Q4_1: return launch<FmtQ4_1, 2, 256>(W, n, out, stream);
        case LW_Q5_0: return launch<FmtQ5_0, 2, 256>(W, n, out, stream);
        case LW_Q5_1: return launch<FmtQ5_1, 2, 256>(W, n, out, stream);
    }
    return (int)cudaErrorInvalidValue;
}

}  // namespace lw
