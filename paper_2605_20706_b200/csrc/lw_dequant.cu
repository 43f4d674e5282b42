// Stand-alone dequantisation kernels: blocks -> fp32, bit-exact [paper Sec 3.3 decode routines].
// Write-bound (4 bytes out per weight): each thread decodes 8 consecutive weights and issues two
// 16-byte stores; consecutive threads write consecutive 32-byte pieces.
#include <cuda_runtime.h>

#include "lw_formats.cuh"
#include "lw_internal.h"

namespace lw {

template <class Fmt, int UNROLL>
__global__ void __launch_bounds__(256) dequant_kernel(const uint8_t* __restrict__ W, int64_t n8,
                                                      float* __restrict__ out) {
    // UNROLL runs of 8 weights per thread and trip, a grid-width apart: all their loads are issued before
    // the first decode, and consecutive threads write consecutive 32-byte pieces (whole sectors)
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t t0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t0 < n8; t0 += stride * UNROLL) {
        float w[UNROLL][8];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int64_t t = t0 + u * stride;
            if (t < n8) Fmt::decode8(W, 8 * t, w[u]);      // the whole buffer is one long "row"
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int64_t t = t0 + u * stride;
            if (t < n8) {
                float4* o = reinterpret_cast<float4*>(out + 8 * t);
                __stcs(o, make_float4(w[u][0], w[u][1], w[u][2], w[u][3]));
                __stcs(o + 1, make_float4(w[u][4], w[u][5], w[u][6], w[u][7]));
            }
        }
    }
}

// Launch shape from a sweep on B200 over 2^28 weights (GB/s of block bytes + 4 bytes per weight): a grid of
// 128 blocks per SM; four runs per trip for f16 (6.4 TB/s), two for the quantised formats (q4_K 5.4 TB/s:
// their decode costs 6-8 instructions per weight, so they are bound by instruction issue before the stores).
template <class Fmt, int UNROLL>
static int launch(const void* W, int64_t n, float* out, cudaStream_t stream) {
    const int64_t n8 = n / 8;
    int64_t blocks = (n8 + 255) / 256;
    const int64_t cap = 148 * 128;
    if (blocks > cap) blocks = cap;
    dequant_kernel<Fmt, UNROLL><<<(unsigned)blocks, 256, 0, stream>>>(static_cast<const uint8_t*>(W), n8, out);
    return (int)cudaGetLastError();
}

int launch_dequant(int fmt, const void* W, int64_t n, float* out, cudaStream_t stream) {
    switch (fmt) {
        case LW_F16: return launch<FmtF16, 4>(W, n, out, stream);
        case LW_Q8_0: return launch<FmtQ8_0, 2>(W, n, out, stream);
        case LW_Q4_0: return launch<FmtQ4_0, 2>(W, n, out, stream);
        case LW_Q4_K: return launch<FmtQ4_K, 2>(W, n, out, stream);
        case LW_Q6_K: return launch<FmtQ6_K, 2>(W, n, out, stream);
        case LW_Q5_K: return launch<FmtQ5_K, 2>(W, n, out, stream);
        case LW_Q2_K: return launch<FmtQ2_K, 2>(W, n, out, stream);
        case LW_Q4_1: return launch<FmtQ4_1, 2>(W, n, out, stream);
        case LW_Q5_0: return launch<FmtQ5_0, 2>(W, n, out, stream);
        case LW_Q5_1: return launch<FmtQ5_1, 2>(W, n, out, stream);
    }
    return (int)cudaErrorInvalidValue;
}

}  // namespace lw
