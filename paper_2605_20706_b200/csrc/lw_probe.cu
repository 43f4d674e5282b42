// Read-only streaming probe: the copy pipeline of the streaming mat-vec kernels (one CTA per SM, a ring of
// 1-D bulk copies into shared memory, L2 evict-first) with no arithmetic behind it.  What it reaches is the
// ceiling any kernel built on that pipeline can approach on a read-only stream; bench.py reports it beside
// the read+write copy figure the roofline fractions are quoted against.
#include <cuda_runtime.h>

#include "lw_internal.h"
#include "lw_stream_common.cuh"

namespace lw {
namespace {

constexpr int kProbeSlots = 4;
constexpr int kProbeStageBytes = 36 * 1024;

__global__ void __launch_bounds__(128, 1) probe_read_kernel(const uint8_t* src, int64_t bytes, int* fault, unsigned* sink) {
    extern __shared__ __align__(128) uint8_t smem[];
    uint64_t* full = reinterpret_cast<uint64_t*>(smem);
    uint8_t* ring = smem + 128;
    if (threadIdx.x != 0) return;
    // contiguous share of this CTA, in 16-byte pieces
    const int64_t pieces = bytes / 16;
    const int64_t p0 = pieces * blockIdx.x / gridDim.x, p1 = pieces * (blockIdx.x + 1) / gridDim.x;
    const uint8_t* base = src + 16 * p0;
    const int64_t mine = 16 * (p1 - p0);
    const int64_t n_stages = (mine + kProbeStageBytes - 1) / kProbeStageBytes;
    for (int s = 0; s < kProbeSlots; ++s) mbar_init(&full[s], 1);
    fence_barrier_init();
    const uint64_t policy = l2_evict_first_policy();
    auto issue = [&](int64_t it) {
        const int64_t off = it * kProbeStageBytes;
        const uint32_t n = (uint32_t)(mine - off < kProbeStageBytes ? mine - off : kProbeStageBytes);
        uint64_t* bar = &full[it % kProbeSlots];
        mbar_expect_tx(bar, n);
        bulk_load(ring + (size_t)(it % kProbeSlots) * kProbeStageBytes, base + off, n, bar, policy);
    };
    for (int64_t it = 0; it < kProbeSlots && it < n_stages; ++it) issue(it);
    unsigned acc = 0;
    int64_t done = 0;
    bool ok = true;
    for (; done < n_stages && ok; ++done) {
        const int slot = (int)(done % kProbeSlots);
        ok = mbar_wait_bounded(&full[slot], (uint32_t)(done / kProbeSlots) & 1u);
        if (!ok) break;
        acc ^= *reinterpret_cast<const unsigned*>(ring + (size_t)slot * kProbeStageBytes);
        if (done + kProbeSlots < n_stages) issue(done + kProbeSlots);
    }
    if (!ok) {
        // a wait gave up: record it and give the copies still in flight one more bounded wait each
        atomicExch(fault, (int)FAULT_BULK_WAIT_TIMEOUT);
        const int64_t issued = done + kProbeSlots < n_stages ? done + kProbeSlots : n_stages;
        for (int64_t it = done; it < issued; ++it)
            if (!mbar_wait_bounded(&full[it % kProbeSlots], (uint32_t)(it / kProbeSlots) & 1u))
                atomicExch(fault, (int)FAULT_DRAIN_TIMEOUT);
    }
    if (acc == 0x9E3779B9u) *sink = acc;      // keeps the reads alive; practically never true
}

__device__ unsigned g_probe_sink;

}  // namespace

int launch_probe_read(const void* src, int64_t bytes, cudaStream_t stream) {
    static bool attr_set[64] = {false};
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return (int)e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return (int)e;
    const size_t smem = 128 + (size_t)kProbeSlots * kProbeStageBytes;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        e = cudaFuncSetAttribute(probe_read_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return (int)e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    int* fault = device_fault_word();
    unsigned* sink = nullptr;
    if (!fault || cudaGetSymbolAddress(reinterpret_cast<void**>(&sink), g_probe_sink) != cudaSuccess) return (int)cudaErrorInvalidValue;
    probe_read_kernel<<<(unsigned)sms, 128, smem, stream>>>(static_cast<const uint8_t*>(src), bytes, fault, sink);
    return (int)cudaGetLastError();
}

}  // namespace lw
