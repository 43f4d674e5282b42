// Persistent sequence kernel: all mat-vecs of a decode step (or any list of batch-1 mat-vecs of one
// format) inside ONE launch of co-resident CTAs, one per SM [paper Sec 3.1 / 3.2: the runtime groups
// operations into compute passes to cut submission and synchronisation cost; here the whole chain of
// a step is one pass].
//
// The sequence is a list of PHASES.  A phase is one activation vector X and the matrices multiplied
// with it (q/k/v share one X, gate/up another; o, down and lm_head are phases of one matrix).  Inside
// a phase the rows of its matrices form one virtual row space that is cut evenly over the CTAs at row
// granularity; each CTA cuts its share into units of at most one ring stage.
//
// What the single launch buys over one launch per phase:
//   * The weight ring never drains between phases.  Weights are constant data, so the producer thread
//     of a worker group claims the next unit -- of whatever phase comes next -- as soon as one of its
//     ring slots falls free: while a CTA waits for the other CTAs at a phase boundary and converts the
//     next activation vector, its ring is already filling with the next phase's rows, and HBM stays
//     busy across the boundary.
//   * A phase boundary costs one grid-wide barrier (only where the next X depends on earlier results)
//     plus the activation fetch, instead of a kernel drain, a launch and a cold ring.
//   * Shares are balanced to one row across the CTAs and to one wave between a CTA's two worker groups.
// The product loop, the activation state in registers and the per-format decode routines are those of
// the single-launch streaming kernel (lw_stream_common.cuh).
//
// Every wait is bounded.  A bulk-copy wait or a grid barrier that gives up records a fault code, stops
// waiting from then on (arrivals continue, so no other CTA is kept waiting by this one), and the
// kernel runs to its end; copies still in flight get one more bounded wait before shared memory is
// released.
#include <cuda_runtime.h>

#include <algorithm>
#include <vector>

#include "lw_internal.h"
#include "lw_stream_common.cuh"

namespace lw {
namespace {

constexpr int kSeqMaxPhases = 320;
constexpr int kSeqMaxMats = 640;
constexpr int kSeqSlots = 2;                       // ring slots per worker group
constexpr int kBarrierThread = 64;                 // the thread of a CTA that arrives at and polls the grid barrier
constexpr int kSeqHeader = 512;                    // barriers, flags, unit records, walkers
constexpr uint32_t kGridSpinLimit = 1u << 20;      // polls of the arrival counter (~0.5 us each) before giving up

struct SeqMat {
    const uint8_t* W;
    float* Y;
    int rows;
    int vrow0;             // first row of this matrix in its phase's virtual row space
};

struct SeqPhase {
    const float* X;
    int units;             // 64-weight units per row (cols / 64)
    int row_bytes;
    int rows_per_wave;     // rows the 256 threads of a group work on at a time
    int unit_cap;          // most rows in one unit (a multiple of rows_per_wave)
    int total_rows;        // rows of all matrices of the phase
    int first_mat;         // index of its first matrix in SeqParams::mat
    int dep_index;         // 0: no barrier before this phase; k > 0: every CTA first waits until all CTAs have
                           // finished everything before the k-th such phase
    int pad;
};

struct SeqParams {
    int n_phases;
    int n_mats;
    unsigned* counter;     // arrival counter of the grid barrier, zero at launch
    int* fault;
    uint32_t x_off;        // byte offset of the activation area in shared memory
    uint32_t ring_off;     // byte offset of the rings
    uint32_t stage_stride; // bytes between ring slots (multiple of 128)
    uint32_t partial_bytes;   // bytes of one partial table
    SeqPhase ph[kSeqMaxPhases];
    SeqMat mat[kSeqMaxMats];
};
static_assert(sizeof(SeqParams) <= 32000, "kernel parameters are limited to 32764 bytes");

// Profiling builds (-DLW_SEQ_TRACE) record globaltimer stamps of the phase boundaries of three CTAs.
#ifdef LW_SEQ_TRACE
constexpr int kTraceEvents = 8;
__device__ unsigned long long g_seq_trace[3][kSeqMaxPhases][kTraceEvents];
__device__ __forceinline__ void seq_stamp(int phase, int ev) {
    const int b = (int)blockIdx.x;
    const int which = b == 0 ? 0 : (b == (int)gridDim.x / 2 ? 1 : (b == (int)gridDim.x - 1 ? 2 : -1));
    if (which < 0 || threadIdx.x != kBarrierThread) return;
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    g_seq_trace[which][phase][ev] = t;
}
#define LW_SEQ_STAMP(phase, ev) seq_stamp(phase, ev)
#else
#define LW_SEQ_STAMP(phase, ev)
#endif

// Where a producer thread stands in its worker group's list of units.  A CTA's share of a phase is cut into
// two contiguous halves of whole waves, one per worker group (a group works through a unit wave by wave,
// rows_per_wave rows at a time, and a partial wave costs as much as a full one); the group that gets the
// larger half alternates from phase to phase.  Each half is cut into full units (large copies keep the most
// bytes in flight) and a remainder, and at the boundaries of the phase's matrices.  The list is a pure
// function of the launch parameters, the CTA index and the group.
struct Walker {
    int ph;        // phase of the unit at the cursor; n_phases when the list is exhausted
    int m;         // matrix of the unit at the cursor
    int v;         // virtual row at the cursor
    int vend;      // end of the group's half of the CTA's share of the phase
    int cap;       // rows of a full unit in this phase
    int claims;    // units this producer has recorded so far
    int pad[2];
};

__device__ __forceinline__ void share_of(const SeqPhase& P, int cta, int grid, int& v0, int& v1) {
    v0 = (int)((unsigned)P.total_rows * (unsigned)cta / (unsigned)grid);
    v1 = (int)((unsigned)P.total_rows * (unsigned)(cta + 1) / (unsigned)grid);
}

// Moves the cursor to the first unit of the next phase in which this group has rows.
__device__ __forceinline__ void walker_next_phase(const SeqParams& p, Walker& w, int wg, int cta, int grid) {
    for (;;) {
        ++w.ph;
        if (w.ph >= p.n_phases) {
            w.ph = p.n_phases;
            return;
        }
        const SeqPhase& P = p.ph[w.ph];
        int v0, v1;
        share_of(P, cta, grid, v0, v1);
        const int rpw = P.rows_per_wave;
        const int waves = (v1 - v0 + rpw - 1) / rpw;
        const int first_half = ((w.ph & 1) ? waves + 1 : waves) / 2;       // waves of the first half
        int vmid = v0 + first_half * rpw;
        if (vmid > v1) vmid = v1;
        w.v = wg == 0 ? v0 : vmid;
        w.vend = wg == 0 ? vmid : v1;
        if (w.v == w.vend) continue;
        w.cap = P.unit_cap;
        int m = P.first_mat;
        while (w.v >= p.mat[m].vrow0 + p.mat[m].rows) ++m;
        w.m = m;
        return;
    }
}

// The unit at the cursor (matrix, first row inside it, rows), then moves the cursor past it.
__device__ __forceinline__ void walker_take(const SeqParams& p, Walker& w, int wg, int cta, int grid, int& phase, int& m,
                                            int& begin, int& n) {
    const SeqMat& mt = p.mat[w.m];
    const int mat_end = mt.vrow0 + mt.rows;
    n = w.cap;
    if (n > w.vend - w.v) n = w.vend - w.v;
    if (n > mat_end - w.v) n = mat_end - w.v;
    phase = w.ph;
    m = w.m;
    begin = w.v - mt.vrow0;
    w.v += n;
    if (w.v == w.vend) walker_next_phase(p, w, wg, cta, grid);
    else if (w.v == mat_end) ++w.m;
}

// The conversion of a phase's activations, kept out of line: it runs once per phase, and its registers
// must not weigh on the allocation of the product loop.
template <int GROUP, bool Q4K_LAYOUT>
__device__ __noinline__ void seq_convert_activations(const float* X, int cols, uint32_t* xq, int tid) {
    quantize_activations8<GROUP, Q4K_LAYOUT, 2 * kThreads, true>(X, cols, xq, tid, [] {});
}

// One claim of a producer thread: the group's next unit (n == 0 when its list is exhausted).
struct Claim {
    int phase, m, begin, n, record_index;
};
__device__ __forceinline__ Claim seq_claim(const SeqParams& p, Walker* walker, int wg, bool stop, int cta, int grid) {
    Walker w = *walker;
    int phase = 0, m = 0, begin = 0, n = 0;
    if (w.ph < p.n_phases && !stop) walker_take(p, w, wg, cta, grid, phase, m, begin, n);
    const int record_index = w.claims & (kUnitRecords - 1);
    ++w.claims;
    *walker = w;
    return Claim{phase, m, begin, n, record_index};
}

template <class T>
__global__ void __launch_bounds__(2 * kThreads, 1) matvec_seq_kernel(const __grid_constant__ SeqParams p) {
    extern __shared__ __align__(128) uint8_t smem[];
    // layout: [0,64) ring barriers | 64 copy-wait-gave-up flag | 72 grid-barrier-gave-up flag |
    //         [80,336) unit records, 16 bytes each, kUnitRecords per group | [336,400) walkers | [400,416) armed counts |
    //         partial tables | activations | rings
    volatile int* copy_gave_up = reinterpret_cast<volatile int*>(smem + 64);
    volatile int* grid_gave_up = reinterpret_cast<volatile int*>(smem + 72);

    const int tid = threadIdx.x;
    const int wg = tid / kThreads;            // worker group of this thread
    const int tg = tid % kThreads;            // index within the group
    const int cta = (int)blockIdx.x, grid = (int)gridDim.x;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem) + wg * kMaxStages;
    const uint32_t rec_base = 80u + (uint32_t)wg * (16u * kUnitRecords);
    Walker* walker = reinterpret_cast<Walker*>(smem + 336 + 32 * wg);
    int* armed = reinterpret_cast<int*>(smem + 400 + 8 * wg);      // copies requested per ring slot
    const uint32_t stage_stride = p.stage_stride;
    const uint32_t ring0 = p.ring_off + (uint32_t)(wg * kSeqSlots) * stage_stride;
    const uint32_t partial_bytes = p.partial_bytes;
    const uint32_t group_part0 = kSeqHeader + (uint32_t)wg * 2u * partial_bytes;

    if (tid == 0) {
        for (int s = 0; s < 2 * kMaxStages; ++s) mbar_init(reinterpret_cast<uint64_t*>(smem) + s, 1);
        *copy_gave_up = 0;
        *grid_gave_up = 0;
        fence_barrier_init();
    }
    if (tg == 0) {
        Walker w;
        w.ph = -1;
        w.m = 0;
        w.v = w.vend = 0;
        w.cap = 1;
        w.claims = 0;
        w.pad[0] = w.pad[1] = 0;
        walker_next_phase(p, w, wg, cta, grid);
        *walker = w;
        armed[0] = armed[1] = 0;
    }
    __syncthreads();

    const uint64_t policy = l2_evict_first_policy();
    // Thread 0 of a group takes the group's next unit, records it for the group and requests its copy
    // into ring slot `slot`; when the list is exhausted it records zero rows.
    auto claim_and_issue = [&](int slot) {
        // (after a copy wait gave up nothing further is requested: a slot's barrier may be out of step)
        const Claim c = seq_claim(p, walker, wg, *copy_gave_up != 0, cta, grid);
        const int phase = c.phase, m = c.m, begin = c.begin, n = c.n;
        uint8_t* rec = smem + rec_base + 16u * (uint32_t)c.record_index;
        if (n > 0) {
            const SeqMat& mt = p.mat[m];
            const int row_bytes = p.ph[phase].row_bytes;
            *reinterpret_cast<float**>(rec) = mt.Y + begin;
            *reinterpret_cast<int*>(rec + 8) = n;
            *reinterpret_cast<int*>(rec + 12) = phase;
            const uint32_t bytes = (uint32_t)(n * row_bytes);
            mbar_expect_tx(&full[slot], bytes);
            bulk_load(smem + ring0 + (uint32_t)slot * stage_stride, mt.W + (int64_t)begin * row_bytes, bytes, &full[slot],
                      policy);
            ++armed[slot];
        } else {
            *reinterpret_cast<float**>(rec) = nullptr;
            *reinterpret_cast<int*>(rec + 8) = 0;
            *reinterpret_cast<int*>(rec + 12) = p.n_phases;
        }
    };
    if (tg == 0)
        for (int s = 0; s < kSeqSlots; ++s) claim_and_issue(s);
    __syncthreads();              // the first unit records are visible to the groups' threads

    // ---- per-phase state of a thread (set by enter_phase) ----
    typename T::X xr;
    typename T::Ctx ctx{};
    int units = 1, rows_per_wave = 1;
    int wave_bytes = 0, wave_part_bytes = 0;
    uint32_t row_off0 = 0, part_off0 = 0;
    bool active = false;
    int my_row_slot = 0;
    int sel = 0;
    // completion of a unit's rows from the partial table by one warp (see the single-launch kernel)
    bool fin_fast = false;
    int vec_shift = -1, fin_lpr_shift = 0, fin_vpl = 1, fin_row = 0, fin_first = 0;
    FinishShape fshape{1, -1};
    const int fin_lane = tid & 31;
    const bool fin_warp = (tg >> 5) == kThreads / 32 - 1;

    // Everything a CTA does between two phases.  Run by all threads of the CTA, once per phase, in order.
    auto enter_phase = [&](int phase) {
        const SeqPhase& P = p.ph[phase];
        LW_SEQ_STAMP(phase, 0);
        __syncthreads();          // both groups have finished (and written the results of) everything before this phase
        LW_SEQ_STAMP(phase, 4);
        if (P.dep_index > 0) {
            if (tid == kBarrierThread) {      // not a producer thread: its fence must not wait behind copies in flight
                // arrival with release semantics: everything the CTA wrote before the barrier above (its
                // threads are ordered before this one by that barrier) is visible device-wide to whoever
                // observes the count with an acquire load
                asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.counter) : "memory");
                if (*grid_gave_up == 0) {
                    const unsigned target = (unsigned)P.dep_index * (unsigned)grid;
                    unsigned seen = 0;
                    for (uint32_t i = 0; i < kGridSpinLimit; ++i) {
                        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(p.counter) : "memory");
                        if (seen >= target) break;
                    }
                    LW_SEQ_STAMP(phase, 5);
                    if (seen < target) {
                        *grid_gave_up = 1;
                        atomicExch(p.fault, (int)FAULT_GRID_BARRIER_TIMEOUT);
                    }
                }
            }
            __syncthreads();
        }
        LW_SEQ_STAMP(phase, 1);
        int v0, v1;
        share_of(P, cta, grid, v0, v1);
        if (v1 == v0) return;     // no rows of this phase here (the same answer for every thread of the CTA)
        units = P.units;
        rows_per_wave = P.rows_per_wave;
        const int row_bytes = P.row_bytes;
        const int cols = units * 64;
        const Mapping m = T::map(tg, units, rows_per_wave);
        if constexpr (T::kIntegerDot) {
            uint32_t* xq = reinterpret_cast<uint32_t*>(smem + p.x_off);
            seq_convert_activations<T::X::kGroups == 2 ? 32 : 16, T::kXqQ4KLayout>(P.X, cols, xq, tid);
            __syncthreads();
            xr.load(xq + xq_unit_offset<T::kXqQ4KLayout>(m.col_slot), m.active);
        } else {
            // fp32 activations: staged in shared memory in padded chunks, then 64 values per thread into registers
            float* xs = reinterpret_cast<float*>(smem + p.x_off);
            for (int i = tid; i < cols / 4; i += 2 * kThreads) {
                const float4 v = __ldcg(reinterpret_cast<const float4*>(P.X) + i);
                *reinterpret_cast<float4*>(xs + x_padded_index<T>((int64_t)i * 4)) = v;
            }
            __syncthreads();
            xr.load(
                [&](int i) {
                    return *reinterpret_cast<const float4*>(xs + x_padded_index<T>(T::x_index(m.col_slot, units, i)));
                },
                m.active);
        }
        LW_SEQ_STAMP(phase, 2);
        T::finish_x(xr);
        ctx = T::make_ctx(m.col_slot, units);
        if constexpr (T::kSplitByGroup) sel = T::split_sel(ctx);
        active = m.active;
        my_row_slot = m.row_slot;
        wave_bytes = rows_per_wave * row_bytes;
        wave_part_bytes = rows_per_wave * units * 4;
        row_off0 = ring0 + (uint32_t)(m.row_slot * row_bytes);
        part_off0 = group_part0 + (uint32_t)(m.row_slot * units + m.col_slot) * 4u;
        fshape = finish_shape(units);
        vec_shift = fshape.vec_shift;
        fin_fast = vec_shift >= 0 && P.unit_cap <= 32;
        fin_lpr_shift = 0;
        if (fin_fast)
            while (fin_lpr_shift < vec_shift && (P.unit_cap << (fin_lpr_shift + 1)) <= 32) ++fin_lpr_shift;
        fin_vpl = fin_fast ? 1 << (vec_shift - fin_lpr_shift) : 1;
        fin_row = fin_lane >> fin_lpr_shift;
        fin_first = fin_fast ? (fin_row << vec_shift) + (fin_lane & ((1 << fin_lpr_shift) - 1)) * fin_vpl : 0;
        LW_SEQ_STAMP(phase, 3);
    };

    // The products of one unit: this thread's rows of the stage against its 64 activations.
    auto compute_unit = [&](auto sel_tag, int n, uint32_t slot_off, uint32_t buf_off) {
        constexpr int SEL = decltype(sel_tag)::value;
        uint32_t roff = row_off0 + slot_off;
        uint32_t poff = part_off0 + buf_off;
        int r = my_row_slot;
        if constexpr (T::kPairRows) {
            // two rows at a time give the scheduler two independent dependency chains to interleave
            for (; r + rows_per_wave < n; r += 2 * rows_per_wave) {
                const float a = T::template dot<SEL>(smem + roff, ctx, xr);
                const float b = T::template dot<SEL>(smem + roff + wave_bytes, ctx, xr);
                *reinterpret_cast<float*>(smem + poff) = a;
                *reinterpret_cast<float*>(smem + poff + wave_part_bytes) = b;
                roff += 2 * wave_bytes;
                poff += 2 * wave_part_bytes;
            }
        }
        for (; r < n; r += rows_per_wave) {
            *reinterpret_cast<float*>(smem + poff) = T::template dot<SEL>(smem + roff, ctx, xr);
            roff += wave_bytes;
            poff += wave_part_bytes;
        }
    };

    const uint32_t full_addr = smem_u32(full);
    int cur_phase = -1;
    int consumed = 0;
    int slot = 0;
    uint32_t parity = 0, slot_off = 0, buf_off = 0, rec_off = 0;
    bool gave_up = false;
    for (;;) {
        const uint32_t rec = rec_base + rec_off;
        const int n = *reinterpret_cast<const int*>(smem + rec + 8);
        if (n == 0) break;                      // the CTA's list ran dry when this slot was last refilled
        const int phase = *reinterpret_cast<const int*>(smem + rec + 12);
        while (cur_phase < phase) enter_phase(++cur_phase);
        if (!gave_up && !mbar_wait_bounded(full_addr + 8u * slot, parity)) {     // after one failure, stop waiting
            gave_up = true;
            *copy_gave_up = 1;
            atomicExch(p.fault, (int)FAULT_BULK_WAIT_TIMEOUT);
        }
        if (active) {
            if constexpr (T::kSplitByGroup) {
                if (sel == 0) compute_unit(std::integral_constant<int, 0>{}, n, slot_off, buf_off);
                else compute_unit(std::integral_constant<int, 1>{}, n, slot_off, buf_off);
            } else {
                compute_unit(std::integral_constant<int, -1>{}, n, slot_off, buf_off);
            }
        }
        group_barrier<2>(wg);                   // stage consumed by the group; partials visible
        if (tg == 0) claim_and_issue(slot);
        if (fin_fast) {
            if (fin_warp) {
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                const float4* run = reinterpret_cast<const float4*>(smem + group_part0 + buf_off) + fin_first;
                if (fin_row < n) {              // lanes beyond the unit's rows idle
                    for (int j = 0; j < fin_vpl; ++j) {
                        const float4 v = run[(j + fin_lane) & (fin_vpl - 1)];
                        acc.x += v.x;
                        acc.y += v.y;
                        acc.z += v.z;
                        acc.w += v.w;
                    }
                }
                float sum = (acc.x + acc.y) + (acc.z + acc.w);
                for (int off = 1; off < (1 << fin_lpr_shift); off <<= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, off);
                if ((fin_lane & ((1 << fin_lpr_shift) - 1)) == 0 && fin_row < n)
                    (*reinterpret_cast<float* const*>(smem + rec))[fin_row] = sum;
            }
        } else {
            finish_stage(reinterpret_cast<const float*>(smem + group_part0 + buf_off), n, fshape,
                         *reinterpret_cast<float* const*>(smem + rec), tg);
        }
        ++consumed;
        rec_off = (rec_off + 16u) & (16u * kUnitRecords - 16u);
        buf_off = buf_off ? 0u : partial_bytes;
        slot_off += stage_stride;
        if (++slot == kSeqSlots) {
            slot = 0;
            slot_off = 0;
            parity ^= 1u;
        }
    }
    // the phases left (none of this group's units are in them) still need this CTA at their barriers
    while (cur_phase < p.n_phases - 1) enter_phase(++cur_phase);
    // If a wait gave up, copies may still be landing: give each slot that has a copy outstanding one
    // more bounded wait so that shared memory is not released under a copy in flight.
    if (*copy_gave_up && tg == 0) {
        for (int s = 0; s < kSeqSlots; ++s) {
            if (armed[s] == 0) continue;
            if (!mbar_wait_bounded(&full[s], (uint32_t)(armed[s] - 1) & 1u)) atomicExch(p.fault, (int)FAULT_DRAIN_TIMEOUT);
        }
    }
}

// ------------------------------------------------------------------ host side ---

int seq_sm_count() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    return n;
}

constexpr size_t kSeqSmemMax = 227 * 1024;

struct SeqShape {
    int units, row_bytes, rows_per_wave;
    size_t x_bytes;
};

bool seq_shape(int fmt, int64_t cols, SeqShape& sh) {
    if (fmt < LW_F16 || fmt > LW_Q5_1) return false;
    if (cols % 256 != 0 || cols / 64 > kThreads) return false;
    const int64_t rb = (int64_t)lw_row_bytes(fmt, cols);
    if (rb == 0 || rb % 16 != 0) return false;                  // bulk copies move whole rows
    const bool kquant = fmt == LW_Q4_K || fmt == LW_Q6_K || fmt == LW_Q5_K || fmt == LW_Q2_K;
    sh.units = (int)(cols / 64);
    sh.row_bytes = (int)rb;
    sh.rows_per_wave = kquant ? (kThreads / 4) / (sh.units / 4) : kThreads / sh.units;
    if (sh.rows_per_wave < 1) return false;
    if (fmt == LW_F16) sh.x_bytes = (size_t)cols * 4u;
    else sh.x_bytes = ((size_t)sh.units * kXqUnitWords + (kquant ? (size_t)(sh.units / 4) * 4 : 0)) * 4u;
    return true;
}

template <class T>
int launch_seq(const SeqParams& sp, int grid, size_t smem_bytes, cudaStream_t stream) {
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return (int)e;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        e = cudaFuncSetAttribute(matvec_seq_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSeqSmemMax);
        if (e != cudaSuccess) return (int)e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(2 * kThreads);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;      // all CTAs resident at once: they wait for one another
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return (int)cudaLaunchKernelEx(&cfg, matvec_seq_kernel<T>, sp);
}

}  // namespace

#ifdef LW_SEQ_TRACE
extern "C" int lw_debug_seq_trace(unsigned long long* out, int n_phases) {
    return (int)cudaMemcpyFromSymbol(out, g_seq_trace, sizeof(unsigned long long) * 3 * kSeqMaxPhases * kTraceEvents);
}
#endif

bool matvec_sequence_supported(int fmt, int n_items, const lw_seq_item* items) {
    if (n_items < 1 || n_items > kSeqMaxMats) return false;
    SeqShape sh;
    int phases = 0;
    for (int j = 0; j < n_items; ++j) {
        if (!seq_shape(fmt, items[j].cols, sh)) return false;
        if (items[j].rows > (1 << 22)) return false;            // shares are computed in 32-bit arithmetic
        const bool joins = j > 0 && !(items[j].flags & LW_SEQ_DEPENDENT) && items[j].X == items[j - 1].X &&
                           items[j].cols == items[j - 1].cols;
        if (!joins) ++phases;
    }
    return phases <= kSeqMaxPhases;
}

// Arguments are validated (pointers, alignment, shapes); returns a cudaError_t as int.
int launch_matvec_sequence(int fmt, int n_items, const lw_seq_item* items, unsigned* counter, cudaStream_t stream) {
    const int grid = seq_sm_count();
    if (grid <= 0) return (int)cudaErrorInvalidDevice;
    int* fault = device_fault_word();
    if (!fault) return (int)cudaErrorInvalidValue;
    static thread_local SeqParams sp;          // 29 KB: kept off the stack
    sp.n_phases = 0;
    sp.n_mats = n_items;
    sp.counter = counter;
    sp.fault = fault;
    int deps = 0;
    std::vector<SeqShape> shapes;
    for (int j = 0; j < n_items; ++j) {
        SeqShape sh;
        if (!seq_shape(fmt, items[j].cols, sh)) return (int)cudaErrorInvalidValue;
        const bool dependent = (items[j].flags & LW_SEQ_DEPENDENT) != 0 && j > 0;
        const bool joins = j > 0 && !dependent && items[j].X == items[j - 1].X && items[j].cols == items[j - 1].cols;
        if (!joins) {
            if (sp.n_phases == kSeqMaxPhases) return (int)cudaErrorInvalidValue;
            SeqPhase& P = sp.ph[sp.n_phases++];
            P.X = items[j].X;
            P.units = sh.units;
            P.row_bytes = sh.row_bytes;
            P.rows_per_wave = sh.rows_per_wave;
            P.unit_cap = 0;
            P.total_rows = 0;
            P.first_mat = j;
            P.dep_index = dependent ? ++deps : 0;
            P.pad = 0;
            shapes.push_back(sh);
        }
        SeqPhase& P = sp.ph[sp.n_phases - 1];
        SeqMat& M = sp.mat[j];
        M.W = static_cast<const uint8_t*>(items[j].W_blocks);
        M.Y = items[j].Y;
        M.rows = (int)items[j].rows;
        M.vrow0 = P.total_rows;
        if ((int64_t)P.total_rows + items[j].rows > (1 << 22)) return (int)cudaErrorInvalidValue;
        P.total_rows += (int)items[j].rows;
    }
    // Ring slot size: the largest target (KB) for which header, partial tables, activations and the four
    // slots fit in shared memory; bulk copies below ~32 KB lose HBM efficiency, so start high.
    size_t x_bytes = 0;
    for (const SeqShape& sh : shapes) x_bytes = std::max(x_bytes, sh.x_bytes);
    x_bytes = (x_bytes + 127) & ~(size_t)127;
    size_t smem_bytes = 0;
    bool fits = false;
    for (int target_kb = 40; target_kb >= 8 && !fits; target_kb -= 2) {
        size_t stride = 0, partial = 0;
        for (int i = 0; i < sp.n_phases; ++i) {
            SeqPhase& P = sp.ph[i];
            int cap = (int)((int64_t)target_kb * 1024 / P.row_bytes) / P.rows_per_wave * P.rows_per_wave;
            if (cap < P.rows_per_wave) cap = P.rows_per_wave;
            P.unit_cap = cap;
            stride = std::max(stride, (size_t)cap * (size_t)P.row_bytes);
            partial = std::max(partial, (size_t)cap * (size_t)P.units * 4u);
        }
        stride = (stride + 127) & ~(size_t)127;
        partial = (partial + 127) & ~(size_t)127;
        const size_t x_off = kSeqHeader + 4 * partial;
        const size_t ring_off = x_off + x_bytes;
        smem_bytes = ring_off + 2 * kSeqSlots * stride;
        if (smem_bytes <= kSeqSmemMax) {
            fits = true;
            sp.x_off = (uint32_t)x_off;
            sp.ring_off = (uint32_t)ring_off;
            sp.stage_stride = (uint32_t)stride;
            sp.partial_bytes = (uint32_t)partial;
        }
    }
    if (!fits) return (int)cudaErrorInvalidValue;
    cudaError_t e = cudaMemsetAsync(counter, 0, sizeof(unsigned), stream);
    if (e != cudaSuccess) return (int)e;
    switch (fmt) {
        case LW_F16: return launch_seq<StreamF16>(sp, grid, smem_bytes, stream);
        case LW_Q8_0: return launch_seq<IdotQ80>(sp, grid, smem_bytes, stream);
        case LW_Q4_0: return launch_seq<IdotQ40>(sp, grid, smem_bytes, stream);
        case LW_Q4_K: return launch_seq<IdotQ4K>(sp, grid, smem_bytes, stream);
        case LW_Q6_K: return launch_seq<IdotQ6K>(sp, grid, smem_bytes, stream);
        case LW_Q5_K: return launch_seq<IdotQ5K>(sp, grid, smem_bytes, stream);
        case LW_Q2_K: return launch_seq<IdotQ2K>(sp, grid, smem_bytes, stream);
        case LW_Q4_1: return launch_seq<IdotQ41>(sp, grid, smem_bytes, stream);
        case LW_Q5_0: return launch_seq<IdotQ50>(sp, grid, smem_bytes, stream);
        case LW_Q5_1: return launch_seq<IdotQ51>(sp, grid, smem_bytes, stream);
    }
    return (int)cudaErrorInvalidValue;
}

}  // namespace lw
