// Streaming mat-vec variants for batch 1 (the decode hot path) on sm_100a.
//
// Design, following the paper's decode kernel in spirit [Sec 3.2: the activation vector is tiled
// into registers and each row is reduced cooperatively; Sec 3.3: weights are decoded straight into
// registers, never staged decoded in shared memory] but built for B200:
//   * Each CTA owns a contiguous range of rows.  Rows are contiguous in memory, so a slab of rows is
//     one contiguous byte range: a single thread streams slab after slab into a ring of shared
//     memory stages with 1-D bulk async copies (cp.async.bulk + mbarrier, L2 evict-first), keeping
//     tens of KB per SM in flight without spending registers on it.
//   * Every thread owns a fixed 64-weight column unit of the row and keeps the matching 64
//     activations in registers for the whole kernel, so the inner loop touches shared memory only
//     for the raw quantised bytes.
//   * Two families of per-format decode routines share that skeleton:
//       - "Stream*": activations stay fp32 (32 packed pairs for fma.rn.f32x2).  4-bit formats never
//         convert integers: a nibble is dropped into the mantissa of 128.0f with one byte-permute
//         (giving 128 + q exactly) and the offset / block scale is applied once per 32-weight block.
//       - "Idot*": activations are converted once per kernel to 24-bit block fixed point (three byte
//         planes) and the products run on dp4a, four weights per instruction, with exact integer
//         sums that are scaled once per block.  This halves the work on the integer pipe, which is
//         what bounds the 4-bit formats on this GPU.
//   * Row sums are completed through a small shared-memory partial table, one CTA barrier per stage.
// All waits are bounded: a wait that gives up records a fault code and the kernel still terminates.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdlib>
#include <type_traits>
#include <vector>

#include "lw_internal.h"
#include "lw_stream_common.cuh"

namespace lw {

__device__ int g_fault_word = 0;

int* device_fault_word() {
    int* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_fault_word) != cudaSuccess) return nullptr;
    return p;
}

namespace {

// Optional phase timestamps for profiling builds (define LW_STAMP(i) before including this file).
#ifndef LW_STAMP
#define LW_STAMP(i)
#endif

// ------------------------------------------------------------------ kernel ---

struct StreamParams {
    const uint8_t* W;
    const float* X;
    float* Y;
    int* fault;
    int64_t rows;
    int64_t cols;
    int64_t row_bytes;
    int units_per_row;    // cols / 64
    int rows_per_wave;    // rows processed concurrently by the CTA
    int stage_rows;       // rows per ring stage (a multiple of rows_per_wave)
    int waves;            // stage_rows / rows_per_wave
    int stages;           // ring depth
    int rows_per_cta;
    uint32_t stage_stride;   // bytes between ring stages in shared memory (multiple of 128)
    uint32_t x_off;          // byte offset of the staged activations in shared memory
    uint32_t ring_off;       // byte offset of the ring
    int batch;               // activation columns handled by this launch (batched kernel only)
    // Grouped launches: several independent matrices (same format and cols) in one grid.  Item j owns
    // the CTAs [first_cta, next item's first_cta); n_items == 0 means the single matrix above.
    int n_items;
    struct Item {
        const uint8_t* W;
        const float* X;
        float* Y;
        int64_t rows;
        int first_cta;
        int rows_per_cta;
    } items[kMaxGroup];
    uint32_t xq_col_words;   // words between the fixed-point activations of consecutive columns
    int drop_unit;           // testing aid: the unit (index in the CTA's pool) whose copy is never requested; -1 = none
};

// One CTA holds NG worker groups of kThreads threads.  The groups share the converted activations
// and a pool of row ranges ("units", one ring stage each) cut from the CTA's rows; each group has its
// own ring, partial tables and barrier, and claims the next unit whenever one of its ring slots
// falls free.  With NG == 2 the CTA fills an SM on its own: the activations are fetched and converted
// once per SM, and the two groups finish within one stage of each other whatever share of the issue
// slots the warp schedulers give them (two independent CTAs on an SM do not: the older one is favoured
// and the younger one runs its last quarter alone at half the SM's throughput).
// DROP builds the testing aid of lw_debug_drop_copy into the kernel (one copy is never requested); the kernels
// that serve ordinary calls are built without it, so it costs them nothing.
template <class T, int NG, bool DROP = false>
__global__ void __launch_bounds__(NG* kThreads, NG == 1 ? T::kMinCtas : 1)
    matvec_stream_kernel(const StreamParams p) {
    extern __shared__ __align__(128) uint8_t smem[];
    // layout: [0,64) ring barriers | 64 x barrier | 72 timeout flag | 76 unit counter |
    //         [80,336) unit records (where the rows go, how many), 16 bytes each, kUnitRecords per group |
    //         partial tables | activations | rings
    uint64_t* xbar = reinterpret_cast<uint64_t*>(smem + 64);
    volatile int* timed_out = reinterpret_cast<volatile int*>(smem + 72);
    int* unit_counter = reinterpret_cast<int*>(smem + 76);
    volatile int* copy_dropped = reinterpret_cast<volatile int*>(smem + 336);    // behind the unit records
    const int partial_stride = p.stage_rows * p.units_per_row;      // floats per buffer
    float* xs = reinterpret_cast<float*>(smem + p.x_off);

    const int tid = threadIdx.x;
    const int wg = NG == 1 ? 0 : tid / kThreads;        // worker group of this thread
    const int tg = NG == 1 ? tid : tid % kThreads;      // index within the group
    uint64_t* full = reinterpret_cast<uint64_t*>(smem) + wg * kMaxStages;
    // The unit a group consumes in its i-th stage is described by record i % kUnitRecords, written by
    // the group's thread 0 when it queues the copy (at least one group barrier before it is read).
    const uint32_t rec_base = 80u + (uint32_t)wg * (16u * kUnitRecords);
    // which matrix this CTA works on (grouped launches), and its row range there
    const uint8_t* Wm = p.W;
    const float* Xm = p.X;
    float* Ym = p.Y;
    int64_t rows_m = p.rows;
    int rpc = p.rows_per_cta, cta = (int)blockIdx.x;
    if (p.n_items > 0) {
        int j = 0;
        while (j + 1 < p.n_items && cta >= p.items[j + 1].first_cta) ++j;
        Wm = p.items[j].W;
        Xm = p.items[j].X;
        Ym = p.items[j].Y;
        rows_m = p.items[j].rows;
        rpc = p.items[j].rows_per_cta;
        cta -= p.items[j].first_cta;
    }
    const int64_t row0 = (int64_t)cta * rpc;
    int rows_here = (int)(rows_m - row0 > rpc ? rpc : rows_m - row0);   // rpc is an int, so this fits
    if (rows_m - row0 < 0) rows_here = 0;
    // Launch constants used by the stage loop, in registers.
    const int stage_rows = p.stage_rows, n_slots = p.stages, units = p.units_per_row;
    const int rows_per_wave = p.rows_per_wave;
    const int row_bytes = (int)p.row_bytes;
    const uint32_t stage_stride = p.stage_stride;
    uint8_t* ring = smem + p.ring_off + (uint32_t)(wg * n_slots) * stage_stride;
    // Units of the CTA's rows.  When every group gets more than one stage, each group's first unit
    // is a single wave, so that the first products can start as soon as a few KB have landed; every
    // later unit holds stage_rows rows (the last one what is left).
    const int n_short = rows_here > NG * stage_rows ? NG : 0;
    const int short_rows = n_short * rows_per_wave;
    const int n_units = n_short + (rows_here - short_rows + stage_rows - 1) / stage_rows;
    const uint8_t* wbase = Wm + row0 * p.row_bytes;

    LW_STAMP(0);
    if (tid == 0) {
        for (int s = 0; s < NG * kMaxStages; ++s) mbar_init(reinterpret_cast<uint64_t*>(smem) + s, 1);
        mbar_init(xbar, 1);
        *timed_out = 0;
        *unit_counter = 0;
        if constexpr (DROP) *copy_dropped = 0;
        fence_barrier_init();
    }
    __syncthreads();
    grid_launch_dependents();     // lets the next kernel on the stream start its own prologue early

    const uint64_t policy = l2_evict_first_policy();
    // Thread 0 of a group claims the next unit for ring slot `slot`, records it for the group and
    // queues its copy; a slot with no unit left records zero rows.
    int next_unit = 0;            // NG == 1: the group's own cursor
    int claims = 0;               // units this thread has asked for (thread 0 of the group only)
    auto claim_and_issue = [&](int slot) {
        int k;
        if constexpr (NG == 1) k = next_unit++;
        else k = atomicAdd(unit_counter, 1);
        int begin = 0, n = 0;
        bool open = true;
        if constexpr (DROP) open = *copy_dropped == 0;
        if (k < n_units && open) {
            begin = k < n_short ? k * rows_per_wave : short_rows + (k - n_short) * stage_rows;
            n = rows_here - begin;
            const int cap = k < n_short ? rows_per_wave : stage_rows;
            if (n > cap) n = cap;
        }
        // Testing aid: the copy of one unit is never requested, so the wait for it must run out.  Nothing
        // is queued in the CTA after that (no later copy can land in a slot whose barrier is out of
        // step), and the rows of the units left over are not computed.
        bool drop = false;
        if constexpr (DROP) {
            drop = n > 0 && k == p.drop_unit;
            if (drop) *copy_dropped = 1;
        }
        {
            uint8_t* rec = smem + rec_base + 16u * (uint32_t)(claims & (kUnitRecords - 1));
            *reinterpret_cast<float**>(rec) = Ym + row0 + begin;
            *reinterpret_cast<int*>(rec + 8) = n;
            ++claims;
        }
        if (n > 0 && !drop) {
            const uint32_t bytes = (uint32_t)(n * row_bytes);
            mbar_expect_tx(&full[slot], bytes);
            bulk_load(ring + slot * stage_stride, wbase + (int64_t)begin * row_bytes, bytes, &full[slot], policy);
        }
    };
    auto issue_prologue = [&]() {
        for (int s = 0; s < n_slots; ++s) claim_and_issue(s);
    };

    LW_STAMP(1);
    grid_dependency_wait();       // X may be produced, and Y still read, by the previous kernel
    LW_STAMP(2);

    // Activations first, weights right behind them: the activation requests must not queue behind
    // a ring's worth of weight traffic, because nothing can be computed before they arrive.
    const Mapping m = T::map(tg, units, rows_per_wave);
    typename T::X xr;
    if constexpr (T::kIntegerDot) {
        // Cooperative conversion to block fixed point straight from global memory (coalesced).
        uint32_t* xq = reinterpret_cast<uint32_t*>(xs);
        bool issued = false;
        // at most one run per thread (up to 8192 columns): a quarter of the code to fetch and execute
        auto after_loads = [&]() {
            if (tg == 0) {
                issue_prologue();
                issued = true;
            }
        };
        if ((p.cols >> 4) <= NG * kThreads)
            quantize_activations<T::X::kGroups == 2 ? 32 : 16, T::kXqQ4KLayout, NG * kThreads, 1>(Xm, (int)p.cols, xq, tid,
                                                                                                after_loads);
        else
            quantize_activations<T::X::kGroups == 2 ? 32 : 16, T::kXqQ4KLayout, NG * kThreads, 4>(Xm, (int)p.cols, xq, tid,
                                                                                                after_loads);
        if (tg == 0 && !issued) issue_prologue();    // no run of the vector fell to this thread
        __syncthreads();
        LW_STAMP(3);
        xr.load(xq + xq_unit_offset<T::kXqQ4KLayout>(m.col_slot), m.active);
    } else {
        // Stage the vector in shared memory with bulk copies (one per padded chunk), then every
        // thread pulls its own 64 values into registers with conflict-free 16-byte loads.
        if (tid == 0) mbar_expect_tx(xbar, (uint32_t)(p.cols * 4));
        if constexpr (T::kXChunk == 0) {
            if (tid == 0) bulk_load_default(xs, Xm, (uint32_t)(p.cols * 4), xbar);
        } else {
            const int chunks = (int)(p.cols / T::kXChunk);
            for (int c = tid; c < chunks; c += NG * kThreads)
                bulk_load_default(xs + (size_t)c * (T::kXChunk + 4), Xm + (size_t)c * T::kXChunk,
                                  T::kXChunk * 4, xbar);
        }
        if (tg == 0) issue_prologue();
        if (!mbar_wait_bounded(xbar, 0)) {
            *timed_out = 1;
            atomicExch(p.fault, (int)FAULT_BULK_WAIT_TIMEOUT);
        }
        __syncthreads();          // the groups' unit records are visible to their threads
        LW_STAMP(3);
        xr.load(
            [&](int i) {
                return *reinterpret_cast<const float4*>(
                    xs + x_padded_index<T>(T::x_index(m.col_slot, units, i)));
            },
            m.active);
    }
    T::finish_x(xr);
    LW_STAMP(4);

    const int waves = p.waves;
    const int wave_bytes = rows_per_wave * row_bytes;                   // bytes between a thread's rows
    const int wave_part_bytes = rows_per_wave * units * 4;              // partial-table bytes likewise
    const uint32_t partial_bytes = (uint32_t)partial_stride * 4u;       // one partial buffer
    // Byte offsets from the start of shared memory: this thread's first row inside its group's ring
    // slot 0, and its first partial inside the group's buffer 0.  All loop state below is 32-bit and
    // advances by additions.
    const uint32_t group_part0 = kSmemHeader + (uint32_t)wg * 2u * partial_bytes;
    const uint32_t row_off0 = p.ring_off + (uint32_t)(wg * n_slots) * stage_stride + (uint32_t)(m.row_slot * row_bytes);
    const uint32_t part_off0 = group_part0 + (uint32_t)(m.row_slot * units + m.col_slot) * 4u;
    const uint32_t full_addr = smem_u32(full);
    const FinishShape fshape = finish_shape(units);
    // Fast completion of a stage by ONE warp of the group (the others go straight on to the next
    // stage), for rows whose partials are a power-of-two number of 16-byte vectors: a row takes fin_lpr
    // lanes, each lane adds up a run of fin_vpl vectors, the lanes of a row are folded with shuffles.
    // Lanes start their runs at different vectors so that a quarter-warp's loads hit distinct banks.
    // Two forms, chosen per trait at compile time (the product loop's schedule is sensitive to the
    // code around it, so the formats tuned first keep the form they were tuned with): the first needs
    // the stage's vectors to fill the 32 lanes evenly; the second takes any stage of at most 32 rows,
    // gives a row the largest power-of-two number of lanes that fits, and idles the lanes left over.
    constexpr bool kAnyRows = any_stage_rows<T>::value;
    const int vec_shift = fshape.vec_shift;
    const int fin_total = vec_shift >= 0 ? stage_rows << vec_shift : 0;        // vectors of a full stage
    bool fin_fast;
    int fin_lpr_shift = 0, fin_vpl;
    if constexpr (kAnyRows) {
        fin_fast = vec_shift >= 0 && stage_rows <= 32;
        if (fin_fast)
            while (fin_lpr_shift < vec_shift && (stage_rows << (fin_lpr_shift + 1)) <= 32) ++fin_lpr_shift;
        fin_vpl = fin_fast ? 1 << (vec_shift - fin_lpr_shift) : 1;
    } else {
        fin_vpl = fin_total >> 5;
        fin_fast = vec_shift >= 0 && (fin_total & 31) == 0 && fin_vpl >= 1 &&
                   (fin_vpl & (fin_vpl - 1)) == 0 && fin_vpl <= (1 << vec_shift);
        fin_lpr_shift = fin_fast ? vec_shift - (31 - __clz(fin_vpl)) : 0;
    }
    const int fin_lpr = 1 << fin_lpr_shift;
    const int fin_lane = tid & 31;
    const int fin_row = fin_lane >> fin_lpr_shift;
    const int fin_first = kAnyRows && fin_fast ? (fin_row << vec_shift) + (fin_lane & (fin_lpr - 1)) * fin_vpl
                                               : fin_lane * fin_vpl;
    const bool fin_warp = (tg >> 5) == kThreads / 32 - 1;
    const typename T::Ctx ctx = T::make_ctx(m.col_slot, units);
    const bool active = m.active;
    const int my_row_slot = m.row_slot;
    int consumed = 0;             // stages this group went through
    auto main_loop = [&](auto sel_tag) {
        constexpr int SEL = decltype(sel_tag)::value;
        int slot = 0;
        uint32_t parity = 0, slot_off = 0, buf_off = 0, rec_off = 0;
        bool gave_up = false;
        for (;;) {
            const uint32_t rec = rec_base + rec_off;
            const int rows_in_stage = *reinterpret_cast<const int*>(smem + rec + 8);
            if (rows_in_stage == 0) break;          // the pool ran dry when this slot was last refilled
            if (!gave_up && !mbar_wait_bounded(full_addr + 8u * slot, parity)) {   // after one failure, stop waiting
                gave_up = true;
                *timed_out = 1;
                atomicExch(p.fault, (int)FAULT_BULK_WAIT_TIMEOUT);
            }
            if (consumed == 0) { LW_STAMP(5); }
            if (active) {
                // running offsets: one add per wave instead of a multiply per product
                uint32_t roff = row_off0 + slot_off;
                uint32_t poff = part_off0 + buf_off;
                int w = 0;
                if (rows_in_stage == stage_rows) {
                    // full stage: no bounds checks; two rows at a time give the scheduler two independent
                    // dependency chains to interleave
                    if constexpr (T::kPairRows) {
                    for (; w + 1 < waves; w += 2) {
                        const float a = T::template dot<SEL>(smem + roff, ctx, xr);
                        const float b = T::template dot<SEL>(smem + roff + wave_bytes, ctx, xr);
                        *reinterpret_cast<float*>(smem + poff) = a;
                        *reinterpret_cast<float*>(smem + poff + wave_part_bytes) = b;
                        roff += 2 * wave_bytes;
                        poff += 2 * wave_part_bytes;
                    }
                    if (w < waves) *reinterpret_cast<float*>(smem + poff) = T::template dot<SEL>(smem + roff, ctx, xr);
                    } else {
                    for (; w < waves; ++w) {
                        *reinterpret_cast<float*>(smem + poff) = T::template dot<SEL>(smem + roff, ctx, xr);
                        roff += wave_bytes;
                        poff += wave_part_bytes;
                    }
                    }
                } else {
                    for (int r = my_row_slot; r < rows_in_stage; r += rows_per_wave) {
                        *reinterpret_cast<float*>(smem + poff) = T::template dot<SEL>(smem + roff, ctx, xr);
                        roff += wave_bytes;
                        poff += wave_part_bytes;
                    }
                }
            }
            group_barrier<NG>(wg);                 // stage consumed by the group; partials visible
            if (tg == 0) claim_and_issue(slot);
            if (fin_fast) {
                if (fin_warp) {
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                    if constexpr (kAnyRows) {
                        const float4* run = reinterpret_cast<const float4*>(smem + group_part0 + buf_off) + fin_first;
                        if (fin_row < rows_in_stage) {       // lanes beyond the stage's rows idle
                            for (int j = 0; j < fin_vpl; ++j) {
                                const float4 v = run[(j + fin_lane) & (fin_vpl - 1)];
                                acc.x += v.x;
                                acc.y += v.y;
                                acc.z += v.z;
                                acc.w += v.w;
                            }
                        }
                    } else {
                        const float4* run = reinterpret_cast<const float4*>(smem + group_part0 + buf_off) + fin_lane * fin_vpl;
                        for (int j = 0; j < fin_vpl; ++j) {
                            const float4 v = run[(j + fin_lane) & (fin_vpl - 1)];
                            acc.x += v.x;
                            acc.y += v.y;
                            acc.z += v.z;
                            acc.w += v.w;
                        }
                    }
                    float sum = (acc.x + acc.y) + (acc.z + acc.w);
                    for (int off = 1; off < fin_lpr; off <<= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, off);
                    if ((fin_lane & (fin_lpr - 1)) == 0 && fin_row < rows_in_stage)
                        (*reinterpret_cast<float* const*>(smem + rec))[fin_row] = sum;
                }
            } else {
                finish_stage(reinterpret_cast<const float*>(smem + group_part0 + buf_off), rows_in_stage, fshape,
                             *reinterpret_cast<float* const*>(smem + rec), tg);
            }
            ++consumed;
            rec_off = (rec_off + 16u) & (16u * kUnitRecords - 16u);
            buf_off = buf_off ? 0u : partial_bytes;
            slot_off += stage_stride;
            if (++slot == n_slots) {
                slot = 0;
                slot_off = 0;
                parity ^= 1u;
            }
        }
    };
    if constexpr (T::kSplitByGroup) {
        if (T::split_sel(ctx) == 0) main_loop(std::integral_constant<int, 0>{});
        else main_loop(std::integral_constant<int, 1>{});
    } else {
        main_loop(std::integral_constant<int, -1>{});
    }
    LW_STAMP(6);
    // If a wait gave up, copies may still be landing: give each of the group's barriers one more
    // bounded wait so that shared memory is not released under a copy in flight.
    if (*timed_out && tg == 0) {
        for (int it = (consumed > n_slots ? consumed - n_slots : 0); it < consumed; ++it)
            if (!mbar_wait_bounded(&full[it % n_slots], (uint32_t)(it / n_slots) & 1u))
                atomicExch(p.fault, (int)FAULT_DRAIN_TIMEOUT);
        if constexpr (!T::kIntegerDot)
            if (!mbar_wait_bounded(xbar, 0)) atomicExch(p.fault, (int)FAULT_DRAIN_TIMEOUT);
    }
}

// Batched integer-dot kernel (2..NB activation columns per launch).  Same ring and thread mapping as
// above, but the block fixed-point activations of all columns stay in shared memory: for every row
// unit the raw weight words and block scales are read and unpacked once and reused for every batch
// column (the per-column products are inlined back to back, so the compiler keeps the unpacked
// words in registers), while each column's 48 plane words are streamed from shared memory.
template <class T, int NB>
__global__ void __launch_bounds__(kThreads, 1) matvec_stream_batched_kernel(const StreamParams p) {
    extern __shared__ __align__(128) uint8_t smem[];
    uint64_t* full = reinterpret_cast<uint64_t*>(smem);
    volatile int* timed_out = reinterpret_cast<volatile int*>(smem + 64);
    float* partial = reinterpret_cast<float*>(smem + kSmemHeader);
    const int table = p.stage_rows * p.units_per_row;               // floats per (buffer, column)
    uint32_t* xq = reinterpret_cast<uint32_t*>(smem + p.x_off);
    uint8_t* ring = smem + p.ring_off;

    const int tid = threadIdx.x;
    const int64_t row0 = (int64_t)blockIdx.x * p.rows_per_cta;
    int64_t rows_here = p.rows - row0;
    if (rows_here > p.rows_per_cta) rows_here = p.rows_per_cta;
    if (rows_here < 0) rows_here = 0;
    const int n_it = (int)((rows_here + p.stage_rows - 1) / p.stage_rows);
    const uint8_t* wbase = p.W + row0 * p.row_bytes;

    if (tid == 0) {
        for (int s = 0; s < kMaxStages; ++s) mbar_init(&full[s], 1);
        *timed_out = 0;
        fence_barrier_init();
    }
    __syncthreads();
    grid_launch_dependents();
    const uint64_t policy = l2_evict_first_policy();
    auto issue = [&](int it) {
        const int64_t r = (int64_t)it * p.stage_rows;
        int64_t nrows = rows_here - r;
        if (nrows > p.stage_rows) nrows = p.stage_rows;
        const uint32_t bytes = (uint32_t)(nrows * p.row_bytes);
        uint64_t* bar = &full[it % p.stages];
        mbar_expect_tx(bar, bytes);
        bulk_load(ring + (size_t)(it % p.stages) * p.stage_stride, wbase + r * p.row_bytes, bytes, bar, policy);
    };
    grid_dependency_wait();

    for (int b = 0; b < p.batch; ++b) {
        bool issued = b > 0;
        quantize_activations<T::X::kGroups == 2 ? 32 : 16, T::kXqQ4KLayout, kThreads>(
            p.X + (int64_t)b * p.cols, (int)p.cols, xq + (size_t)b * p.xq_col_words, tid, [&]() {
                if (tid == 0 && !issued)
                    for (int it = 0; it < p.stages && it < n_it; ++it) issue(it);
                issued = true;
            });
    }
    __syncthreads();

    const Mapping m = T::map(tid, p.units_per_row, p.rows_per_wave);
    const uint32_t* my_xq = xq + xq_unit_offset<T::kXqQ4KLayout>(m.col_slot);
    const typename T::Ctx ctx = T::make_ctx(m.col_slot, p.units_per_row);
    const int waves = p.stage_rows / p.rows_per_wave;
    for (int it = 0; it < n_it; ++it) {
        const int slot = it % p.stages;
        const uint32_t parity = (uint32_t)(it / p.stages) & 1u;
        const uint8_t* stage = ring + (size_t)slot * p.stage_stride;
        int64_t rows_in_stage = rows_here - (int64_t)it * p.stage_rows;
        if (rows_in_stage > p.stage_rows) rows_in_stage = p.stage_rows;
        float* part = partial + (it & 1) * NB * table;
        if (*timed_out == 0 && !mbar_wait_bounded(&full[slot], parity)) {
            *timed_out = 1;
            atomicExch(p.fault, (int)FAULT_BULK_WAIT_TIMEOUT);
        }
        if (m.active) {
            for (int w = 0; w < waves; ++w) {
                const int r = w * p.rows_per_wave + m.row_slot;
                if (r >= rows_in_stage) break;
                const uint8_t* rowp = stage + (size_t)r * p.row_bytes;
                float acc[NB];
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    acc[b] = 0.f;
                    if (b < p.batch) {
                        typename T::X xr;
                        xr.load(my_xq + (size_t)b * p.xq_col_words, true);
                        T::finish_x(xr);
                        acc[b] = T::dot(rowp, ctx, xr);
                    }
                }
#pragma unroll
                for (int b = 0; b < NB; ++b) part[b * table + r * p.units_per_row + m.col_slot] = acc[b];
            }
        }
        __syncthreads();
        if (tid == 0 && it + p.stages < n_it) issue(it + p.stages);
        for (int b = 0; b < p.batch; ++b)
            finish_stage(part + b * table, (int)rows_in_stage, finish_shape(p.units_per_row),
                         p.Y + (int64_t)b * p.rows + row0 + (int64_t)it * p.stage_rows, tid);
    }
    if (*timed_out && tid == 0) {
        for (int it = (n_it > p.stages ? n_it - p.stages : 0); it < n_it; ++it)
            if (!mbar_wait_bounded(&full[it % p.stages], (uint32_t)(it / p.stages) & 1u))
                atomicExch(p.fault, (int)FAULT_DRAIN_TIMEOUT);
    }
}

// ------------------------------------------------------------------ host side ---

struct Plan {
    StreamParams p;
    int groups;          // worker groups of kThreads threads per CTA (1 or 2)
    unsigned grid;
    size_t smem_bytes;
    bool ok;
};

int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

// Launch heuristics [paper Sec 3.2: tunable work-group, tile and per-thread sizes chosen from a
// sweep].  Tunables: CTAs per SM, ring depth and bytes per ring stage.  The defaults below come
// from a sweep on B200 over the Llama-shaped matrices; the environment variables LW_CTAS_PER_SM,
// LW_STAGES and LW_STAGE_KB override them (read once) for further sweeps.
struct Tuning {
    int groups;        // worker groups per CTA; 0 = automatic
    int ctas_per_sm;   // 0 = automatic
    int stages;        // 0 = automatic
    int stage_kb;      // 0 = automatic
};

// Process-wide; starts from the environment, changed by set_stream_tuning (lw_set_tuning).  Plain
// ints: a change is meant to happen between launches, from the thread that launches.
Tuning& tuning_storage() {
    static Tuning t = [] {
        Tuning v{0, 0, 0, 0};
        if (const char* e = std::getenv("LW_WORKER_GROUPS")) v.groups = std::atoi(e);
        if (const char* e = std::getenv("LW_CTAS_PER_SM")) v.ctas_per_sm = std::atoi(e);
        if (const char* e = std::getenv("LW_STAGES")) v.stages = std::atoi(e);
        if (const char* e = std::getenv("LW_STAGE_KB")) v.stage_kb = std::atoi(e);
        return v;
    }();
    return t;
}
const Tuning& tuning() { return tuning_storage(); }

// Per-shape settings found by a sweep (lw_set_shape_tuning, filled from the table the sweep writes): consulted
// by make_plan for every parameter the process-wide tuning leaves to the heuristics.
struct ShapeTuning {
    int fmt;
    int64_t rows, cols;
    int groups, stages, stage_kb;
};
std::vector<ShapeTuning>& shape_table() {
    static std::vector<ShapeTuning> t;
    return t;
}

// Testing aid (lw_debug_drop_copy): the next batch-1 streaming launch leaves out the copy of one unit.
std::atomic<int>& drop_unit_storage() {
    static std::atomic<int> v{-1};
    return v;
}

constexpr size_t kSmemPerSm = 233472;      // 228 KB of shared memory per SM, 1 KB reserved per CTA
constexpr size_t kSmemMaxCta = 227 * 1024;    // largest opt-in dynamic shared memory of a CTA

Plan make_plan(int fmt, bool integer_dot, int64_t rows, int64_t cols, int num_sms) {
    Plan pl{};
    pl.ok = false;
    if (fmt < LW_F16 || fmt > LW_Q5_1) return pl;
    if (cols % 256 != 0 || cols / 64 > kThreads) return pl;
    const int units = (int)(cols / 64);
    const int64_t rb = (int64_t)lw_row_bytes(fmt, cols);
    if (rb % 16 != 0) return pl;                    // bulk copies move whole rows (q6_K: cols % 2048 == 0)
    const bool kquant = fmt == LW_Q4_K || fmt == LW_Q6_K || fmt == LW_Q5_K || fmt == LW_Q2_K;
    int rows_per_wave;
    if (kquant) rows_per_wave = (kThreads / 4) / (units / 4);   // 64 super-block slots per wave
    else rows_per_wave = kThreads / units;
    if (rows_per_wave < 1) return pl;
    const int64_t wave_bytes = rb * rows_per_wave;
    const int xchunk = kquant ? 256 : (fmt == LW_F16 ? 0 : 64);
    size_t x_bytes = (size_t)(cols + (xchunk ? 4 * (cols / xchunk) : 0)) * 4u;     // padded fp32 staging
    const bool idot = (integer_dot && fmt != LW_F16) || fmt >= LW_Q6_K;   // the later formats have the integer-dot trait only
    if (idot) x_bytes = ((size_t)units * kXqUnitWords + (kquant ? (size_t)(units / 4) * 4 : 0)) * 4u;
    Tuning tn = tuning();
    for (const ShapeTuning& e : shape_table())
        if (e.fmt == fmt && e.rows == rows && e.cols == cols) {
            if (tn.groups == 0) tn.groups = e.groups;
            if (tn.stages == 0) tn.stages = e.stages;
            if (tn.stage_kb == 0) tn.stage_kb = e.stage_kb;
        }
    // One CTA per SM made of two worker groups (512 threads) by default; LW_WORKER_GROUPS=1 selects
    // single-group CTAs instead, two per SM (the decode routines need more than 80 registers to
    // schedule well, so not three), or one per SM with larger stages for rows wider than 8192 columns.
    const int groups = tn.groups == 1 ? 1 : 2;
    const bool wide = units > 128;
    const int max_ctas = groups == 2 || wide ? 1 : 2;

    // Candidate (CTAs per SM, waves per stage, stages): prefer more CTAs per SM, then a stage of
    // about the target size, then the deepest ring that fits.
    int best_ctas = 0, best_waves = 0, best_stages = 0;
    size_t best_x_off = 0, best_ring_off = 0, best_smem = 0;
    uint32_t best_stride = 0;
    for (int ctas = max_ctas; ctas >= 1 && best_ctas == 0; --ctas) {
        if (tn.ctas_per_sm > 0 && ctas > tn.ctas_per_sm) continue;
        size_t budget = kSmemPerSm / ctas - 1024;
        if (budget > kSmemMaxCta) budget = kSmemMaxCta;
        const int target_kb = tn.stage_kb > 0 ? tn.stage_kb : (wide && groups == 1 ? 64 : 40);
        int waves = (int)((int64_t)target_kb * 1024 / wave_bytes);
        if (waves < 1) waves = 1;
        for (; waves >= 1 && best_ctas == 0; --waves) {
            const int stage_rows = waves * rows_per_wave;
            const uint32_t stride = (uint32_t)((rb * stage_rows + 127) & ~(int64_t)127);
            const size_t partial_bytes = (size_t)groups * 2u * (size_t)stage_rows * units * 4u;
            const size_t x_off = (kSmemHeader + partial_bytes + 127) & ~(size_t)127;
            const size_t ring_off = (x_off + x_bytes + 127) & ~(size_t)127;
            // two slots per group unless asked otherwise: a third one, where it fits (f16), measured
            // slower (1B f16 step 0.560 ms against 0.542 ms)
            int stages = tn.stages > 0 ? tn.stages : 2;
            if (stages > kMaxStages) stages = kMaxStages;
            if (stages < 2) stages = 2;      // a slot is refilled while the other one is being read
            while (stages > 2 && ring_off + (size_t)groups * stages * stride > budget) --stages;
            if (ring_off + (size_t)groups * stages * stride > budget) continue;
            best_ctas = ctas;
            best_waves = waves;
            best_stages = stages;
            best_x_off = x_off;
            best_ring_off = ring_off;
            best_stride = stride;
            best_smem = ring_off + (size_t)groups * stages * stride;
        }
    }
    if (best_ctas == 0) return pl;
    const int stage_rows = best_waves * rows_per_wave;
    // rows split evenly over the resident CTAs, in multiples of a wave
    const int64_t max_grid = (int64_t)num_sms * best_ctas;
    int64_t rpc = (rows + max_grid - 1) / max_grid;
    rpc = (rpc + rows_per_wave - 1) / rows_per_wave * rows_per_wave;
    const int64_t grid = (rows + rpc - 1) / rpc;
    if (rpc > INT32_MAX || grid > INT32_MAX) return pl;
    pl.p.rows = rows;
    pl.p.cols = cols;
    pl.p.row_bytes = rb;
    pl.p.units_per_row = units;
    pl.p.rows_per_wave = rows_per_wave;
    pl.p.stage_rows = stage_rows;
    pl.p.waves = best_waves;
    pl.p.stages = best_stages;
    pl.p.rows_per_cta = (int)rpc;
    pl.p.stage_stride = best_stride;
    pl.p.x_off = (uint32_t)best_x_off;
    pl.p.ring_off = (uint32_t)best_ring_off;
    pl.p.drop_unit = -1;
    pl.groups = groups;
    pl.grid = (unsigned)grid;
    pl.smem_bytes = best_smem;
    pl.ok = true;
    return pl;
}

template <class T, int NG, bool DROP = false>
int launch_groups(Plan& pl, bool overlap, cudaStream_t stream) {
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return (int)e;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        e = cudaFuncSetAttribute(matvec_stream_kernel<T, NG, DROP>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kSmemMaxCta);
        if (e != cudaSuccess) return (int)e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(pl.grid);
    cfg.blockDim = dim3(NG * kThreads);
    cfg.dynamicSmemBytes = pl.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    return (int)cudaLaunchKernelEx(&cfg, matvec_stream_kernel<T, NG, DROP>, pl.p);
}

template <class T>
int launch_one(Plan& pl, bool overlap, cudaStream_t stream) {
    // the testing aid exists in one kernel only (q4_K, two worker groups)
    if constexpr (std::is_same<T, IdotQ4K>::value)
        if (pl.p.drop_unit >= 0 && pl.groups == 2) return launch_groups<T, 2, true>(pl, overlap, stream);
    return pl.groups == 2 ? launch_groups<T, 2>(pl, overlap, stream) : launch_groups<T, 1>(pl, overlap, stream);
}

// Plan for the batched kernel: one CTA per SM, `nb` columns of fixed-point activations resident.
Plan make_plan_batched(int fmt, int64_t rows, int64_t cols, int nb, int num_sms) {
    Plan pl{};
    pl.ok = false;
    if (fmt <= LW_F16 || fmt > LW_Q4_K || cols % 256 != 0 || cols / 64 > kThreads) return pl;
    const int units = (int)(cols / 64);
    const int64_t rb = (int64_t)lw_row_bytes(fmt, cols);
    const int rows_per_wave = fmt == LW_Q4_K ? (kThreads / 4) / (units / 4) : kThreads / units;
    if (rows_per_wave < 1) return pl;
    const size_t col_words = (size_t)units * kXqUnitWords + (fmt == LW_Q4_K ? (size_t)(units / 4) * 4 : 0);
    const int64_t wave_bytes = rb * rows_per_wave;
    for (int waves = (int)(36 * 1024 / wave_bytes) > 0 ? (int)(36 * 1024 / wave_bytes) : 1; waves >= 1; --waves) {
        const int stage_rows = waves * rows_per_wave;
        const uint32_t stride = (uint32_t)((rb * stage_rows + 127) & ~(int64_t)127);
        const size_t partial_bytes = 2u * (size_t)nb * stage_rows * units * 4u;
        const size_t x_off = (kSmemHeader + partial_bytes + 127) & ~(size_t)127;
        const size_t ring_off = (x_off + (size_t)nb * col_words * 4u + 127) & ~(size_t)127;
        const size_t smem = ring_off + 2u * stride;
        if (smem > kSmemMaxCta) continue;
        int64_t rpc = (rows + num_sms - 1) / num_sms;
        rpc = (rpc + rows_per_wave - 1) / rows_per_wave * rows_per_wave;
        const int64_t grid = (rows + rpc - 1) / rpc;
        if (rpc > INT32_MAX || grid > INT32_MAX) return pl;
        pl.p.rows = rows;
        pl.p.cols = cols;
        pl.p.row_bytes = rb;
        pl.p.units_per_row = units;
        pl.p.rows_per_wave = rows_per_wave;
        pl.p.stage_rows = stage_rows;
        pl.p.waves = waves;
        pl.p.stages = 2;
        pl.p.rows_per_cta = (int)rpc;
        pl.p.stage_stride = stride;
        pl.p.x_off = (uint32_t)x_off;
        pl.p.ring_off = (uint32_t)ring_off;
        pl.p.xq_col_words = (uint32_t)col_words;
        pl.grid = (unsigned)grid;
        pl.smem_bytes = smem;
        pl.ok = true;
        return pl;
    }
    return pl;
}

template <class T, int NB>
int launch_batched_one(Plan& pl, bool overlap, cudaStream_t stream) {
    static bool attr_set[64] = {false};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return (int)e;
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        e = cudaFuncSetAttribute(matvec_stream_batched_kernel<T, NB>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kSmemMaxCta);
        if (e != cudaSuccess) return (int)e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(pl.grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = pl.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = overlap ? 1 : 0;
    return (int)cudaLaunchKernelEx(&cfg, matvec_stream_batched_kernel<T, NB>, pl.p);
}

template <class T>
int launch_batched_fmt(Plan& pl, int nb, bool overlap, cudaStream_t stream) {
    return nb <= 2 ? launch_batched_one<T, 2>(pl, overlap, stream) : launch_batched_one<T, 4>(pl, overlap, stream);
}

// Largest number of resident activation columns (4, 2 or 1) for which the batched kernel fits.
int batched_columns(int fmt, int64_t rows, int64_t cols) {
    for (int nb = 4; nb >= 1; nb >>= 1)
        if (make_plan_batched(fmt, rows, cols, nb, 148).ok) return nb;
    return 0;
}

}  // namespace

void set_drop_unit(int unit) { drop_unit_storage().store(unit < 0 ? -1 : unit); }
int take_drop_unit() { return drop_unit_storage().exchange(-1); }

void set_shape_tuning(int fmt, int64_t rows, int64_t cols, int worker_groups, int stages, int stage_kb) {
    std::vector<ShapeTuning>& t = shape_table();
    for (size_t i = 0; i < t.size(); ++i)
        if (t[i].fmt == fmt && t[i].rows == rows && t[i].cols == cols) {
            t.erase(t.begin() + (long)i);
            break;
        }
    if (worker_groups != 0 || stages != 0 || stage_kb != 0) t.push_back(ShapeTuning{fmt, rows, cols, worker_groups, stages, stage_kb});
}

void clear_shape_tuning() { shape_table().clear(); }

void set_stream_tuning(int worker_groups, int stages, int stage_kb) {
    Tuning& t = tuning_storage();
    t.groups = worker_groups;
    t.stages = stages;
    t.stage_kb = stage_kb;
}

// Geometry the launch heuristics pick for a shape under the current tuning (for reports).
bool stream_plan_info(int fmt, int64_t rows, int64_t cols, int* groups, int* stages, int* stage_rows, int* stage_bytes,
                      int* grid, int* smem_bytes) {
    const Plan pl = make_plan(fmt, true, rows, cols, sm_count());
    if (!pl.ok) return false;
    *groups = pl.groups;
    *stages = pl.p.stages;
    *stage_rows = pl.p.stage_rows;
    *stage_bytes = (int)pl.p.stage_stride;
    *grid = (int)pl.grid;
    *smem_bytes = (int)pl.smem_bytes;
    return true;
}

bool matvec_stream_supported(int fmt, int64_t rows, int64_t cols, int batch) {
    if (batch != 1) return fmt != LW_F16 && batched_columns(fmt, rows, cols) >= 2;
    return make_plan(fmt, false, rows, cols, 148).ok;
}

// Several independent matrices of one format and width in a single grid (batch 1).  The CTAs are
// shared out in proportion to the rows, so all matrices finish together and the launch, activation
// and ring-fill latencies are paid once instead of once per matrix.
bool matvec_group_supported(int fmt, int64_t cols, int n_items) {
    return n_items >= 1 && n_items <= kMaxGroup && make_plan(fmt, true, 1, cols, 148).ok;
}

int launch_matvec_stream_group(int fmt, bool integer_dot, int64_t cols, int n_items, const void* const* W,
                               const int64_t* rows, const float* const* X, float* const* Y, bool overlap,
                               cudaStream_t stream) {
    if (n_items < 1 || n_items > kMaxGroup) return (int)cudaErrorInvalidValue;
    int64_t total_rows = 0;
    for (int j = 0; j < n_items; ++j) total_rows += rows[j];
    Plan pl = make_plan(fmt, integer_dot, total_rows, cols, sm_count());     // geometry for the whole group
    if (!pl.ok) return (int)cudaErrorInvalidValue;
    int* fault = device_fault_word();
    if (!fault) return (int)cudaErrorInvalidValue;
    const int rpw = pl.p.rows_per_wave;
    const int64_t budget = (int64_t)pl.grid;          // CTAs the single-matrix plan would have used
    int next_cta = 0;
    for (int j = 0; j < n_items; ++j) {
        int64_t ctas = (budget * rows[j] + total_rows - 1) / total_rows;
        if (ctas < 1) ctas = 1;
        int64_t rpc = (rows[j] + ctas - 1) / ctas;
        rpc = (rpc + rpw - 1) / rpw * rpw;
        ctas = (rows[j] + rpc - 1) / rpc;
        if (rpc > INT32_MAX) return (int)cudaErrorInvalidValue;
        pl.p.items[j].W = static_cast<const uint8_t*>(W[j]);
        pl.p.items[j].X = X[j];
        pl.p.items[j].Y = Y[j];
        pl.p.items[j].rows = rows[j];
        pl.p.items[j].first_cta = next_cta;
        pl.p.items[j].rows_per_cta = (int)rpc;
        next_cta += (int)ctas;
    }
    pl.p.n_items = n_items;
    pl.p.fault = fault;
    pl.grid = (unsigned)next_cta;
    switch (fmt) {
        case LW_F16:
            return launch_one<StreamF16>(pl, overlap, stream);
        case LW_Q8_0:
            return integer_dot ? launch_one<IdotQ80>(pl, overlap, stream) : launch_one<StreamQ80>(pl, overlap, stream);
        case LW_Q4_0:
            return integer_dot ? launch_one<IdotQ40>(pl, overlap, stream) : launch_one<StreamQ40>(pl, overlap, stream);
        case LW_Q4_K:
            return integer_dot ? launch_one<IdotQ4K>(pl, overlap, stream) : launch_one<StreamQ4K>(pl, overlap, stream);
        case LW_Q6_K:
            return launch_one<IdotQ6K>(pl, overlap, stream);
        case LW_Q5_K:
            return launch_one<IdotQ5K>(pl, overlap, stream);
        case LW_Q2_K:
            return launch_one<IdotQ2K>(pl, overlap, stream);
        case LW_Q4_1:
            return launch_one<IdotQ41>(pl, overlap, stream);
        case LW_Q5_0:
            return launch_one<IdotQ50>(pl, overlap, stream);
        case LW_Q5_1:
            return launch_one<IdotQ51>(pl, overlap, stream);
    }
    return (int)cudaErrorInvalidValue;
}

// Batch 2..16 through the batched integer-dot kernel, in passes of as many columns as fit in
// shared memory (the weights are streamed once per pass).
int launch_matvec_stream_batched(int fmt, const void* W, int64_t rows, int64_t cols, const float* X, float* Y,
                                 int batch, bool overlap, cudaStream_t stream) {
    const int nb_max = batched_columns(fmt, rows, cols);
    if (nb_max < 2) return (int)cudaErrorInvalidValue;
    int* fault = device_fault_word();
    if (!fault) return (int)cudaErrorInvalidValue;
    for (int b0 = 0; b0 < batch; b0 += nb_max) {
        const int nb = batch - b0 < nb_max ? batch - b0 : nb_max;
        Plan pl = make_plan_batched(fmt, rows, cols, nb <= 2 ? 2 : 4, sm_count());
        if (!pl.ok) return (int)cudaErrorInvalidValue;
        pl.p.W = static_cast<const uint8_t*>(W);
        pl.p.X = X + (int64_t)b0 * cols;
        pl.p.Y = Y + (int64_t)b0 * rows;
        pl.p.fault = fault;
        pl.p.batch = nb;
        int err;
        switch (fmt) {
            case LW_Q8_0: err = launch_batched_fmt<IdotQ80>(pl, nb, overlap, stream); break;
            case LW_Q4_0: err = launch_batched_fmt<IdotQ40>(pl, nb, overlap, stream); break;
            case LW_Q4_K: err = launch_batched_fmt<IdotQ4K>(pl, nb, overlap, stream); break;
            default: return (int)cudaErrorInvalidValue;
        }
        if (err != 0) return err;
    }
    return 0;
}

int launch_matvec_stream(int fmt, bool integer_dot, const void* W, int64_t rows, int64_t cols, const float* X,
                         float* Y, bool overlap, cudaStream_t stream) {
    Plan pl = make_plan(fmt, integer_dot, rows, cols, sm_count());
    if (!pl.ok) return (int)cudaErrorInvalidValue;
    int* fault = device_fault_word();
    if (!fault) return (int)cudaErrorInvalidValue;
    pl.p.W = static_cast<const uint8_t*>(W);
    pl.p.X = X;
    pl.p.Y = Y;
    pl.p.fault = fault;
    pl.p.drop_unit = take_drop_unit();
    switch (fmt) {
        case LW_F16:
            return launch_one<StreamF16>(pl, overlap, stream);
        case LW_Q8_0:
            return integer_dot ? launch_one<IdotQ80>(pl, overlap, stream) : launch_one<StreamQ80>(pl, overlap, stream);
        case LW_Q4_0:
            return integer_dot ? launch_one<IdotQ40>(pl, overlap, stream) : launch_one<StreamQ40>(pl, overlap, stream);
        case LW_Q4_K:
            return integer_dot ? launch_one<IdotQ4K>(pl, overlap, stream) : launch_one<StreamQ4K>(pl, overlap, stream);
        case LW_Q6_K:
            return launch_one<IdotQ6K>(pl, overlap, stream);
        case LW_Q5_K:
            return launch_one<IdotQ5K>(pl, overlap, stream);
        case LW_Q2_K:
            return launch_one<IdotQ2K>(pl, overlap, stream);
        case LW_Q4_1:
            return launch_one<IdotQ41>(pl, overlap, stream);
        case LW_Q5_0:
            return launch_one<IdotQ50>(pl, overlap, stream);
        case LW_Q5_1:
            return launch_one<IdotQ51>(pl, overlap, stream);
    }
    return (int)cudaErrorInvalidValue;
}

}  // namespace lw
