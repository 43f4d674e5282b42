// Piecewise host <-> device copies around a chain of mat-vecs, overlapped with the chain.
//
// The host forms of the chain calls take the chain's inputs as one block of host memory and return its results as
// one block.  Copying the input block before the first kernel and the result block after the last one leaves the
// copy engines idle while the kernels run and the SMs idle while the copies run.  Here the input block goes to
// the device in pieces on a copy stream of the library, in address order, and the kernels of a phase wait only
// for the piece that ends behind the activations they read; the result block leaves in pieces on a second copy
// stream as soon as no later item of the chain writes into a piece.  The caller's stream waits for both copy
// streams at the end, so that stream order (and a stream capture) sees one operation.
//
// Nothing here depends on the order of the items' X and Y inside the blocks: an item waits for the prefix of the
// input block that covers its X, and a piece of the result block leaves when it lies below the Y of every later
// item.  Activations in ascending order (the usual layout of a step) give the full overlap, any other order less.
// When an item writes into the input block, a late piece could overwrite a result, so the input is then copied
// whole before the first kernel.
#include <cuda_runtime.h>

#include <algorithm>
#include <mutex>
#include <vector>

#include "lw_internal.h"

namespace lw {

namespace {

constexpr int kMaxPieces = 32;                     // per direction, plus a first and a last piece
constexpr int kEvents = 2 * (kMaxPieces + 3) + 4;
constexpr int64_t kMinPiece = 64 << 10;

struct PipeSet {
    int device = -1;
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t ev[kEvents] = {};
    bool busy = false;
};

std::mutex g_pool_mutex;
std::vector<PipeSet*> g_pool;

PipeSet* create_set(int dev) {
    PipeSet* p = new PipeSet;
    p->device = dev;
    bool ok = cudaStreamCreateWithFlags(&p->in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&p->out, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; i < kEvents && ok; ++i) ok = cudaEventCreateWithFlags(&p->ev[i], cudaEventDisableTiming) == cudaSuccess;
    if (ok) return p;
    for (int i = 0; i < kEvents; ++i)
        if (p->ev[i]) cudaEventDestroy(p->ev[i]);
    if (p->in) cudaStreamDestroy(p->in);
    if (p->out) cudaStreamDestroy(p->out);
    delete p;
    (void)cudaGetLastError();
    return nullptr;
}

// Is `stream` part of a stream capture, and of which one?
bool capture_of(cudaStream_t stream, unsigned long long* id) {
    cudaStreamCaptureStatus status = cudaStreamCaptureStatusNone;
    *id = 0;
    if (cudaStreamGetCaptureInfo(stream, &status, id) != cudaSuccess) {
        (void)cudaGetLastError();
        return true;                    // unknown: treat as taken
    }
    return status != cudaStreamCaptureStatusNone;
}

// A set of two copy streams and events for the current device that no other call is using; nullptr when the
// driver refuses to create one.  Sets are created on first use and kept for the life of the process.  A set whose
// streams still belong to an open stream capture (an earlier call was captured and the capture has not ended)
// serves only further calls of that same capture: anything else enqueued on them would land in that graph.
PipeSet* acquire_set(cudaStream_t caller) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    unsigned long long caller_id = 0, id = 0;
    const bool caller_captures = capture_of(caller, &caller_id);
    std::lock_guard<std::mutex> lock(g_pool_mutex);
    for (PipeSet* p : g_pool)
        if (!p->busy && p->device == dev) {
            if (capture_of(p->in, &id) && !(caller_captures && id == caller_id)) continue;
            if (capture_of(p->out, &id) && !(caller_captures && id == caller_id)) continue;
            p->busy = true;
            return p;
        }
    // none free: make one -- and a spare with the very first, so that a call issued while the first set is held
    // by an open stream capture need not create streams in the middle of that capture
    const bool first = g_pool.empty();
    PipeSet* p = create_set(dev);
    if (!p) return nullptr;
    g_pool.push_back(p);
    if (first)
        if (PipeSet* spare = create_set(dev)) g_pool.push_back(spare);
    p->busy = true;
    return p;
}

void release_set(PipeSet* p) {
    if (!p) return;
    std::lock_guard<std::mutex> lock(g_pool_mutex);
    p->busy = false;
}

// [lo, hi) of the byte range [p, p + n) inside the block [base, base + size), or false when they are disjoint
bool range_in_block(const void* p, int64_t n, const void* base, int64_t size, int64_t* lo, int64_t* hi) {
    const uintptr_t a = reinterpret_cast<uintptr_t>(p), b = reinterpret_cast<uintptr_t>(base);
    if (size <= 0 || n <= 0 || a + (uintptr_t)n <= b || a >= b + (uintptr_t)size) return false;
    *lo = a > b ? (int64_t)(a - b) : 0;
    *hi = std::min<int64_t>(size, (int64_t)(a + (uintptr_t)n - b));
    return true;
}

}  // namespace

struct HostPipe::State {
    PipeSet* set = nullptr;
    int next_event = 0;
    bool in_pieces = false, out_pieces = false;
    std::vector<int64_t> need;         // per item: the prefix of the input block that has to be on the device
    std::vector<int64_t> safe;         // per item index e: the prefix of the result block no item >= e writes
    int64_t copied = 0, sent = 0;
    int64_t in_piece = 0, out_piece = 0;
    bool in_joined = true;             // has the caller's stream waited for the last input piece?
    cudaEvent_t last_in = nullptr;
};

HostPipe::HostPipe(int n_items, const lw_seq_item* items, int batch, const void* in_host, void* in_dev, int64_t in_bytes,
                   const void* out_dev, void* out_host, int64_t out_bytes, cudaStream_t stream)
    : in_host_(static_cast<const char*>(in_host)), in_dev_(static_cast<char*>(in_dev)), in_bytes_(in_bytes),
      out_dev_(static_cast<const char*>(out_dev)), out_host_(static_cast<char*>(out_host)), out_bytes_(out_bytes),
      s_(stream), st_(new State) {
    State& st = *st_;
    st.need.assign(n_items, 0);
    st.safe.assign(n_items + 1, out_bytes);
    bool writes_into_input = false;
    for (int j = 0; j < n_items; ++j) {
        int64_t lo, hi;
        if (range_in_block(items[j].X, 4 * (int64_t)batch * items[j].cols, in_dev, in_bytes, &lo, &hi)) st.need[j] = hi;
        if (range_in_block(items[j].Y, 4 * (int64_t)batch * items[j].rows, in_dev, in_bytes, &lo, &hi)) writes_into_input = true;
    }
    for (int j = n_items - 1; j >= 0; --j) {
        int64_t lo, hi;
        st.safe[j] = st.safe[j + 1];
        if (range_in_block(items[j].Y, 4 * (int64_t)batch * items[j].rows, out_dev, out_bytes, &lo, &hi))
            st.safe[j] = std::min(st.safe[j], lo);
    }
    st.in_piece = kMinPiece;
    st.out_piece = std::max(kMinPiece, (out_bytes + kMaxPieces - 1) / kMaxPieces);
    st.in_pieces = in_bytes > 2 * kMinPiece && !writes_into_input;
    st.out_pieces = out_bytes > 2 * kMinPiece;
}

HostPipe::~HostPipe() {
    release_set(st_->set);
    delete st_;
}

void HostPipe::whole_copies_only() { st_->in_pieces = st_->out_pieces = false; }

cudaEvent_t HostPipe::event() {
    State& st = *st_;
    return st.set->ev[st.next_event++ % kEvents];
}

bool HostPipe::begin() {
    State& st = *st_;
    if (st.in_pieces || st.out_pieces) {
        st.set = acquire_set(s_);
        if (!st.set) st.in_pieces = st.out_pieces = false;
    }
    if (st.set) {
        // the copy streams start where the caller's stream stands: earlier work on it may still use the blocks
        cudaEvent_t fork = event();
        if (cudaEventRecord(fork, s_) != cudaSuccess) return false;
        if (cudaStreamWaitEvent(st.set->in, fork, 0) != cudaSuccess) return false;
        if (cudaStreamWaitEvent(st.set->out, fork, 0) != cudaSuccess) return false;
    }
    if (!st.in_pieces && in_bytes_ > 0) {
        if (cudaMemcpyAsync(in_dev_, in_host_, (size_t)in_bytes_, cudaMemcpyHostToDevice, s_) != cudaSuccess) return false;
        st.copied = in_bytes_;
    }
    return true;
}

// One more piece of the input block, up to `upto`, on the input copy stream.
bool HostPipe::copy_in(int64_t upto) {
    State& st = *st_;
    if (cudaMemcpyAsync(in_dev_ + st.copied, in_host_ + st.copied, (size_t)(upto - st.copied), cudaMemcpyHostToDevice,
                        st.set->in) != cudaSuccess)
        return false;
    st.copied = upto;
    st.last_in = event();
    st.in_joined = false;
    return cudaEventRecord(st.last_in, st.set->in) == cudaSuccess;
}

bool HostPipe::before(int j, int n) {
    State& st = *st_;
    if (!st.in_pieces) return true;
    int64_t required = 0;
    for (int k = 0; k < n; ++k) required = std::max(required, st.need[j + k]);
    if (required <= st.copied) return true;        // the caller's stream has waited for that piece already
    // The first piece is what the first kernels need and no more, so that they start early; every later piece is
    // four times the one before (up to a quarter of the block).  Each piece costs the chain one wait between two
    // kernels; where the copy engine is faster than the chain consumes activations, pieces that grow keep ahead of
    // it with a handful of waits, and where it is slower a kernel waits at most for its own piece.
    int64_t upto = required;
    if (st.copied > 0) {
        upto = std::min(in_bytes_, std::max(required, st.copied + st.in_piece));
        st.in_piece = std::min(4 * st.in_piece, std::max(kMinPiece, in_bytes_ / 4));
    }
    if (!copy_in(upto)) return false;
    st.in_joined = true;
    return cudaStreamWaitEvent(s_, st.last_in, 0) == cudaSuccess;
}

// The result block up to `upto` may leave once everything enqueued on the caller's stream so far has finished.
bool HostPipe::copy_out(int64_t upto) {
    State& st = *st_;
    cudaEvent_t done = event();
    if (cudaEventRecord(done, s_) != cudaSuccess) return false;
    if (cudaStreamWaitEvent(st.set->out, done, 0) != cudaSuccess) return false;
    if (cudaMemcpyAsync(out_host_ + st.sent, out_dev_ + st.sent, (size_t)(upto - st.sent), cudaMemcpyDeviceToHost,
                        st.set->out) != cudaSuccess)
        return false;
    st.sent = upto;
    return true;
}

bool HostPipe::after(int j, int n) {
    State& st = *st_;
    if (!st.out_pieces) return true;
    const int64_t final_below = st.safe[j + n];
    if (final_below - st.sent < st.out_piece) return true;
    return copy_out(final_below);
}

bool HostPipe::end() {
    State& st = *st_;
    if (st.in_pieces) {
        if (st.copied < in_bytes_ && !copy_in(in_bytes_)) return false;    // the block is copied whole, read or not
        if (!st.in_joined && cudaStreamWaitEvent(s_, st.last_in, 0) != cudaSuccess) return false;
        st.in_joined = true;
    }
    if (st.out_pieces) {
        if (st.sent < out_bytes_ && !copy_out(out_bytes_)) return false;
    } else if (out_bytes_ > 0) {
        if (cudaMemcpyAsync(out_host_, out_dev_, (size_t)out_bytes_, cudaMemcpyDeviceToHost, s_) != cudaSuccess) return false;
    }
    if (st.set) {
        // join: the caller's stream is done when both copy streams are
        cudaEvent_t a = event(), b = event();
        if (cudaEventRecord(a, st.set->in) != cudaSuccess || cudaStreamWaitEvent(s_, a, 0) != cudaSuccess) return false;
        if (cudaEventRecord(b, st.set->out) != cudaSuccess || cudaStreamWaitEvent(s_, b, 0) != cudaSuccess) return false;
    }
    return true;
}

}  // namespace lw
