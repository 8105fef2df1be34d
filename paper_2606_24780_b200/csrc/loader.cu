// Prefetching batch production (what the paper's Algorithm 2, "Double-Buffered Batch Production",
// specifies: which token windows a rank sees, staged through pinned host memory and copied on a
// stream of their own while the compute stream works).
//
// The algorithm fixes WHAT is produced; this file chooses how:
//  * The window sequence is not walked with a cursor.  A rank takes a fixed number of windows from
//    every shard, n_s = max(1, floor((len_s - 1 - B*T*rank) / (B*T*world))), at positions
//    B*T*rank + k*B*T*world, and then moves to the next shard, cyclically; window i is found from the
//    prefix sums of n_s.  (This is the closed form of the printed cursor rules; the tests compare it
//    with a cursor that follows those rules step by step.)
//  * Batches live in a ring of n_slots slots (2 = the paper's double buffering), each with its own
//    device buffers, pinned staging buffers and two events: "copy landed" (recorded on the copy
//    stream, waited on by the compute stream before the consumer reads) and "consumer done"
//    (recorded on the compute stream when the caller RELEASES the slot, waited on by the copy stream
//    before it overwrites the slot).  A slot is therefore never rewritten before the work that reads
//    it has finished, however far the host runs ahead, and the ordering does not depend on when the
//    next batch is asked for.
//  * Ids can be checked against the vocabulary while they are copied into the staging buffer.
// Host code only: the caller owns every buffer (device and pinned); this file creates one stream and
// two events per slot.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/bt.h"
#include "common.cuh"

namespace {
bt_status lfail(bt_status st, const char* fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof(buf), fmt, ap);
    va_end(ap);
    return (bt_status)bt_internal_fail_int((int)st, buf);
}
#define BT_CUDA_RET(call)                                                                        \
    do {                                                                                         \
        cudaError_t e__ = (call);                                                                \
        if (e__ != cudaSuccess) return lfail(BT_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e__)); \
    } while (0)

// Which windows a rank reads: per shard a count, cyclically.
struct WindowPlan {
    std::vector<int64_t> first;   // first[s] = number of windows taken from shards 0 .. s-1 in one cycle
    int64_t per_cycle = 0;
    int64_t BT = 0, start = 0, stride = 0;

    bt_status init(const int64_t* lens, int n_shards, int64_t bt, int rank, int world, const char* who) {
        BT = bt;
        start = bt * rank;
        stride = bt * world;
        first.assign((size_t)n_shards + 1, 0);
        for (int s = 0; s < n_shards; ++s) {
            if (lens[s] < stride + 1) return lfail(BT_ERR_INVALID_ARG, "%s: shard %d shorter than one global batch + 1", who, s);
            int64_t n = (lens[s] - 1 - start) / stride;
            if (n < 1) n = 1;
            first[(size_t)s + 1] = first[(size_t)s] + n;
        }
        per_cycle = first[(size_t)n_shards];
        return BT_OK;
    }
    void window(int64_t i, int* shard, int64_t* pos) const {
        const int64_t j = i % per_cycle;
        size_t lo = 0, hi = first.size() - 1;          // first[lo] <= j < first[hi]
        while (hi - lo > 1) {
            const size_t mid = (lo + hi) / 2;
            if (first[mid] <= j) lo = mid; else hi = mid;
        }
        *shard = (int)lo;
        *pos = start + (j - first[lo]) * stride;
    }
};

enum SlotState { kFree = 0, kFilled = 1, kLent = 2 };
constexpr int kMaxSlots = 8;
}  // namespace

struct bt_loader {
    std::vector<const int32_t*> shard;
    WindowPlan plan;
    int64_t next_window = 0;     // index of the next window to stage
    int n_slots = 2, vocab = 0;
    bool pinned = false, primed = false;
    bt_status failed = BT_OK;    // sticky: a staged window held an invalid id, or a CUDA call failed
    int head = 0;                // slot the next bt_loader_next hands out (slots are used in ring order)
    int state[kMaxSlots];
    int32_t *dX[kMaxSlots], *dY[kMaxSlots], *hX[kMaxSlots], *hY[kMaxSlots];
    cudaStream_t compute = nullptr, copy = nullptr;
    cudaEvent_t landed[kMaxSlots], consumed[kMaxSlots];
    bool landed_recorded[kMaxSlots], consumed_recorded[kMaxSlots];
};

namespace {

// Stages the next window into slot i and enqueues its copy.
bt_status fill_slot(bt_loader* L, int i) {
    int s;
    int64_t pos;
    L->plan.window(L->next_window, &s, &pos);
    const int32_t* t = L->shard[(size_t)s] + pos;
    const int64_t BT = L->plan.BT;
    if (L->vocab > 0) {
        const int64_t bad = bt_first_invalid_id(t, BT + 1, L->vocab);   // tokens and targets: BT + 1 ids
        if (bad >= 0)
            return lfail(BT_ERR_INVALID_ARG, "loader: id %d outside [0, %d) at position %lld of shard %d", t[bad], L->vocab,
                         (long long)(pos + bad), s);
    }
    const size_t bytes = (size_t)BT * sizeof(int32_t);
    // the copy stream may overwrite the slot only after the work that read it
    if (L->consumed_recorded[i]) BT_CUDA_RET(cudaStreamWaitEvent(L->copy, L->consumed[i], 0));
    if (L->pinned) {
        // and the host may rewrite the staging buffers only after the copy that last read them
        if (L->landed_recorded[i]) BT_CUDA_RET(cudaEventSynchronize(L->landed[i]));
        std::memcpy(L->hX[i], t, bytes);
        std::memcpy(L->hY[i], t + 1, bytes);
        BT_CUDA_RET(cudaMemcpyAsync(L->dX[i], L->hX[i], bytes, cudaMemcpyHostToDevice, L->copy));
        BT_CUDA_RET(cudaMemcpyAsync(L->dY[i], L->hY[i], bytes, cudaMemcpyHostToDevice, L->copy));
    } else {
        // no staging buffers: the same windows straight from the (pageable) shards, synchronously
        BT_CUDA_RET(cudaMemcpyAsync(L->dX[i], t, bytes, cudaMemcpyHostToDevice, L->copy));
        BT_CUDA_RET(cudaMemcpyAsync(L->dY[i], t + 1, bytes, cudaMemcpyHostToDevice, L->copy));
        BT_CUDA_RET(cudaStreamSynchronize(L->copy));
    }
    BT_CUDA_RET(cudaEventRecord(L->landed[i], L->copy));
    L->landed_recorded[i] = true;
    L->state[i] = kFilled;
    L->next_window += 1;
    return BT_OK;
}

}  // namespace

extern "C" bt_status bt_loader_plan(const int64_t* shard_lens, int32_t n_shards, int32_t B, int32_t T, int32_t rank,
                                    int32_t world, int32_t n_batches, int32_t* out_shard, int64_t* out_pos) {
    if (!shard_lens || !out_shard || !out_pos) return lfail(BT_ERR_INVALID_ARG, "loader_plan: NULL argument");
    if (n_shards < 1 || B < 1 || T < 1 || world < 1 || rank < 0 || rank >= world || n_batches < 0)
        return lfail(BT_ERR_INVALID_ARG, "loader_plan: bad sizes");
    WindowPlan plan;
    bt_status st = plan.init(shard_lens, n_shards, (int64_t)B * T, rank, world, "loader_plan");
    if (st != BT_OK) return st;
    for (int i = 0; i < n_batches; ++i) {
        int s;
        plan.window(i, &s, &out_pos[i]);
        out_shard[i] = s;
    }
    return BT_OK;
}

extern "C" bt_status bt_loader_create(const int32_t* const* shards, const int64_t* shard_lens, int32_t n_shards,
                                      int32_t B, int32_t T, int32_t rank, int32_t world, int32_t vocab_size,
                                      int32_t n_slots, int32_t* d_buffers, int32_t* h_pinned, void* compute_stream,
                                      bt_loader** out) {
    if (!out) return lfail(BT_ERR_INVALID_ARG, "loader: out is NULL");
    *out = nullptr;
    if (!shards || !shard_lens || !d_buffers) return lfail(BT_ERR_INVALID_ARG, "loader: NULL argument");
    if (n_shards < 1 || B < 1 || T < 1 || world < 1 || rank < 0 || rank >= world || vocab_size < 0)
        return lfail(BT_ERR_INVALID_ARG, "loader: bad sizes");
    if (n_slots < 2 || n_slots > kMaxSlots) return lfail(BT_ERR_INVALID_ARG, "loader: n_slots %d not in [2, %d]", n_slots, kMaxSlots);
    for (int s = 0; s < n_shards; ++s)
        if (!shards[s]) return lfail(BT_ERR_INVALID_ARG, "loader: shard %d is NULL", s);
    bt_loader* L = new (std::nothrow) bt_loader();
    if (!L) return lfail(BT_ERR_OOM, "loader: host allocation failed");
    const int64_t BT = (int64_t)B * T;
    bt_status st = L->plan.init(shard_lens, n_shards, BT, rank, world, "loader");
    if (st != BT_OK) {
        delete L;
        return st;
    }
    L->shard.assign(shards, shards + n_shards);
    L->n_slots = n_slots;
    L->vocab = vocab_size;
    L->pinned = h_pinned != nullptr;
    for (int i = 0; i < n_slots; ++i) {
        L->dX[i] = d_buffers + (2 * i) * BT;
        L->dY[i] = d_buffers + (2 * i + 1) * BT;
        L->hX[i] = h_pinned ? h_pinned + (2 * i) * BT : nullptr;
        L->hY[i] = h_pinned ? h_pinned + (2 * i + 1) * BT : nullptr;
        L->state[i] = kFree;
        L->landed_recorded[i] = L->consumed_recorded[i] = false;
        L->landed[i] = L->consumed[i] = nullptr;
    }
    L->compute = static_cast<cudaStream_t>(compute_stream);
    cudaError_t e = cudaStreamCreateWithFlags(&L->copy, cudaStreamNonBlocking);
    for (int i = 0; i < n_slots && e == cudaSuccess; ++i) {
        e = cudaEventCreateWithFlags(&L->landed[i], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&L->consumed[i], cudaEventDisableTiming);
    }
    if (e != cudaSuccess) {
        bt_loader_destroy(L);
        return lfail(BT_ERR_CUDA, "loader: stream / event creation failed: %s", cudaGetErrorString(e));
    }
    *out = L;
    return BT_OK;
}

extern "C" bt_status bt_loader_next(bt_loader* L, const int32_t** d_tokens, const int32_t** d_targets, int32_t* slot) {
    if (!L || !d_tokens || !d_targets || !slot) return lfail(BT_ERR_INVALID_ARG, "loader_next: NULL argument");
    if (L->failed != BT_OK) return lfail(L->failed, "loader: an earlier call failed; the loader is unusable");
    if (!L->primed) {
        for (int i = 0; i < L->n_slots; ++i) {
            bt_status st = fill_slot(L, i);
            if (st != BT_OK) return L->failed = st;
        }
        L->primed = true;
    }
    const int i = L->head;
    if (L->state[i] != kFilled)
        return lfail(BT_ERR_INVALID_ARG, "loader_next: all %d slots are lent out; release one with bt_loader_release first",
                     L->n_slots);
    BT_CUDA_RET(cudaStreamWaitEvent(L->compute, L->landed[i], 0));
    L->state[i] = kLent;
    L->head = (i + 1) % L->n_slots;
    *d_tokens = L->dX[i];
    *d_targets = L->dY[i];
    *slot = i;
    return BT_OK;
}

extern "C" bt_status bt_loader_release(bt_loader* L, int32_t slot) {
    if (!L) return lfail(BT_ERR_INVALID_ARG, "loader_release: loader is NULL");
    if (slot < 0 || slot >= L->n_slots || L->state[slot] != kLent)
        return lfail(BT_ERR_INVALID_ARG, "loader_release: slot %d is not lent out", slot);
    if (L->failed != BT_OK) return lfail(L->failed, "loader: an earlier call failed; the loader is unusable");
    // everything enqueued on the compute stream up to here -- which by contract includes every
    // reader of this slot -- precedes the copy that refills it
    BT_CUDA_RET(cudaEventRecord(L->consumed[slot], L->compute));
    L->consumed_recorded[slot] = true;
    L->state[slot] = kFree;
    bt_status st = fill_slot(L, slot);
    if (st != BT_OK) L->failed = st;
    return st;
}

extern "C" void bt_loader_destroy(bt_loader* L) {
    if (!L) return;
    if (L->copy) cudaStreamSynchronize(L->copy);
    for (int i = 0; i < L->n_slots; ++i) {
        if (L->landed[i]) cudaEventDestroy(L->landed[i]);
        if (L->consumed[i]) cudaEventDestroy(L->consumed[i]);
    }
    if (L->copy) cudaStreamDestroy(L->copy);
    delete L;
}
