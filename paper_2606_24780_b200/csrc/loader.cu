// Double-buffered batch production (the paper's Algorithm 2): token windows are staged through two
// pinned host buffers and copied to two device buffers on a dedicated copy stream while the compute
// stream works on the previous batch; two kinds of events order the streams ("copy landed" before
// the consumer reads, "consumer done" before the copy stream overwrites).  Host code only: the
// caller owns every buffer (device and pinned); this file creates one stream and three events.
#include <cstring>
#include <new>
#include <vector>

#include <cstdarg>
#include <cstdio>

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
}  // namespace

struct bt_loader {
    std::vector<const int32_t*> shard;
    std::vector<int64_t> len;
    int64_t BT, pos;
    int cur, rank, world;
    bool primed, pinned;
    int buf;
    int32_t* dX[2];
    int32_t* dY[2];
    int32_t* hX[2];
    int32_t* hY[2];
    cudaStream_t compute, copy;
    cudaEvent_t h2d_done[2], consumer_done;
    bool h2d_recorded[2];
};

namespace {

// The cursor of Algorithm 2 without any CUDA: where the next window starts, then the advance.
struct Cursor {
    int cur;
    int64_t pos;
};
inline void advance_shard(Cursor& c, int n_shards, int64_t BT, int rank) {
    c.cur = (c.cur + 1) % n_shards;
    c.pos = BT * rank;
}
// Returns the (shard, position) the next prefetch reads and moves the cursor on.
inline Cursor take_window(Cursor& c, const int64_t* lens, int n_shards, int64_t BT, int rank, int world) {
    if (c.pos + BT + 1 > lens[c.cur]) advance_shard(c, n_shards, BT, rank);
    const Cursor here = c;
    c.pos += BT * world;
    if (c.pos + BT * world + 1 > lens[c.cur]) advance_shard(c, n_shards, BT, rank);
    return here;
}

bt_status issue_prefetch(bt_loader* L, int i) {
    std::vector<int64_t>& len = L->len;
    Cursor c{L->cur, L->pos};
    const Cursor w = take_window(c, len.data(), (int)len.size(), L->BT, L->rank, L->world);
    L->cur = c.cur;
    L->pos = c.pos;
    const int32_t* t = L->shard[(size_t)w.cur] + w.pos;
    const size_t bytes = (size_t)L->BT * sizeof(int32_t);
    if (L->pinned) {
        // the copy that last read these pinned buffers must have run before the host rewrites them
        if (L->h2d_recorded[i]) BT_CUDA_RET(cudaEventSynchronize(L->h2d_done[i]));
        std::memcpy(L->hX[i], t, bytes);
        std::memcpy(L->hY[i], t + 1, bytes);
        BT_CUDA_RET(cudaMemcpyAsync(L->dX[i], L->hX[i], bytes, cudaMemcpyHostToDevice, L->copy));
        BT_CUDA_RET(cudaMemcpyAsync(L->dY[i], L->hY[i], bytes, cudaMemcpyHostToDevice, L->copy));
    } else {
        // no pinned staging: the same windows, copied synchronously (pageable source)
        BT_CUDA_RET(cudaMemcpyAsync(L->dX[i], t, bytes, cudaMemcpyHostToDevice, L->copy));
        BT_CUDA_RET(cudaMemcpyAsync(L->dY[i], t + 1, bytes, cudaMemcpyHostToDevice, L->copy));
        BT_CUDA_RET(cudaStreamSynchronize(L->copy));
    }
    BT_CUDA_RET(cudaEventRecord(L->h2d_done[i], L->copy));
    L->h2d_recorded[i] = true;
    return BT_OK;
}

}  // namespace

extern "C" bt_status bt_loader_plan(const int64_t* shard_lens, int32_t n_shards, int32_t B, int32_t T, int32_t rank,
                                    int32_t world, int32_t n_batches, int32_t* out_shard, int64_t* out_pos) {
    if (!shard_lens || !out_shard || !out_pos) return lfail(BT_ERR_INVALID_ARG, "loader_plan: NULL argument");
    if (n_shards < 1 || B < 1 || T < 1 || world < 1 || rank < 0 || rank >= world || n_batches < 0)
        return lfail(BT_ERR_INVALID_ARG, "loader_plan: bad sizes");
    const int64_t BT = (int64_t)B * T;
    for (int s = 0; s < n_shards; ++s)
        if (shard_lens[s] < BT * world + 1)
            return lfail(BT_ERR_INVALID_ARG, "loader_plan: shard %d shorter than one global batch + 1", s);
    Cursor c{0, BT * rank};
    for (int i = 0; i < n_batches; ++i) {
        const Cursor w = take_window(c, shard_lens, n_shards, BT, rank, world);
        out_shard[i] = w.cur;
        out_pos[i] = w.pos;
    }
    return BT_OK;
}

extern "C" bt_status bt_loader_create(const int32_t* const* shards, const int64_t* shard_lens, int32_t n_shards,
                                      int32_t B, int32_t T, int32_t rank, int32_t world, int32_t* d_buffers,
                                      int32_t* h_pinned, void* compute_stream, bt_loader** out) {
    if (!out) return lfail(BT_ERR_INVALID_ARG, "loader: out is NULL");
    *out = nullptr;
    if (!shards || !shard_lens || !d_buffers) return lfail(BT_ERR_INVALID_ARG, "loader: NULL argument");
    if (n_shards < 1 || B < 1 || T < 1 || world < 1 || rank < 0 || rank >= world)
        return lfail(BT_ERR_INVALID_ARG, "loader: bad sizes");
    const int64_t BT = (int64_t)B * T;
    for (int s = 0; s < n_shards; ++s)
        if (!shards[s] || shard_lens[s] < BT * world + 1)
            return lfail(BT_ERR_INVALID_ARG, "loader: shard %d missing or shorter than one global batch + 1", s);
    bt_loader* L = new (std::nothrow) bt_loader();
    if (!L) return lfail(BT_ERR_OOM, "loader: host allocation failed");
    L->shard.assign(shards, shards + n_shards);
    L->len.assign(shard_lens, shard_lens + n_shards);
    L->BT = BT;
    L->pos = BT * rank;
    L->cur = 0;
    L->rank = rank;
    L->world = world;
    L->primed = false;
    L->pinned = h_pinned != nullptr;
    L->buf = 0;
    for (int i = 0; i < 2; ++i) {
        L->dX[i] = d_buffers + (2 * i) * BT;
        L->dY[i] = d_buffers + (2 * i + 1) * BT;
        L->hX[i] = h_pinned ? h_pinned + (2 * i) * BT : nullptr;
        L->hY[i] = h_pinned ? h_pinned + (2 * i + 1) * BT : nullptr;
        L->h2d_recorded[i] = false;
    }
    L->compute = static_cast<cudaStream_t>(compute_stream);
    cudaError_t e = cudaStreamCreateWithFlags(&L->copy, cudaStreamNonBlocking);
    for (int i = 0; i < 2 && e == cudaSuccess; ++i) e = cudaEventCreateWithFlags(&L->h2d_done[i], cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&L->consumer_done, cudaEventDisableTiming);
    if (e != cudaSuccess) {
        delete L;
        return lfail(BT_ERR_CUDA, "loader: stream / event creation failed: %s", cudaGetErrorString(e));
    }
    *out = L;
    return BT_OK;
}

extern "C" bt_status bt_loader_next(bt_loader* L, const int32_t** d_tokens, const int32_t** d_targets) {
    if (!L || !d_tokens || !d_targets) return lfail(BT_ERR_INVALID_ARG, "loader_next: NULL argument");
    if (!L->primed) {
        bt_status st = issue_prefetch(L, 0);
        if (st == BT_OK) st = issue_prefetch(L, 1);
        if (st != BT_OK) return st;
        L->primed = true;
        L->buf = 0;
    } else {
        // the channel handed out by the previous call is refilled once the work enqueued so far
        // (which includes its consumer) has finished
        BT_CUDA_RET(cudaEventRecord(L->consumer_done, L->compute));
        BT_CUDA_RET(cudaStreamWaitEvent(L->copy, L->consumer_done, 0));
        bt_status st = issue_prefetch(L, 1 - L->buf);
        if (st != BT_OK) return st;
    }
    BT_CUDA_RET(cudaStreamWaitEvent(L->compute, L->h2d_done[L->buf], 0));
    *d_tokens = L->dX[L->buf];
    *d_targets = L->dY[L->buf];
    L->buf = (L->buf + 1) % 2;
    return BT_OK;
}

extern "C" void bt_loader_destroy(bt_loader* L) {
    if (!L) return;
    cudaStreamSynchronize(L->copy);
    cudaEventDestroy(L->h2d_done[0]);
    cudaEventDestroy(L->h2d_done[1]);
    cudaEventDestroy(L->consumer_done);
    cudaStreamDestroy(L->copy);
    delete L;
}
