// Memory-bound kernels of the training step: TF32 split, embedding gather and its
// deterministic scatter-add backward, GELU, column sums (bias gradients), gradient norm,
// multi-tensor AdamW, split-K reduction, parameter initialisation.
//
// All of them stream their operands once with 128-bit accesses; reductions use warp
// shuffles and fixed summation orders (no floating-point atomics anywhere).
#include <mutex>

#include "../../include/bt.h"
#include "common.cuh"

static inline bt_status bt_internal_fail(bt_status st, const char* msg) {
    return (bt_status)bt_internal_fail_int((int)st, msg);
}

namespace bt {

std::atomic<long long> g_launches{0};

static inline int grid_for(int64_t work, int block, int cap) {
    int64_t g = (work + block - 1) / block;
    if (g < 1) g = 1;
    if (g > cap) g = cap;
    return (int)g;
}
// Grid-stride kernels: enough CTAs to fill 148 SMs several times over.
constexpr int kStreamGridCap = 148 * 16;

// ------------------------------------------------------------------ split

__global__ void __launch_bounds__(256) split_kernel(const float* __restrict__ x, float* __restrict__ hi,
                                                    float* __restrict__ lo, int64_t n4) {
    pdl_wait();
    pdl_trigger();
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
        float4 v = ld4(x, i), h, l;
        split_tf32(v, h, l);
        reinterpret_cast<float4*>(hi)[i] = h;
        reinterpret_cast<float4*>(lo)[i] = l;
    }
}

cudaError_t launch_split(const float* x, float* hi, float* lo, int64_t n, cudaStream_t s) {
    int64_t n4 = n / 4;
    BT_KERNEL_LAUNCH((split_kernel), grid_for(n4, 256, kStreamGridCap), 256, 0, s, x, hi, lo, n4);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

// Weight matrices -> split planes in both orientations.  A CTA takes 64x64 tiles: the tile is read
// once with 128-bit loads, its hi/lo planes are written in place, the values pass through shared
// memory and the transposed tile's hi/lo planes are written with 128-bit stores too.  The forward
// GEMMs read the transposed copy (so that the weight is the tensor core's "N-contiguous" operand,
// whose TMA boxes are 128-byte rows), the backward GEMMs the original orientation.
__global__ void __launch_bounds__(256) split_matrices_kernel(const float* __restrict__ params, float* __restrict__ w_hi,
                                                             float* __restrict__ wt_hi, int64_t plane,
                                                             const MatDesc* __restrict__ descs, int nmats,
                                                             int ntiles) {
    pdl_wait();
    pdl_trigger();
    __shared__ MatDesc sd[kMaxSplitMats];
    __shared__ float tile[64][65];
    for (int i = threadIdx.x; i < nmats; i += blockDim.x) sd[i] = descs[i];
    __syncthreads();
    for (int t = blockIdx.x; t < ntiles; t += gridDim.x) {
        int mi = 0;
        while (mi + 1 < nmats && sd[mi + 1].tile0 <= t) ++mi;   // few matrices: a linear scan
        const MatDesc d = sd[mi];
        const int lt = t - d.tile0, r0 = (lt / d.tiles_c) * 64, c0 = (lt % d.tiles_c) * 64;
        const float* src = params + d.off;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int idx = threadIdx.x + 256 * k, r = idx >> 4, c = (idx & 15) * 4;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (r0 + r < d.rows && c0 + c < d.cols) {
                const int64_t i4 = ((int64_t)(r0 + r) * d.cols + c0 + c) >> 2;
                v = ld4(src, i4);
                float4 h, l;
                split_tf32(v, h, l);
                reinterpret_cast<float4*>(w_hi + d.off)[i4] = h;
                reinterpret_cast<float4*>(w_hi + plane + d.off)[i4] = l;
            }
            tile[r][c] = v.x; tile[r][c + 1] = v.y; tile[r][c + 2] = v.z; tile[r][c + 3] = v.w;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int idx = threadIdx.x + 256 * k, c = idx >> 4, r = (idx & 15) * 4;
            if (c0 + c < d.cols && r0 + r < d.rows) {
                const float4 v = make_float4(tile[r][c], tile[r + 1][c], tile[r + 2][c], tile[r + 3][c]);
                float4 h, l;
                split_tf32(v, h, l);
                const int64_t i4 = ((int64_t)(c0 + c) * d.rows + r0 + r) >> 2;
                reinterpret_cast<float4*>(wt_hi + d.off)[i4] = h;
                reinterpret_cast<float4*>(wt_hi + plane + d.off)[i4] = l;
            }
        }
        __syncthreads();
    }
}

cudaError_t launch_split_matrices(const float* params, float* w_hi, float* wt_hi, int64_t plane,
                                  const MatDesc* descs_dev, int nmats, int ntiles, cudaStream_t s) {
    if (nmats < 1 || nmats > kMaxSplitMats) return cudaErrorInvalidValue;
    const int grid = ntiles < 148 * 8 ? ntiles : 148 * 8;
    BT_KERNEL_LAUNCH((split_matrices_kernel), grid, 256, 0, s, params, w_hi, wt_hi, plane, descs_dev, nmats, ntiles);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

// ------------------------------------------------------------------ embedding forward

// An id outside [0, V) is never used as an index: it is treated as id 0 and position + 1 is
// recorded in *bad (first writer wins; bad may be null).
__device__ __forceinline__ int checked_id(int id, int V, int64_t position, int* bad) {
    if ((unsigned)id < (unsigned)V) return id;
    if (bad) atomicCAS(bad, 0, (int)position + 1);
    return 0;
}

// One thread per float4 of the output: x[n,:] = wte[tok[n],:] + wpe[n mod T,:].
__global__ void __launch_bounds__(256) embedding_fwd_kernel(const int32_t* __restrict__ tok,
                                                            const float* __restrict__ wte,
                                                            const float* __restrict__ wpe, int64_t N, int T, int C4,
                                                            int V, float* __restrict__ x, int* bad) {
    pdl_wait();
    pdl_trigger();
    int64_t total = N * C4;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        int64_t n = i / C4;
        int c = (int)(i - n * C4);
        const int id = checked_id(tok[n], V, n, bad);
        float4 e = ld4(wte, (int64_t)id * C4 + c);
        float4 p = ld4(wpe, (n % T) * C4 + c);
        float4 r;
        r.x = __fadd_rn(e.x, p.x);
        r.y = __fadd_rn(e.y, p.y);
        r.z = __fadd_rn(e.z, p.z);
        r.w = __fadd_rn(e.w, p.w);
        reinterpret_cast<float4*>(x)[i] = r;
    }
}

cudaError_t launch_embedding_fwd(const int32_t* tok, const float* wte, const float* wpe, int64_t N, int T, int C,
                                 int V, float* x, int* bad, cudaStream_t s) {
    BT_KERNEL_LAUNCH((embedding_fwd_kernel), grid_for(N * (C / 4), 256, kStreamGridCap), 256, 0, s, tok, wte, wpe, N, T,
                     C / 4, V, x, bad);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

// ------------------------------------------------------------------ embedding backward
//
// dwte[id,:] += sum over the positions n with tok[n] == id of dx[n,:], in ascending n, without
// atomics and with the work spread evenly although the ids are heavy-tailed (under a Zipf law one id
// owns a seventh of all positions).  Two stages over chunks of kEmbChunk (128) consecutive positions:
//   1. one CTA per chunk groups the chunk's positions by id (all in shared memory), reads every row
//      of dx exactly once, eight rows in flight, and writes one partial row per (chunk, id) group to
//      `partial` at the slot of the group's first position; a byte table [Vp][chunks] records that
//      position (offset in the chunk + 1, 0 = the id does not occur in the chunk);
//   2. one CTA per eight ids reads their table rows; for an id that occurs it adds the partial rows
//      of its chunks in ascending chunk order and then the sum to dwte[id,:].
// Every CTA of stage 1 moves the same number of bytes; the longest serial chain of stage 2 is one
// row per chunk.  The order of every addition is fixed by the positions alone.
constexpr int kEmbChunk = 128;

__global__ void __launch_bounds__(256) embedding_bwd_group_kernel(const int32_t* __restrict__ tok,
                                                                  const float* __restrict__ dx, int N, int C4, int V,
                                                                  int n_chunks, float* __restrict__ partial,
                                                                  uint8_t* __restrict__ table) {
    pdl_wait();
    pdl_trigger();
    __shared__ int ids[kEmbChunk];      // id of position p of the chunk (-1 beyond N)
    __shared__ int lead[kEmbChunk];     // first position of the chunk with the same id
    __shared__ int order[kEmbChunk];    // positions sorted by (lead, position): the groups, concatenated
    __shared__ int ends[kEmbChunk];     // 1 where a group ends in `order`
    const int chunk = blockIdx.x, base = chunk * kEmbChunk, p = threadIdx.x;
    const int nvalid = min(kEmbChunk, N - base);
    if (p < kEmbChunk) ids[p] = p < nvalid ? checked_id(tok[base + p], V, base + p, nullptr) : -1;
    __syncthreads();
    if (p < kEmbChunk) {
        int g = p;
        const int id = ids[p];
        for (int j = 0; j < p; ++j)
            if (ids[j] == id) { g = j; break; }
        lead[p] = g;
        if (g == p && p < nvalid) table[(int64_t)id * n_chunks + chunk] = (uint8_t)(p + 1);
    }
    __syncthreads();
    if (p < nvalid) {
        const int g = lead[p];
        int slot = 0;
        for (int q = 0; q < nvalid; ++q) {
            const int gq = lead[q];
            slot += (gq < g || (gq == g && q < p)) ? 1 : 0;
        }
        order[slot] = p;
    }
    __syncthreads();
    if (p < nvalid) ends[p] = (p == nvalid - 1 || lead[order[p + 1]] != lead[order[p]]) ? 1 : 0;
    __syncthreads();
    for (int c = threadIdx.x; c < C4; c += 256) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int i0 = 0; i0 < nvalid; i0 += 8) {
            float4 r[8];
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (i0 + q < nvalid) r[q] = ld4(dx, (int64_t)(base + order[i0 + q]) * C4 + c);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                if (i0 + q < nvalid) {
                    acc = add4(acc, r[q]);
                    if (ends[i0 + q]) {
                        reinterpret_cast<float4*>(partial)[(int64_t)(base + lead[order[i0 + q]]) * C4 + c] = acc;
                        acc = make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
            }
        }
    }
}

constexpr int kEmbIdsPerCta = 8;
__global__ void __launch_bounds__(256) embedding_bwd_combine_kernel(const uint8_t* __restrict__ table, int n_chunks,
                                                                    const float* __restrict__ partial, int C4, int Vp,
                                                                    float* __restrict__ dwte) {
    pdl_wait();
    pdl_trigger();
    __shared__ int present[kEmbIdsPerCta];
    __shared__ int list[256];
    __shared__ int wcount[8];
    // the CTA's ids are blockIdx.x, blockIdx.x + gridDim.x, ...: frequent ids are neighbours under a
    // rank-ordered vocabulary (id = frequency rank), and every one of them has a partial row in
    // every chunk, so consecutive ids must not share a CTA
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x < kEmbIdsPerCta) present[threadIdx.x] = 0;
    __syncthreads();
    int any[kEmbIdsPerCta];      // all table reads are issued before any of them is looked at
#pragma unroll
    for (int w = 0; w < kEmbIdsPerCta; ++w) {
        const int id = blockIdx.x + w * gridDim.x;
        any[w] = 0;
        if (id < Vp)
            for (int k = threadIdx.x; k < n_chunks; k += 256) any[w] |= table[(int64_t)id * n_chunks + k];
    }
#pragma unroll
    for (int w = 0; w < kEmbIdsPerCta; ++w)
        if (any[w]) present[w] = 1;
    __syncthreads();
#pragma unroll
    for (int w = 0; w < kEmbIdsPerCta; ++w) {
        if (!present[w]) continue;   // uniform over the CTA
        const int id = blockIdx.x + w * gridDim.x;
        for (int c0 = 0; c0 < C4; c0 += 256) {
            const int c = c0 + threadIdx.x;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int k0 = 0; k0 < n_chunks; k0 += 256) {
                const int k = k0 + threadIdx.x;
                // up to 256 chunks the byte read during the presence test is this thread's entry
                const int b = n_chunks <= 256 ? any[w] : (k < n_chunks ? table[(int64_t)id * n_chunks + k] : 0);
                // ordered list of the round's partial rows: chunk order = thread order
                const unsigned bal = __ballot_sync(0xffffffffu, b != 0);
                if (lane == 0) wcount[warp] = __popc(bal);
                __syncthreads();
                int off = __popc(bal & ((1u << lane) - 1u)), total = 0;
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    if (q < warp) off += wcount[q];
                    total += wcount[q];
                }
                if (b) list[off] = k * kEmbChunk + (b - 1);
                __syncthreads();
                if (c < C4) {
                    int i = 0;
                    for (; i + 8 <= total; i += 8) {
                        float4 r[8];
#pragma unroll
                        for (int q = 0; q < 8; ++q) r[q] = ld4(partial, (int64_t)list[i + q] * C4 + c);
#pragma unroll
                        for (int q = 0; q < 8; ++q) acc = add4(acc, r[q]);
                    }
                    for (; i < total; ++i) acc = add4(acc, ld4(partial, (int64_t)list[i] * C4 + c));
                }
                __syncthreads();
            }
            if (c < C4) {
                float4* dst = reinterpret_cast<float4*>(dwte) + (int64_t)id * C4 + c;
                *dst = add4(*dst, acc);
            }
        }
    }
}

// dwpe[t,:] = sum over sequences b (ascending) of dx[b*T + t,:].
__global__ void __launch_bounds__(256) embedding_bwd_wpe_kernel(const float* __restrict__ dx, int B, int T, int C4,
                                                                float* __restrict__ dwpe) {
    pdl_wait();
    pdl_trigger();
    int64_t total = (int64_t)T * C4;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int b = 0; b < B; ++b) acc = add4(acc, ld4(dx, (int64_t)b * total + i));
        reinterpret_cast<float4*>(dwpe)[i] = acc;
    }
}

size_t embedding_bwd_partial_bytes(int64_t N, int C) { return ((size_t)N * C * sizeof(float) + 255) & ~(size_t)255; }
size_t embedding_bwd_scratch_bytes(int64_t N, int C, int Vp) {
    const int64_t chunks = (N + kEmbChunk - 1) / kEmbChunk;
    return embedding_bwd_partial_bytes(N, C) + (size_t)Vp * (size_t)chunks;
}

cudaError_t launch_embedding_bwd(const int32_t* tok, const float* dx, int64_t N, int T, int C, int V, int Vp,
                                 float* dwte, float* dwpe, float* partial, uint8_t* table, cudaStream_t s) {
    const int chunks = (int)((N + kEmbChunk - 1) / kEmbChunk);
    cudaError_t e = cudaMemsetAsync(table, 0, (size_t)Vp * chunks, s);
    if (e != cudaSuccess) return e;
    BT_KERNEL_LAUNCH((embedding_bwd_group_kernel), chunks, 256, 0, s, tok, dx, (int)N, C / 4, V, chunks, partial, table);
    BT_COUNT_LAUNCH();
    BT_KERNEL_LAUNCH((embedding_bwd_combine_kernel), (Vp + kEmbIdsPerCta - 1) / kEmbIdsPerCta, 256, 0, s,
                     (const uint8_t*)table, chunks, (const float*)partial, C / 4, Vp, dwte);
    BT_COUNT_LAUNCH();
    BT_KERNEL_LAUNCH((embedding_bwd_wpe_kernel), grid_for((int64_t)T * (C / 4), 256, kStreamGridCap), 256, 0, s,
        dx, (int)(N / T), T, C / 4, dwpe);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

// ------------------------------------------------------------------ GELU

__global__ void __launch_bounds__(256) gelu_fwd_kernel(const float* __restrict__ x, int64_t n4, int tanh_form,
                                                       float* y, float* y_hi, float* y_lo) {
    pdl_wait();
    pdl_trigger();
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
        float4 v = ld4(x, i), r;
        r.x = gelu_f(v.x, tanh_form);
        r.y = gelu_f(v.y, tanh_form);
        r.z = gelu_f(v.z, tanh_form);
        r.w = gelu_f(v.w, tanh_form);
        store_raw_split(r, y, y_hi, y_lo, i);
    }
}

__global__ void __launch_bounds__(256) gelu_bwd_kernel(const float* __restrict__ x, const float* __restrict__ dy,
                                                       int64_t n4, int tanh_form, float* dx, float* dx_hi,
                                                       float* dx_lo) {
    pdl_wait();
    pdl_trigger();
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
        float4 v = ld4(x, i), d = ld4(dy, i), r;
        r.x = d.x * gelu_grad_f(v.x, tanh_form);
        r.y = d.y * gelu_grad_f(v.y, tanh_form);
        r.z = d.z * gelu_grad_f(v.z, tanh_form);
        r.w = d.w * gelu_grad_f(v.w, tanh_form);
        store_raw_split(r, dx, dx_hi, dx_lo, i);
    }
}

cudaError_t launch_gelu_fwd(const float* x, int64_t n, int tanh_form, float* y, float* y_hi, float* y_lo,
                            cudaStream_t s) {
    BT_KERNEL_LAUNCH((gelu_fwd_kernel), grid_for(n / 4, 256, kStreamGridCap), 256, 0, s, x, n / 4, tanh_form, y, y_hi, y_lo);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}
cudaError_t launch_gelu_bwd(const float* x, const float* dy, int64_t n, int tanh_form, float* dx, float* dx_hi,
                            float* dx_lo, cudaStream_t s) {
    BT_KERNEL_LAUNCH((gelu_bwd_kernel), grid_for(n / 4, 256, kStreamGridCap), 256, 0, s, x, dy, n / 4, tanh_form, dx, dx_hi, dx_lo);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

// ------------------------------------------------------------------ column sums

// Stage 1: CTA (cb, st) sums rows of strip st for the 128 columns of block cb; warp w takes
// rows w, w+8, ... of the strip, lanes hold one float4 column group; warps are combined in
// warp order.  Stage 2 adds the strips in strip order.
static inline int colsum_strips(int64_t N, int C) {
    int cblocks = (C + 127) / 128;
    int64_t strips = (4 * 148) / cblocks;  // 4 resident CTAs per SM: one wave
    int64_t max_strips = (N + 63) / 64;
    if (strips > max_strips) strips = max_strips;
    if (strips < 1) strips = 1;
    return (int)strips;
}
size_t colsum_scratch_floats(int64_t N, int C) { return (size_t)colsum_strips(N, C) * C; }

__global__ void __launch_bounds__(256) colsum_stage1_kernel(const float* __restrict__ x,
                                                            const float* __restrict__ x_lo, int64_t N, int C4,
                                                            int strips, float* __restrict__ partial) {
    pdl_wait();
    pdl_trigger();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int c = blockIdx.x * 32 + lane;
    const int st = blockIdx.y;
    const int64_t rows_per = (N + strips - 1) / strips;
    const int64_t r0 = st * rows_per, r1 = (r0 + rows_per < N) ? r0 + rows_per : N;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (c < C4) {
        int64_t r = r0 + warp;
        for (; r + 24 < r1; r += 32) {  // four rows in flight per lane
            float4 v0 = ld4(x, r * C4 + c), v1 = ld4(x, (r + 8) * C4 + c), v2 = ld4(x, (r + 16) * C4 + c),
                   v3 = ld4(x, (r + 24) * C4 + c);
            if (x_lo) {
                v0 = add4(v0, ld4(x_lo, r * C4 + c));
                v1 = add4(v1, ld4(x_lo, (r + 8) * C4 + c));
                v2 = add4(v2, ld4(x_lo, (r + 16) * C4 + c));
                v3 = add4(v3, ld4(x_lo, (r + 24) * C4 + c));
            }
            acc = add4(add4(add4(add4(acc, v0), v1), v2), v3);
        }
        for (; r < r1; r += 8) {
            float4 v = ld4(x, r * C4 + c);
            if (x_lo) v = add4(v, ld4(x_lo, r * C4 + c));
            acc = add4(acc, v);
        }
    }
    __shared__ float4 sm[8][32];
    sm[warp][lane] = acc;
    __syncthreads();
    if (warp == 0 && c < C4) {
        float4 t = sm[0][lane];
#pragma unroll
        for (int w = 1; w < 8; ++w) t = add4(t, sm[w][lane]);
        reinterpret_cast<float4*>(partial)[(int64_t)st * C4 + c] = t;
    }
}

// Stage 2: lane = float4 column, warp w adds strips w, w+8, ... (four loads in flight), the eight
// warp sums are combined in warp order: a fixed summation order.
__global__ void __launch_bounds__(256) colsum_stage2_kernel(const float* __restrict__ partial, int strips, int C4,
                                                            float* __restrict__ out) {
    pdl_wait();
    pdl_trigger();
    __shared__ float4 sm[8][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int c = blockIdx.x * 32 + lane;
    float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
    if (c < C4) {
        int s = warp;
        for (; s + 120 < strips; s += 128) {   // sixteen rows in flight per lane, added in the same (ascending) order
            float4 a[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) a[j] = ld4(partial, (int64_t)(s + 8 * j) * C4 + c);
#pragma unroll
            for (int j = 0; j < 16; ++j) t = add4(t, a[j]);
        }
        for (; s + 24 < strips; s += 32) {
            float4 a0 = ld4(partial, (int64_t)s * C4 + c), a1 = ld4(partial, (int64_t)(s + 8) * C4 + c);
            float4 a2 = ld4(partial, (int64_t)(s + 16) * C4 + c), a3 = ld4(partial, (int64_t)(s + 24) * C4 + c);
            t = add4(add4(add4(add4(t, a0), a1), a2), a3);
        }
        for (; s < strips; s += 8) t = add4(t, ld4(partial, (int64_t)s * C4 + c));
    }
    sm[warp][lane] = t;
    __syncthreads();
    if (warp == 0 && c < C4) {
        float4 r = sm[0][lane];
#pragma unroll
        for (int w = 1; w < 8; ++w) r = add4(r, sm[w][lane]);
        reinterpret_cast<float4*>(out)[c] = r;
    }
}

// GELU backward with the column sums of its own output (the bias gradient of the layer that
// produced x): the strip layout of stage 1 above, so each lane keeps one float4 column and the
// sums cost no extra pass over dx.
__global__ void __launch_bounds__(256) gelu_bwd_colsum_kernel(const float* __restrict__ x,
                                                              const float* __restrict__ dy, int64_t N, int C4,
                                                              int strips, int tanh_form, float* dx, float* dx_hi,
                                                              float* dx_lo, float* __restrict__ partial) {
    pdl_wait();
    pdl_trigger();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int c = blockIdx.x * 32 + lane;
    const int st = blockIdx.y;
    const int64_t rows_per = (N + strips - 1) / strips;
    const int64_t r0 = st * rows_per, r1 = (r0 + rows_per < N) ? r0 + rows_per : N;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    auto one = [&](float4 v, float4 d, int64_t i) {
        float4 r;
        r.x = d.x * gelu_grad_f(v.x, tanh_form);
        r.y = d.y * gelu_grad_f(v.y, tanh_form);
        r.z = d.z * gelu_grad_f(v.z, tanh_form);
        r.w = d.w * gelu_grad_f(v.w, tanh_form);
        store_raw_split(r, dx, dx_hi, dx_lo, i);
        acc = add4(acc, r);
    };
    if (c < C4) {
        int64_t r = r0 + warp;
        for (; r + 24 < r1; r += 32) {  // four rows in flight per lane
            const int64_t i0 = r * C4 + c, i1 = (r + 8) * C4 + c, i2 = (r + 16) * C4 + c, i3 = (r + 24) * C4 + c;
            float4 v0 = ld4(x, i0), v1 = ld4(x, i1), v2 = ld4(x, i2), v3 = ld4(x, i3);
            float4 d0 = ld4(dy, i0), d1 = ld4(dy, i1), d2 = ld4(dy, i2), d3 = ld4(dy, i3);
            one(v0, d0, i0);
            one(v1, d1, i1);
            one(v2, d2, i2);
            one(v3, d3, i3);
        }
        for (; r < r1; r += 8) one(ld4(x, r * C4 + c), ld4(dy, r * C4 + c), r * C4 + c);
    }
    __shared__ float4 sm[8][32];
    sm[warp][lane] = acc;
    __syncthreads();
    if (warp == 0 && c < C4) {
        float4 t = sm[0][lane];
#pragma unroll
        for (int w = 1; w < 8; ++w) t = add4(t, sm[w][lane]);
        reinterpret_cast<float4*>(partial)[(int64_t)st * C4 + c] = t;
    }
}

cudaError_t launch_gelu_bwd_colsum(const float* x, const float* dy, int64_t N, int C, int tanh_form, float* dx,
                                   float* dx_hi, float* dx_lo, float* colsum, float* scratch, cudaStream_t s) {
    // One wave: no more strips than the CTAs that are resident at once (the kernel's register
    // count decides that, so it is asked for), and never more than the scratch was sized for.
    static int resident = 0;
    if (resident == 0) {
        int per_sm = 0, sms = 0, dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, gelu_bwd_colsum_kernel, 256, 0);
        resident = (per_sm > 0 && sms > 0) ? per_sm * sms : 296;
    }
    int C4 = C / 4, strips = colsum_strips(N, C);
    const int cblocks = (C4 + 31) / 32;
    if (strips * cblocks > resident && resident / cblocks >= 1) strips = resident / cblocks;
    dim3 grid(cblocks, strips);
    BT_KERNEL_LAUNCH((gelu_bwd_colsum_kernel), grid, 256, 0, s, x, dy, N, C4, strips, tanh_form, dx, dx_hi, dx_lo, scratch);
    BT_COUNT_LAUNCH();
    BT_KERNEL_LAUNCH((colsum_stage2_kernel), (C4 + 31) / 32, 256, 0, s, scratch, strips, C4, colsum);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

cudaError_t launch_colsum(const float* x, const float* x_lo, int64_t N, int C, float* out, float* scratch,
                          cudaStream_t s) {
    int C4 = C / 4, strips = colsum_strips(N, C);
    dim3 grid((C4 + 31) / 32, strips);
    BT_KERNEL_LAUNCH((colsum_stage1_kernel), grid, 256, 0, s, x, x_lo, N, C4, strips, scratch);
    BT_COUNT_LAUNCH();
    BT_KERNEL_LAUNCH((colsum_stage2_kernel), (C4 + 31) / 32, 256, 0, s, scratch, strips, C4, out);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

// Stage 2 alone: out[c] = the sum over the `groups` rows of partial [groups][C], in row order (for
// producers that leave per-row-group column sums themselves).
cudaError_t launch_colsum_stage2(const float* partial, int groups, int C, float* out, cudaStream_t s) {
    const int C4 = C / 4;
    BT_KERNEL_LAUNCH((colsum_stage2_kernel), (C4 + 31) / 32, 256, 0, s, partial, groups, C4, out);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

// ------------------------------------------------------------------ column sums without allocation

// Scratch for bt_op_colsum_static: lives in the library image, so every GPU that loads the
// library holds these 384 KB until the process exits.  All calls share it.
constexpr size_t kStaticColsumFloats = 96 * 1024;
static __device__ __align__(256) float g_colsum_static_scratch[kStaticColsumFloats];

static std::mutex g_static_mutex;
static float* g_static_scratch_ptr[64] = {nullptr};  // device address of the array, per device ordinal

// In host code the array's name is only a handle; the device address must be asked for, once
// per device, with that device current.
static cudaError_t static_scratch_address(float** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (g_static_scratch_ptr[dev] == nullptr) {
        float* p = nullptr;
        e = cudaGetSymbolAddress((void**)&p, g_colsum_static_scratch);
        if (e != cudaSuccess) return e;
        g_static_scratch_ptr[dev] = p;
    }
    *out = g_static_scratch_ptr[dev];
    return cudaSuccess;
}

}  // namespace bt

extern "C" size_t bt_op_colsum_static_max_floats(void) { return bt::kStaticColsumFloats; }

extern "C" bt_status bt_op_colsum_static(const float* x, int64_t N, int32_t C, float* out, void* stream) {
    using namespace bt;
    if (!x || !out) return bt_internal_fail(BT_ERR_INVALID_ARG, "colsum_static: NULL argument");
    if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(out)) & 15u)
        return bt_internal_fail(BT_ERR_INVALID_ARG, "colsum_static: pointers must be 16-byte aligned");
    if (N < 1 || C < 4 || C % 4) return bt_internal_fail(BT_ERR_INVALID_ARG, "colsum_static: bad sizes");
    if (colsum_scratch_floats(N, C) > kStaticColsumFloats)
        return bt_internal_fail(BT_ERR_UNSUPPORTED, "colsum_static: N x C needs more than the built-in scratch "
                                                    "(98304 floats); use bt_op_colsum with caller scratch");
    float* scratch = nullptr;
    cudaError_t e = static_scratch_address(&scratch);
    if (e == cudaSuccess) e = launch_colsum(x, nullptr, N, C, out, scratch, (cudaStream_t)stream);
    if (e != cudaSuccess) return bt_internal_fail(BT_ERR_CUDA, cudaGetErrorString(e));
    return BT_OK;
}

namespace bt {

// ------------------------------------------------------------------ gradient norm

constexpr int kNormBlocks = 148 * 8;
size_t grad_norm_scratch_bytes(int64_t) { return kNormBlocks * sizeof(double); }

__global__ void __launch_bounds__(256) sumsq_kernel(const float* __restrict__ g, int64_t n4, int64_t n,
                                                    double* __restrict__ partial) {
    pdl_wait();
    pdl_trigger();
    float acc = 0.f;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
        float4 v = ld4(g, i);
        acc += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
    // scalar tail (n not a multiple of 4)
    if (blockIdx.x == 0 && threadIdx.x < (n - n4 * 4)) {
        float v = g[n4 * 4 + threadIdx.x];
        acc += v * v;
    }
    double d = warp_sum_d((double)acc);
    __shared__ double sm[8];
    if ((threadIdx.x & 31) == 0) sm[threadIdx.x >> 5] = d;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < 8; ++w) t += sm[w];
        partial[blockIdx.x] = t;
    }
}

__global__ void __launch_bounds__(256) norm_finalize_kernel(const double* __restrict__ partial, int nb, float clip,
                                                            float* __restrict__ out2) {
    pdl_wait();
    pdl_trigger();
    __shared__ double sm[256];
    double t = 0.0;
    for (int i = threadIdx.x; i < nb; i += 256) t += partial[i];
    sm[threadIdx.x] = t;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) sm[threadIdx.x] += sm[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        double norm = sqrt(sm[0]);
        double sc = 1.0;
        if (clip > 0.f) {
            sc = (double)clip / (norm + 1e-6);
            if (sc > 1.0) sc = 1.0;
        }
        out2[0] = (float)norm;
        out2[1] = (float)sc;
    }
}

cudaError_t launch_grad_norm(const float* g, int64_t n, float clip, float* out2, void* scratch, cudaStream_t s) {
    int nb = grid_for(n / 4, 256, kNormBlocks);
    BT_KERNEL_LAUNCH((sumsq_kernel), nb, 256, 0, s, g, n / 4, n, (double*)scratch);
    BT_COUNT_LAUNCH();
    BT_KERNEL_LAUNCH((norm_finalize_kernel), 1, 256, 0, s, (const double*)scratch, nb, clip, out2);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

// ------------------------------------------------------------------ AdamW

__device__ __forceinline__ void adamw_elem(float& p, float g, float& m, float& v, bool decay, const AdamParams& hp,
                                           float scale) {
    g *= scale;
    float pp = decay ? p * (1.0f - hp.lr * hp.weight_decay) : p;
    m = hp.beta1 * m + (1.0f - hp.beta1) * g;
    v = hp.beta2 * v + (1.0f - hp.beta2) * g * g;
    float mh = m * hp.inv_c1;
    float vh = v * hp.inv_c2;
    p = pp - hp.lr * mh / (sqrtf(vh) + hp.eps);
}
__device__ __forceinline__ void adamw_vec(float4& p, float4 g, float4& m, float4& v, bool decay,
                                          const AdamParams& hp, float scale) {
    adamw_elem(p.x, g.x, m.x, v.x, decay, hp, scale);
    adamw_elem(p.y, g.y, m.y, v.y, decay, hp, scale);
    adamw_elem(p.z, g.z, m.z, v.z, decay, hp, scale);
    adamw_elem(p.w, g.w, m.w, v.w, decay, hp, scale);
}

// Flat arena: all tensors live back to back (each padded to 1024 floats), so the whole
// optimizer step is ONE grid-stride pass; decay_flags has one byte per 1024-float chunk.
__global__ void __launch_bounds__(256) adamw_flat_kernel(float* __restrict__ p, const float* __restrict__ g,
                                                         float* __restrict__ m, float* __restrict__ v, int64_t n4,
                                                         const uint8_t* __restrict__ decay_flags, AdamParams hp,
                                                         const float* __restrict__ d_scale) {
    pdl_wait();
    pdl_trigger();
    const float scale = d_scale ? *d_scale : 1.0f;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
        float4 pv = ld4(p, i), gv = ld4(g, i), mv = ld4(m, i), vv = ld4(v, i);
        adamw_vec(pv, gv, mv, vv, decay_flags[i >> 8] != 0, hp, scale);
        reinterpret_cast<float4*>(p)[i] = pv;
        reinterpret_cast<float4*>(m)[i] = mv;
        reinterpret_cast<float4*>(v)[i] = vv;
    }
}

cudaError_t launch_adamw_flat(float* p, const float* g, float* m, float* v, int64_t n, const uint8_t* decay_flags,
                              AdamParams hp, const float* d_scale, cudaStream_t s) {
    BT_KERNEL_LAUNCH((adamw_flat_kernel), grid_for(n / 4, 256, kStreamGridCap), 256, 0, s, p, g, m, v, n / 4, decay_flags, hp,
                                                                            d_scale);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

// Explicit tensor list: CTA b works on one 4096-element chunk of one tensor; the chunk table
// balances the load across tensors of very different sizes.
constexpr int kAdamChunk = 4096;
__global__ void __launch_bounds__(256) adamw_multi_kernel(const __grid_constant__ AdamTensorList tl, AdamParams hp,
                                                          const float* __restrict__ d_scale) {
    pdl_wait();
    pdl_trigger();
    const float scale = d_scale ? *d_scale : 1.0f;
    int t = 0;
    while (t + 1 < tl.n && (int)blockIdx.x >= tl.chunk_begin[t + 1]) ++t;
    const int64_t start = (int64_t)(blockIdx.x - tl.chunk_begin[t]) * kAdamChunk;
    const int64_t numel = tl.numel[t];
    const int64_t end = (start + kAdamChunk < numel) ? start + kAdamChunk : numel;
    float* p = tl.p[t];
    const float* g = tl.g[t];
    float* m = tl.m[t];
    float* v = tl.v[t];
    const bool decay = tl.decay[t] != 0;
    const int64_t vec_end = start + ((end - start) / 4) * 4;
    for (int64_t i = start + threadIdx.x * 4; i < vec_end; i += 256 * 4) {
        float4 pv = ld4(p, i / 4), gv = ld4(g, i / 4), mv = ld4(m, i / 4), vv = ld4(v, i / 4);
        adamw_vec(pv, gv, mv, vv, decay, hp, scale);
        reinterpret_cast<float4*>(p)[i / 4] = pv;
        reinterpret_cast<float4*>(m)[i / 4] = mv;
        reinterpret_cast<float4*>(v)[i / 4] = vv;
    }
    for (int64_t i = vec_end + threadIdx.x; i < end; i += 256) adamw_elem(p[i], g[i], m[i], v[i], decay, hp, scale);
}

cudaError_t launch_adamw_multi(const AdamTensorList& tl, AdamParams hp, const float* d_scale, cudaStream_t s) {
    int chunks = tl.chunk_begin[tl.n];
    if (chunks <= 0) return cudaSuccess;
    BT_KERNEL_LAUNCH((adamw_multi_kernel), chunks, 256, 0, s, tl, hp, d_scale);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}
int adamw_chunk_elems() { return kAdamChunk; }

// ------------------------------------------------------------------ gradient accumulation

// Micro-step i of n with weight w = 1/n: mode 0 (first) acc = w g; mode 1 acc += w g; mode 2 (last)
// g = acc + w g, so that after the last micro-step the gradient arena holds the gradient of the
// mean loss over all micro-batches.  The scalar loss is averaged the same way.
__global__ void __launch_bounds__(256) grad_accumulate_kernel(float* __restrict__ acc, float* __restrict__ g, int64_t n4,
                                                              float w, int mode, float* loss_acc, float* loss) {
    pdl_wait();
    pdl_trigger();
    if (loss != nullptr && blockIdx.x == 0 && threadIdx.x == 0) {
        const float l = w * loss[0];
        if (mode == 0) loss_acc[0] = l;
        else if (mode == 1) loss_acc[0] += l;
        else loss[0] = loss_acc[0] + l;
    }
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
        float4 v = ld4(g, i);
        v = make_float4(w * v.x, w * v.y, w * v.z, w * v.w);
        if (mode == 0) {
            reinterpret_cast<float4*>(acc)[i] = v;
        } else {
            const float4 a = ld4(acc, i);
            v = add4(a, v);
            if (mode == 1) reinterpret_cast<float4*>(acc)[i] = v;
            else reinterpret_cast<float4*>(g)[i] = v;
        }
    }
}
cudaError_t launch_grad_accumulate(float* acc, float* g, int64_t n, float w, int mode, float* loss_acc, float* loss,
                                   cudaStream_t s) {
    BT_KERNEL_LAUNCH((grad_accumulate_kernel), grid_for(n / 4, 256, kStreamGridCap), 256, 0, s, acc, g, n / 4, w, mode, loss_acc, loss);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

// ------------------------------------------------------------------ split-K reduction

__global__ void __launch_bounds__(256) splitk_reduce_kernel(const float* __restrict__ partials, int splits,
                                                            int64_t n4, float* __restrict__ out) {
    pdl_wait();
    pdl_trigger();
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
        float4 t = ld4(partials, i);
        for (int s = 1; s < splits; ++s) t = add4(t, ld4(partials, (int64_t)s * n4 + i));
        reinterpret_cast<float4*>(out)[i] = t;
    }
}
cudaError_t launch_splitk_reduce(const float* partials, int splits, int64_t n, float* out, cudaStream_t s) {
    BT_KERNEL_LAUNCH((splitk_reduce_kernel), grid_for(n / 4, 256, kStreamGridCap), 256, 0, s, partials, splits, n / 4, out);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

// ------------------------------------------------------------------ initialisation

// Counter-based normal generator: SplitMix64 of (seed, element index) -> two uniforms ->
// Box-Muller.  Only the distribution matters (the paper fixes std, not bit values).
__device__ __forceinline__ uint64_t splitmix64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
__global__ void __launch_bounds__(256) init_normal_kernel(float* __restrict__ p, int64_t n, float std, uint64_t seed,
                                                          uint64_t offset) {
    pdl_wait();
    pdl_trigger();
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        uint64_t r = splitmix64(splitmix64(seed) ^ (offset + (uint64_t)i));
        float u1 = ((float)(uint32_t)(r >> 40) + 0.5f) * (1.0f / 16777216.0f);
        float u2 = ((float)(uint32_t)((r >> 8) & 0xFFFFFFu) + 0.5f) * (1.0f / 16777216.0f);
        p[i] = std * sqrtf(-2.0f * logf(u1)) * cospif(2.0f * u2);
    }
}
__global__ void __launch_bounds__(256) fill_kernel(float* __restrict__ p, int64_t n, float v) {
    pdl_wait();
    pdl_trigger();
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        p[i] = v;
}
cudaError_t launch_init_normal(float* p, int64_t n, float std, uint64_t seed, uint64_t offset, cudaStream_t s) {
    BT_KERNEL_LAUNCH((init_normal_kernel), grid_for(n, 256, kStreamGridCap), 256, 0, s, p, n, std, seed, offset);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}
cudaError_t launch_fill(float* p, int64_t n, float v, cudaStream_t s) {
    BT_KERNEL_LAUNCH((fill_kernel), grid_for(n, 256, kStreamGridCap), 256, 0, s, p, n, v);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

}  // namespace bt
