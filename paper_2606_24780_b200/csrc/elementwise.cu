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

// One thread per float4 of the output: x[n,:] = wte[tok[n],:] + wpe[n mod T,:].
__global__ void __launch_bounds__(256) embedding_fwd_kernel(const int32_t* __restrict__ tok,
                                                            const float* __restrict__ wte,
                                                            const float* __restrict__ wpe, int64_t N, int T, int C4,
                                                            float* __restrict__ x) {
    pdl_wait();
    pdl_trigger();
    int64_t total = N * C4;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        int64_t n = i / C4;
        int c = (int)(i - n * C4);
        float4 e = ld4(wte, (int64_t)tok[n] * C4 + c);
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
                                 float* x, cudaStream_t s) {
    BT_KERNEL_LAUNCH((embedding_fwd_kernel), grid_for(N * (C / 4), 256, kStreamGridCap), 256, 0, s, tok, wte, wpe, N, T, C / 4, x);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

// ------------------------------------------------------------------ embedding backward

// One CTA per position n.  The CTA owning the FIRST occurrence of a token id gathers all
// later positions with that id, in ascending order, and adds the row sum to dwte[id,:]; all
// other CTAs exit.  One writer per row and a fixed order: deterministic, no atomics, and the
// heavy-tailed (Zipf) token distribution costs one long row sum instead of contended atomics.
// Both scans read the token array four ids per thread (128-bit loads); a round of 1024 positions
// without a match -- nearly all of them for a rare token -- costs one load and one barrier.
constexpr int kEmbRound = 1024;   // positions per round: 256 threads x 4
__device__ __forceinline__ int4 load_tok4(const int32_t* __restrict__ tok, int j, int lo, int hi, int fill, bool vec) {
    // ids at positions j .. j+3; positions outside [lo, hi) read as `fill`
    if (vec && j >= lo && j + 3 < hi) return *reinterpret_cast<const int4*>(tok + j);
    int4 v;
    v.x = (j >= lo && j < hi) ? tok[j] : fill;
    v.y = (j + 1 >= lo && j + 1 < hi) ? tok[j + 1] : fill;
    v.z = (j + 2 >= lo && j + 2 < hi) ? tok[j + 2] : fill;
    v.w = (j + 3 >= lo && j + 3 < hi) ? tok[j + 3] : fill;
    return v;
}
__global__ void __launch_bounds__(256) embedding_bwd_wte_kernel(const int32_t* __restrict__ tok,
                                                                const float* __restrict__ dx, int N, int C4,
                                                                float* __restrict__ dwte, int vec) {
    pdl_wait();
    pdl_trigger();
    const int n = blockIdx.x;
    const int t = tok[n];
    int found = 0;
    for (int j = 4 * threadIdx.x; j < n; j += kEmbRound) {
        const int4 v = load_tok4(tok, j, 0, n, ~t, vec != 0);
        found |= (v.x == t) | (v.y == t) | (v.z == t) | (v.w == t);
    }
    if (__syncthreads_or(found)) return;

    __shared__ int list[kEmbRound];
    __shared__ int wcount[8];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int a0 = n & ~3;   // rounds start on a multiple of four so that the 128-bit loads stay aligned
    for (int c0 = 0; c0 < C4; c0 += 256) {
        const int c = c0 + threadIdx.x;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int base = a0; base < N; base += kEmbRound) {
            const int j = base + 4 * threadIdx.x;
            const int4 v = load_tok4(tok, j, n, N, ~t, vec != 0);
            const int m = (v.x == t ? 1 : 0) | (v.y == t ? 2 : 0) | (v.z == t ? 4 : 0) | (v.w == t ? 8 : 0);
            if (!__syncthreads_or(m)) continue;
            // ordered list of the round's matches: thread order, then position inside the thread
            const int cnt = __popc(m);
            int pre = cnt;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, pre, d);
                if (lane >= d) pre += y;
            }
            if (lane == 31) wcount[warp] = pre;
            __syncthreads();
            int off = pre - cnt, total = 0;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                if (k < warp) off += wcount[k];
                total += wcount[k];
            }
#pragma unroll
            for (int q = 0; q < 4; ++q)
                if (m & (1 << q)) list[off++] = j + q;
            __syncthreads();
            if (c < C4) {   // eight rows in flight (a frequent token has dozens per round), added in list order
                int k = 0;
                for (; k + 8 <= total; k += 8) {
                    float4 r[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) r[q] = ld4(dx, (int64_t)list[k + q] * C4 + c);
#pragma unroll
                    for (int q = 0; q < 8; ++q) acc = add4(acc, r[q]);
                }
                for (; k < total; ++k) acc = add4(acc, ld4(dx, (int64_t)list[k] * C4 + c));
            }
            __syncthreads();
        }
        if (c < C4) {
            float4* dst = reinterpret_cast<float4*>(dwte) + (int64_t)t * C4 + c;
            *dst = add4(*dst, acc);
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

cudaError_t launch_embedding_bwd(const int32_t* tok, const float* dx, int64_t N, int T, int C, float* dwte,
                                 float* dwpe, cudaStream_t s) {
    const int vec = (reinterpret_cast<uintptr_t>(tok) & 15u) == 0 ? 1 : 0;
    BT_KERNEL_LAUNCH((embedding_bwd_wte_kernel), (int)N, 256, 0, s, tok, dx, (int)N, C / 4, dwte, vec);
    BT_COUNT_LAUNCH();
    BT_KERNEL_LAUNCH((embedding_bwd_wpe_kernel), grid_for((int64_t)T * (C / 4), 256, kStreamGridCap), 256, 0, s, 
        dx, (int)(N / T), T, C / 4, dwpe);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

// ------------------------------------------------------------------ GELU

__device__ __forceinline__ float gelu_grad_f(float x, bool tanh_form) {
    if (tanh_form) {
        float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
        float t = tanhf(u);
        float du = 0.7978845608028654f * (1.0f + 3.0f * 0.044715f * x * x);
        return 0.5f * (1.0f + t) + 0.5f * x * (1.0f - t * t) * du;
    }
    // Phi(x) + x phi(x)
    return 0.5f * (1.0f + erff(x * 0.7071067811865476f)) + x * 0.3989422804014327f * expf(-0.5f * x * x);
}

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
    if (blockIdx.x == 0 && threadIdx.x == 0) {
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
