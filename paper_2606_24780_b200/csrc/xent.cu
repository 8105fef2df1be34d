// Fused softmax cross-entropy forward + backward over the padded vocabulary.
//
// One CTA of 512 threads owns one row of logits.  The row (201 KB at Vp = 50304) is read
// from HBM exactly once into registers with 128-bit loads, reduced (max, then sum of
// exponentials) with warp shuffles plus one shared-memory hop, and the gradient
// (softmax - onehot) * inv_count is written once, raw and/or as TF32 hi/lo planes for the two
// LM-head backward GEMMs.  Per-row losses go to an array that a second one-CTA kernel sums in
// index order, so the mean loss is deterministic.
#include "common.cuh"

namespace bt {

constexpr int kXentThreads = 512;

__device__ __forceinline__ float block_reduce(float v, bool is_max, float* sm) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v = is_max ? warp_max(v) : warp_sum(v);
    __syncthreads();  // protect sm reuse between consecutive reductions
    if (lane == 0) sm[warp] = v;
    __syncthreads();
    float r = sm[0];
    for (int w = 1; w < kXentThreads / 32; ++w) r = is_max ? fmaxf(r, sm[w]) : r + sm[w];
    return r;
}

// A target outside [0, V) is never used as an index: it is treated as class 0 and row + 1 is
// recorded in *bad (first writer wins; bad may be null).
__device__ __forceinline__ int checked_target(int t, int V, int64_t row, int* bad) {
    if ((unsigned)t < (unsigned)V) return t;
    if (bad && threadIdx.x == 0) atomicCAS(bad, 0, (int)row + 1);
    return 0;
}

template <int ITEMS>
__global__ void __launch_bounds__(kXentThreads) xent_kernel(const float* logits,   // may alias dl_hi (in place)
                                                            const int32_t* __restrict__ targets, int V4,
                                                            float inv_count, float* __restrict__ losses, float* dl,
                                                            float* dl_hi, float* dl_lo, int V, int* bad) {
    pdl_wait();
    pdl_trigger();
    __shared__ float sm[kXentThreads / 32];
    const int64_t row = blockIdx.x;
    const int64_t base = row * V4;
    float4 v[ITEMS];
    float mx = -INFINITY;
#pragma unroll
    for (int k = 0; k < ITEMS; ++k) {
        int idx = threadIdx.x + kXentThreads * k;
        if (idx < V4) {
            v[k] = __ldcs(reinterpret_cast<const float4*>(logits) + base + idx);
            mx = fmaxf(mx, fmaxf(fmaxf(v[k].x, v[k].y), fmaxf(v[k].z, v[k].w)));
        }
    }
    mx = block_reduce(mx, true, sm);
    float sum = 0.f;
#pragma unroll
    for (int k = 0; k < ITEMS; ++k) {
        int idx = threadIdx.x + kXentThreads * k;
        if (idx < V4) {
            v[k].x = expf(v[k].x - mx);
            v[k].y = expf(v[k].y - mx);
            v[k].z = expf(v[k].z - mx);
            v[k].w = expf(v[k].w - mx);
            sum += (v[k].x + v[k].y) + (v[k].z + v[k].w);
        }
    }
    sum = block_reduce(sum, false, sm);
    const int t = checked_target(targets[row], V, row, bad);
    if (threadIdx.x == 0) losses[row] = (mx + logf(sum)) - logits[row * V4 * 4 + t];
    if (dl == nullptr && dl_hi == nullptr) return;
    // the gradient may be written over the logits themselves (in place): every thread has its part of
    // the row in registers by now, and the target's logit has been read before anyone stores
    __syncthreads();
    const float sc = inv_count / sum;
#pragma unroll
    for (int k = 0; k < ITEMS; ++k) {
        int idx = threadIdx.x + kXentThreads * k;
        if (idx < V4) {
            float4 r = make_float4(v[k].x * sc, v[k].y * sc, v[k].z * sc, v[k].w * sc);
            if ((t >> 2) == idx) {
                int j = t & 3;
                if (j == 0) r.x -= inv_count;
                else if (j == 1) r.y -= inv_count;
                else if (j == 2) r.z -= inv_count;
                else r.w -= inv_count;
            }
            store_raw_split(r, dl, dl_hi, dl_lo, base + idx);
        }
    }
}

// The same row arithmetic for long rows and many more rows than SMs, as a row loop: one CTA per SM
// keeps the NEXT row on its way into shared memory (16-byte asynchronous copies, each thread copying
// exactly the elements it will read, so that completion needs no barrier) while the current row, held
// in registers, is reduced and its gradient stored.  With the grid-per-row kernel an SM alternates
// between a load phase, an arithmetic phase and a store phase (the row fills the register file, so a
// second CTA cannot be resident); here the loads of row r + 1 run under the arithmetic and the
// stores of row r.  Element-to-thread assignment and reduction order are those of xent_kernel, so the
// results are bit-identical.
__device__ __forceinline__ void cp_async16(float4* dst_smem, const float4* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst_smem)), "l"(src)
                 : "memory");
}

template <int ITEMS>
__global__ void __launch_bounds__(kXentThreads) xent_stream_kernel(const float* logits,   // may alias dl_hi (in place)
                                                                   const int32_t* __restrict__ targets, int V4,
                                                                   float inv_count, float* __restrict__ losses,
                                                                   float* dl, float* dl_hi, float* dl_lo, int V, int* bad,
                                                                   int64_t N) {
    extern __shared__ float4 row_s[];
    __shared__ float sm[kXentThreads / 32];
    pdl_wait();
    pdl_trigger();
    auto fetch = [&](int64_t r) {
        const float4* src = reinterpret_cast<const float4*>(logits) + r * V4;
#pragma unroll
        for (int k = 0; k < ITEMS; ++k) {
            int idx = threadIdx.x + kXentThreads * k;
            if (idx < V4) cp_async16(row_s + idx, src + idx);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    if ((int64_t)blockIdx.x < N) fetch(blockIdx.x);
    for (int64_t row = blockIdx.x; row < N; row += gridDim.x) {
        const int64_t base = row * V4;
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        float4 v[ITEMS];
        float mx = -INFINITY;
#pragma unroll
        for (int k = 0; k < ITEMS; ++k) {
            int idx = threadIdx.x + kXentThreads * k;
            if (idx < V4) {
                v[k] = row_s[idx];
                mx = fmaxf(mx, fmaxf(fmaxf(v[k].x, v[k].y), fmaxf(v[k].z, v[k].w)));
            }
        }
        // this thread's part of the row is in registers (the maximum has consumed it): its shared-memory
        // slots may take the next row
        if (row + gridDim.x < N) fetch(row + gridDim.x);
        mx = block_reduce(mx, true, sm);
        float sum = 0.f;
#pragma unroll
        for (int k = 0; k < ITEMS; ++k) {
            int idx = threadIdx.x + kXentThreads * k;
            if (idx < V4) {
                v[k].x = expf(v[k].x - mx);
                v[k].y = expf(v[k].y - mx);
                v[k].z = expf(v[k].z - mx);
                v[k].w = expf(v[k].w - mx);
                sum += (v[k].x + v[k].y) + (v[k].z + v[k].w);
            }
        }
        sum = block_reduce(sum, false, sm);
        const int t = checked_target(targets[row], V, row, bad);
        if (threadIdx.x == 0) losses[row] = (mx + logf(sum)) - logits[row * V4 * 4 + t];
        if (dl == nullptr && dl_hi == nullptr) continue;
        __syncthreads();   // in place: the target's logit has been read before anyone stores
        const float sc = inv_count / sum;
#pragma unroll
        for (int k = 0; k < ITEMS; ++k) {
            int idx = threadIdx.x + kXentThreads * k;
            if (idx < V4) {
                float4 r = make_float4(v[k].x * sc, v[k].y * sc, v[k].z * sc, v[k].w * sc);
                if ((t >> 2) == idx) {
                    int j = t & 3;
                    if (j == 0) r.x -= inv_count;
                    else if (j == 1) r.y -= inv_count;
                    else if (j == 2) r.z -= inv_count;
                    else r.w -= inv_count;
                }
                store_raw_split(r, dl, dl_hi, dl_lo, base + idx);
            }
        }
    }
}

// Rows longer than the register path covers: three passes over global memory (the second and
// third are served by L2 for rows of a few hundred KB).
__global__ void __launch_bounds__(kXentThreads) xent_generic_kernel(const float* __restrict__ logits,
                                                                    const int32_t* __restrict__ targets, int V4,
                                                                    float inv_count, float* __restrict__ losses,
                                                                    float* dl, float* dl_hi, float* dl_lo, int V,
                                                                    int* bad) {
    pdl_wait();
    pdl_trigger();
    __shared__ float sm[kXentThreads / 32];
    const int64_t row = blockIdx.x;
    const int64_t base = row * V4;
    float mx = -INFINITY;
    for (int idx = threadIdx.x; idx < V4; idx += kXentThreads) {
        float4 a = ld4(logits, base + idx);
        mx = fmaxf(mx, fmaxf(fmaxf(a.x, a.y), fmaxf(a.z, a.w)));
    }
    mx = block_reduce(mx, true, sm);
    float sum = 0.f;
    for (int idx = threadIdx.x; idx < V4; idx += kXentThreads) {
        float4 a = ld4(logits, base + idx);
        sum += (expf(a.x - mx) + expf(a.y - mx)) + (expf(a.z - mx) + expf(a.w - mx));
    }
    sum = block_reduce(sum, false, sm);
    const int t = checked_target(targets[row], V, row, bad);
    if (threadIdx.x == 0) losses[row] = (mx + logf(sum)) - logits[row * V4 * 4 + t];
    if (dl == nullptr && dl_hi == nullptr) return;
    const float sc = inv_count / sum;
    for (int idx = threadIdx.x; idx < V4; idx += kXentThreads) {
        float4 a = ld4(logits, base + idx);
        float4 r = make_float4(expf(a.x - mx) * sc, expf(a.y - mx) * sc, expf(a.z - mx) * sc, expf(a.w - mx) * sc);
        if ((t >> 2) == idx) {
            int j = t & 3;
            if (j == 0) r.x -= inv_count;
            else if (j == 1) r.y -= inv_count;
            else if (j == 2) r.z -= inv_count;
            else r.w -= inv_count;
        }
        store_raw_split(r, dl, dl_hi, dl_lo, base + idx);
    }
}

// loss_mean = inv_count * sum_n losses[n], summed in a fixed tree order by one CTA.
__global__ void __launch_bounds__(1024) loss_mean_kernel(const float* __restrict__ losses, int64_t N, float inv_count,
                                                         float* __restrict__ loss_mean) {
    pdl_wait();
    pdl_trigger();
    __shared__ double sm[1024];
    double t = 0.0;
    for (int64_t i = threadIdx.x; i < N; i += 1024) t += (double)losses[i];
    sm[threadIdx.x] = t;
    __syncthreads();
    for (int o = 512; o > 0; o >>= 1) {
        if (threadIdx.x < o) sm[threadIdx.x] += sm[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) *loss_mean = (float)(sm[0] * (double)inv_count);
}

// BT_XENT_STREAM=0 keeps long rows on the grid-per-row kernel (for comparison runs).
static const bool g_xent_stream = []() {
    const char* v = getenv("BT_XENT_STREAM");
    return !(v && v[0] == '0');
}();

// Rows up to this many columns take the one-pass kernel, which may write its output over its input.
int softmax_xent_max_in_place_columns() { return 25 * kXentThreads * 4; }

cudaError_t launch_softmax_xent(const float* logits, const int32_t* targets, int64_t N, int Vp, float inv_count,
                                float* losses, float* loss_mean, float* dl, float* dl_hi, float* dl_lo, int V,
                                int* bad, cudaStream_t s) {
    const int V4 = Vp / 4;
    const int items = (V4 + kXentThreads - 1) / kXentThreads;
#define BT_XENT(I)                                                                                              \
    BT_KERNEL_LAUNCH((xent_kernel<I>), (int)N, kXentThreads, 0, s, logits, targets, V4, inv_count, losses, dl, dl_hi, dl_lo, V, bad)
    if (items <= 1) BT_XENT(1);
    else if (items <= 2) BT_XENT(2);
    else if (items <= 4) BT_XENT(4);
    else if (items <= 8) BT_XENT(8);
    else if (items <= 16) BT_XENT(16);
    else if (items <= 25) {
        int dev = 0, sms = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const size_t row_bytes = (size_t)V4 * sizeof(float4);
        if (g_xent_stream && N >= 4 * (int64_t)sms && row_bytes <= 220 * 1024) {
            // set per call: the attribute is kept per device, and this runs once per step
            cudaError_t e = cudaFuncSetAttribute(xent_stream_kernel<25>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
            if (e != cudaSuccess) return e;
            BT_KERNEL_LAUNCH((xent_stream_kernel<25>), sms, kXentThreads, row_bytes, s, logits, targets, V4, inv_count, losses,
                             dl, dl_hi, dl_lo, V, bad, N);
        } else {
            BT_XENT(25);
        }
    }
    else BT_KERNEL_LAUNCH((xent_generic_kernel), (int)N, kXentThreads, 0, s, logits, targets, V4, inv_count, losses, dl, dl_hi, dl_lo, V, bad);
#undef BT_XENT
    BT_COUNT_LAUNCH();
    if (loss_mean) {
        BT_KERNEL_LAUNCH((loss_mean_kernel), 1, 1024, 0, s, losses, N, inv_count, loss_mean);
        BT_COUNT_LAUNCH();
    }
    return cudaGetLastError();
}

}  // namespace bt
