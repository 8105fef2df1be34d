// Plain FP32 causal attention, forward and backward: the bring-up reference for the
// tensor-core kernels (selected with BT_FLAG_ATTN_SIMT).  One warp owns one (sequence, head,
// position); lanes own head dimensions; every dot product is a warp-shuffle reduction.  The
// forward is the textbook two-pass softmax (row maximum first), deliberately not the online
// recurrence the fast kernel uses.
#include "common.cuh"

namespace bt {

constexpr int kAsWarps = 8;

template <int DPL>
__device__ __forceinline__ void load_vec(const float* p, int d, int lane, float (&r)[DPL]) {
#pragma unroll
    for (int k = 0; k < DPL; ++k) {
        int c = lane + 32 * k;
        r[k] = (c < d) ? p[c] : 0.f;
    }
}
template <int DPL>
__device__ __forceinline__ float dot_vec(const float (&a)[DPL], const float (&b)[DPL]) {
    float s = 0.f;
#pragma unroll
    for (int k = 0; k < DPL; ++k) s = fmaf(a[k], b[k], s);
    return warp_sum(s);
}

template <int DPL>
__global__ void __launch_bounds__(kAsWarps * 32) attn_fwd_simt_kernel(const float* __restrict__ qkv, int B, int T,
                                                                       int C, int H, float* o, float* o_hi,
                                                                       float* o_lo, float* __restrict__ lse) {
    pdl_wait();
    pdl_trigger();
    const int lane = threadIdx.x & 31;
    const int64_t gw = (int64_t)blockIdx.x * kAsWarps + (threadIdx.x >> 5);
    if (gw >= (int64_t)B * H * T) return;
    const int i = (int)(gw % T), h = (int)((gw / T) % H), b = (int)(gw / ((int64_t)T * H));
    const int d = C / H;
    const float scale = 1.0f / sqrtf((float)d);
    const float* base = qkv + (int64_t)b * T * 3 * C + h * d;
    float q[DPL], kv[DPL], acc[DPL];
    load_vec<DPL>(base + (int64_t)i * 3 * C, d, lane, q);
    float mx = -INFINITY;
    for (int j = 0; j <= i; ++j) {
        load_vec<DPL>(base + (int64_t)j * 3 * C + C, d, lane, kv);
        mx = fmaxf(mx, dot_vec<DPL>(q, kv) * scale);
    }
    float l = 0.f;
#pragma unroll
    for (int k = 0; k < DPL; ++k) acc[k] = 0.f;
    for (int j = 0; j <= i; ++j) {
        load_vec<DPL>(base + (int64_t)j * 3 * C + C, d, lane, kv);
        float p = expf(dot_vec<DPL>(q, kv) * scale - mx);
        l += p;
        load_vec<DPL>(base + (int64_t)j * 3 * C + 2 * C, d, lane, kv);
#pragma unroll
        for (int k = 0; k < DPL; ++k) acc[k] = fmaf(p, kv[k], acc[k]);
    }
    const int64_t orow = ((int64_t)b * T + i) * C + h * d;
#pragma unroll
    for (int k = 0; k < DPL; ++k) {
        int c = lane + 32 * k;
        if (c < d) {
            float v = acc[k] / l;
            if (o) o[orow + c] = v;
            if (o_hi) {
                float hi, lo;
                split_tf32(v, hi, lo);
                o_hi[orow + c] = hi;
                o_lo[orow + c] = lo;
            }
        }
    }
    if (lane == 0 && lse) lse[((int64_t)b * H + h) * T + i] = mx + logf(l);
}

// dvec[b,h,i] = sum_c do[i,c] * o[i,c] over the head's columns.
template <int DPL>
__global__ void __launch_bounds__(kAsWarps * 32) attn_dvec_kernel(const float* __restrict__ o,
                                                                   const float* __restrict__ o_lo,
                                                                   const float* __restrict__ d_o,
                                                                   const float* __restrict__ d_o_lo, int B, int T,
                                                                   int C, int H, float* __restrict__ dvec) {
    pdl_wait();
    pdl_trigger();
    const int lane = threadIdx.x & 31;
    const int64_t gw = (int64_t)blockIdx.x * kAsWarps + (threadIdx.x >> 5);
    if (gw >= (int64_t)B * H * T) return;
    const int i = (int)(gw % T), h = (int)((gw / T) % H), b = (int)(gw / ((int64_t)T * H));
    const int d = C / H;
    const int64_t row = ((int64_t)b * T + i) * C + h * d;
    float a[DPL], g[DPL];
    load_vec<DPL>(o + row, d, lane, a);
    if (o_lo) {
        float t[DPL];
        load_vec<DPL>(o_lo + row, d, lane, t);
#pragma unroll
        for (int k = 0; k < DPL; ++k) a[k] += t[k];
    }
    load_vec<DPL>(d_o + row, d, lane, g);
    if (d_o_lo) {
        float t[DPL];
        load_vec<DPL>(d_o_lo + row, d, lane, t);
#pragma unroll
        for (int k = 0; k < DPL; ++k) g[k] += t[k];
    }
    float s = dot_vec<DPL>(a, g);
    if (lane == 0) dvec[gw] = s;
}

template <int DPL>
__device__ __forceinline__ void store_head(const float (&v)[DPL], int d, int lane, int64_t off, float* raw,
                                           float* hi, float* lo) {
#pragma unroll
    for (int k = 0; k < DPL; ++k) {
        int c = lane + 32 * k;
        if (c < d) {
            if (raw) raw[off + c] = v[k];
            if (hi) {
                float a, b;
                split_tf32(v[k], a, b);
                hi[off + c] = a;
                lo[off + c] = b;
            }
        }
    }
}

// dq_i = scale * sum_{j<=i} dS_ij k_j
template <int DPL>
__global__ void __launch_bounds__(kAsWarps * 32) attn_bwd_dq_simt_kernel(
    const float* __restrict__ qkv, const float* __restrict__ lse, const float* __restrict__ d_o,
    const float* __restrict__ dvec, int B, int T, int C, int H, float* dqkv, float* dqkv_hi, float* dqkv_lo) {
    pdl_wait();
    pdl_trigger();
    const int lane = threadIdx.x & 31;
    const int64_t gw = (int64_t)blockIdx.x * kAsWarps + (threadIdx.x >> 5);
    if (gw >= (int64_t)B * H * T) return;
    const int i = (int)(gw % T), h = (int)((gw / T) % H), b = (int)(gw / ((int64_t)T * H));
    const int d = C / H;
    const float scale = 1.0f / sqrtf((float)d);
    const float* base = qkv + (int64_t)b * T * 3 * C + h * d;
    float q[DPL], g[DPL], kk[DPL], vv[DPL], acc[DPL];
    load_vec<DPL>(base + (int64_t)i * 3 * C, d, lane, q);
    load_vec<DPL>(d_o + ((int64_t)b * T + i) * C + h * d, d, lane, g);
    const float L = lse[gw], D = dvec[gw];
#pragma unroll
    for (int k = 0; k < DPL; ++k) acc[k] = 0.f;
    for (int j = 0; j <= i; ++j) {
        load_vec<DPL>(base + (int64_t)j * 3 * C + C, d, lane, kk);
        load_vec<DPL>(base + (int64_t)j * 3 * C + 2 * C, d, lane, vv);
        float p = expf(dot_vec<DPL>(q, kk) * scale - L);
        float ds = p * (dot_vec<DPL>(g, vv) - D) * scale;
#pragma unroll
        for (int k = 0; k < DPL; ++k) acc[k] = fmaf(ds, kk[k], acc[k]);
    }
    store_head<DPL>(acc, d, lane, ((int64_t)b * T + i) * 3 * C + h * d, dqkv, dqkv_hi, dqkv_lo);
}

// dk_j = scale * sum_{i>=j} dS_ij q_i ;  dv_j = sum_{i>=j} P_ij do_i
template <int DPL>
__global__ void __launch_bounds__(kAsWarps * 32) attn_bwd_dkv_simt_kernel(
    const float* __restrict__ qkv, const float* __restrict__ lse, const float* __restrict__ d_o,
    const float* __restrict__ dvec, int B, int T, int C, int H, float* dqkv, float* dqkv_hi, float* dqkv_lo) {
    pdl_wait();
    pdl_trigger();
    const int lane = threadIdx.x & 31;
    const int64_t gw = (int64_t)blockIdx.x * kAsWarps + (threadIdx.x >> 5);
    if (gw >= (int64_t)B * H * T) return;
    const int j = (int)(gw % T), h = (int)((gw / T) % H), b = (int)(gw / ((int64_t)T * H));
    const int d = C / H;
    const float scale = 1.0f / sqrtf((float)d);
    const float* base = qkv + (int64_t)b * T * 3 * C + h * d;
    float kk[DPL], vv[DPL], q[DPL], g[DPL], dk[DPL], dv[DPL];
    load_vec<DPL>(base + (int64_t)j * 3 * C + C, d, lane, kk);
    load_vec<DPL>(base + (int64_t)j * 3 * C + 2 * C, d, lane, vv);
#pragma unroll
    for (int k = 0; k < DPL; ++k) dk[k] = dv[k] = 0.f;
    const int64_t srow = ((int64_t)b * H + h) * T;
    for (int i = j; i < T; ++i) {
        load_vec<DPL>(base + (int64_t)i * 3 * C, d, lane, q);
        load_vec<DPL>(d_o + ((int64_t)b * T + i) * C + h * d, d, lane, g);
        float p = expf(dot_vec<DPL>(q, kk) * scale - lse[srow + i]);
        float ds = p * (dot_vec<DPL>(g, vv) - dvec[srow + i]) * scale;
#pragma unroll
        for (int k = 0; k < DPL; ++k) {
            dv[k] = fmaf(p, g[k], dv[k]);
            dk[k] = fmaf(ds, q[k], dk[k]);
        }
    }
    const int64_t off = ((int64_t)b * T + j) * 3 * C + h * d;
    store_head<DPL>(dk, d, lane, off + C, dqkv, dqkv_hi, dqkv_lo);
    store_head<DPL>(dv, d, lane, off + 2 * C, dqkv, dqkv_hi, dqkv_lo);
}

cudaError_t launch_attention_fwd_simt(const float* qkv, int B, int T, int C, int H, float* o, float* o_hi,
                                      float* o_lo, float* lse, cudaStream_t s) {
    const int d = C / H;
    const int64_t warps = (int64_t)B * H * T;
    const int grid = (int)((warps + kAsWarps - 1) / kAsWarps);
    if (d <= 32) BT_KERNEL_LAUNCH((attn_fwd_simt_kernel<1>), grid, kAsWarps * 32, 0, s, qkv, B, T, C, H, o, o_hi, o_lo, lse);
    else if (d <= 64) BT_KERNEL_LAUNCH((attn_fwd_simt_kernel<2>), grid, kAsWarps * 32, 0, s, qkv, B, T, C, H, o, o_hi, o_lo, lse);
    else BT_KERNEL_LAUNCH((attn_fwd_simt_kernel<4>), grid, kAsWarps * 32, 0, s, qkv, B, T, C, H, o, o_hi, o_lo, lse);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

cudaError_t launch_attention_dvec(const float* o, const float* o_lo, const float* d_o, const float* d_o_lo, int B,
                                  int T, int C, int H, float* dvec, cudaStream_t s) {
    const int d = C / H;
    const int64_t warps = (int64_t)B * H * T;
    const int grid = (int)((warps + kAsWarps - 1) / kAsWarps);
    if (d <= 32) BT_KERNEL_LAUNCH((attn_dvec_kernel<1>), grid, kAsWarps * 32, 0, s, o, o_lo, d_o, d_o_lo, B, T, C, H, dvec);
    else if (d <= 64) BT_KERNEL_LAUNCH((attn_dvec_kernel<2>), grid, kAsWarps * 32, 0, s, o, o_lo, d_o, d_o_lo, B, T, C, H, dvec);
    else BT_KERNEL_LAUNCH((attn_dvec_kernel<4>), grid, kAsWarps * 32, 0, s, o, o_lo, d_o, d_o_lo, B, T, C, H, dvec);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

cudaError_t launch_attention_bwd_simt(const float* qkv, const float* o, const float* o_lo, const float* lse,
                                      const float* d_o, int B, int T, int C, int H, float* dqkv, float* dqkv_hi,
                                      float* dqkv_lo, float* dvec, cudaStream_t s) {
    cudaError_t e = launch_attention_dvec(o, o_lo, d_o, nullptr, B, T, C, H, dvec, s);
    if (e != cudaSuccess) return e;
    const int d = C / H;
    const int64_t warps = (int64_t)B * H * T;
    const int grid = (int)((warps + kAsWarps - 1) / kAsWarps);
#define BT_AB(DPL)                                                                                                  \
    BT_KERNEL_LAUNCH((attn_bwd_dq_simt_kernel<DPL>), grid, kAsWarps * 32, 0, s, qkv, lse, d_o, dvec, B, T, C, H, dqkv, dqkv_hi,     \
                                                                 dqkv_lo);                                          \
    BT_KERNEL_LAUNCH((attn_bwd_dkv_simt_kernel<DPL>), grid, kAsWarps * 32, 0, s, qkv, lse, d_o, dvec, B, T, C, H, dqkv, dqkv_hi,    \
                                                                  dqkv_lo)
    if (d <= 32) { BT_AB(1); } else if (d <= 64) { BT_AB(2); } else { BT_AB(4); }
#undef BT_AB
    BT_COUNT_LAUNCH();
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

}  // namespace bt
