// LayerNorm forward and backward.  One warp owns one row: the row is read once into
// registers with 128-bit loads, both row reductions are warp shuffles (no shared memory on
// the row path), and the output is written once -- raw and/or as TF32 hi/lo planes for the
// GEMM that consumes it.  The backward's parameter gradients are accumulated per lane over a
// strip of rows, combined across the CTA's warps in warp order, written as per-CTA partials
// and summed by a second kernel in CTA order (deterministic).
#include "common.cuh"

namespace bt {

constexpr int kLnWarps = 8;   // most warps a CTA of the warp-per-row kernels has

// Launch shape of the warp-per-row kernels: ctas_per_sm * 148 CTAs of w warps, every warp walking
// rows warp, warp + total, ...  All warps are resident at once and the kernel is memory-bound, so
// its time goes like (rows per warp) x (warps per SM); w in 4..8 is chosen to minimise
// ceil(N / total warps) * w, i.e. the work lost to a last, partly filled pass over the warps
// (N = 8192 rows on 148 SMs: with eight warps per CTA the fourth pass is 46 % full, with seven 99 %).
struct LnShape { int ctas, warps; };
static inline LnShape ln_shape(int64_t N, int ctas_per_sm) {
    const int64_t slots = 148LL * ctas_per_sm;
    if (N <= slots * 4) return LnShape{(int)((N + 3) / 4), 4};   // fewer rows than one round of the smallest shape
    int best_w = kLnWarps;
    int64_t best = -1;
    for (int w = kLnWarps; w >= 4; --w) {
        const int64_t cost = ((N + slots * w - 1) / (slots * w)) * w;
        if (best < 0 || cost < best) { best = cost; best_w = w; }
    }
    return LnShape{(int)slots, best_w};
}

// VPL = float4 values per lane (C <= 128 * VPL).
template <int VPL>
__global__ void __launch_bounds__(kLnWarps * 32) ln_fwd_kernel(const float* __restrict__ x,
                                                               const float* __restrict__ gamma,
                                                               const float* __restrict__ beta, int64_t N, int C4,
                                                               float* y, float* y_hi, float* y_lo,
                                                               float* __restrict__ mean, float* __restrict__ rstd) {
    pdl_wait();
    pdl_trigger();
    // one row per warp and no row loop: the loop form costs 32 more registers (80 against 48) and with
    // them two resident CTAs per SM
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t row = (int64_t)blockIdx.x * kLnWarps + warp;
    if (row >= N) return;
    const float inv_c = 1.0f / (float)(C4 * 4);
    float4 v[VPL];
    float s = 0.f;
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        int idx = lane + 32 * k;
        if (idx < C4) {
            v[k] = ld4(x, row * C4 + idx);
            s += (v[k].x + v[k].y) + (v[k].z + v[k].w);
        }
    }
    const float mu = warp_sum(s) * inv_c;
    float q = 0.f;
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        int idx = lane + 32 * k;
        if (idx < C4) {
            float a = v[k].x - mu, b = v[k].y - mu, c = v[k].z - mu, d = v[k].w - mu;
            q += (a * a + b * b) + (c * c + d * d);
        }
    }
    const float var = warp_sum(q) * inv_c;
    const float rs = 1.0f / sqrtf(var + kLnEps);
#pragma unroll
    for (int k = 0; k < VPL; ++k) {
        int idx = lane + 32 * k;
        if (idx < C4) {
            float4 g = ld4(gamma, idx), b = ld4(beta, idx), r;
            r.x = g.x * ((v[k].x - mu) * rs) + b.x;
            r.y = g.y * ((v[k].y - mu) * rs) + b.y;
            r.z = g.z * ((v[k].z - mu) * rs) + b.z;
            r.w = g.w * ((v[k].w - mu) * rs) + b.w;
            store_raw_split(r, y, y_hi, y_lo, row * C4 + idx);
        }
    }
    if (lane == 0) {
        if (mean) mean[row] = mu;
        if (rstd) rstd[row] = rs;
    }
}

// Rows wider than 1024 floats: the whole CTA works on a row (thread i = float4 column i), two
// rows per round; the mean and then the centred sum of squares go through block reductions.
template <int R>
__global__ void __launch_bounds__(1024, 1) ln_fwd_wide_kernel(const float* __restrict__ x,
                                                              const float* __restrict__ gamma,
                                                              const float* __restrict__ beta, int64_t N, int C4,
                                                              float* y, float* y_hi, float* y_lo,
                                                              float* __restrict__ mean, float* __restrict__ rstd) {
    pdl_wait();
    pdl_trigger();
    __shared__ float red[32][R];
    __shared__ float tot[R];
    const int idx = threadIdx.x, lane = idx & 31, warp = idx >> 5, nwarps = blockDim.x >> 5;
    const bool active = idx < C4;
    const float inv_c = 1.0f / (float)(C4 * 4);
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    const float4 g = active ? ld4(gamma, idx) : zero, b = active ? ld4(beta, idx) : zero;
    // block-wide sums of R values (one per row of the round), warps combined in warp order
    auto block_sums = [&](float (&v)[R]) {
#pragma unroll
        for (int j = 0; j < R; ++j) {
            const float w = warp_sum(v[j]);
            if (lane == 0) red[warp][j] = w;
        }
        __syncthreads();
        if (idx < R) {
            float t = 0.f;
            for (int w = 0; w < nwarps; ++w) t += red[w][idx];
            tot[idx] = t;
        }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < R; ++j) v[j] = tot[j];
        __syncthreads();   // tot and red are rewritten by the next reduction
    };
    for (int64_t row0 = (int64_t)blockIdx.x * R; row0 < N; row0 += (int64_t)gridDim.x * R) {
        float4 v[R];
        float s[R];
#pragma unroll
        for (int j = 0; j < R; ++j) {
            v[j] = (row0 + j < N && active) ? ld4(x, (row0 + j) * C4 + idx) : zero;
            s[j] = (v[j].x + v[j].y) + (v[j].z + v[j].w);
        }
        block_sums(s);
        float mu[R], q[R];
#pragma unroll
        for (int j = 0; j < R; ++j) {
            mu[j] = s[j] * inv_c;
            const float a = v[j].x - mu[j], c = v[j].y - mu[j], d = v[j].z - mu[j], e = v[j].w - mu[j];
            q[j] = active ? (a * a + c * c) + (d * d + e * e) : 0.f;
        }
        block_sums(q);
#pragma unroll
        for (int j = 0; j < R; ++j) {
            const int64_t row = row0 + j;
            if (row >= N) continue;
            const float rs = 1.0f / sqrtf(q[j] * inv_c + kLnEps);
            if (active) {
                float4 r;
                r.x = g.x * ((v[j].x - mu[j]) * rs) + b.x;
                r.y = g.y * ((v[j].y - mu[j]) * rs) + b.y;
                r.z = g.z * ((v[j].z - mu[j]) * rs) + b.z;
                r.w = g.w * ((v[j].w - mu[j]) * rs) + b.w;
                store_raw_split(r, y, y_hi, y_lo, row * C4 + idx);
            }
            if (idx == 0) {
                if (mean) mean[row] = mu[j];
                if (rstd) rstd[row] = rs;
            }
        }
    }
}

cudaError_t launch_layernorm_fwd(const float* x, const float* gamma, const float* beta, int64_t N, int C, float* y,
                                 float* y_hi, float* y_lo, float* mean, float* rstd, cudaStream_t s) {
    const int C4 = C / 4;
    const int vpl = (C4 + 31) / 32;
    if (vpl > 8) {   // C > 1024: CTA per row
        if (C > 4096) return cudaErrorInvalidValue;
        constexpr int R = 2;
        const int64_t rounds = (N + R - 1) / R;
        const int wgrid = (int)(rounds < 2 * 148 ? rounds : 2 * 148);
        BT_KERNEL_LAUNCH((ln_fwd_wide_kernel<R>), wgrid, vpl * 32, 0, s, x, gamma, beta, N, C4, y, y_hi, y_lo, mean, rstd);
        BT_COUNT_LAUNCH();
        return cudaGetLastError();
    }
    const LnShape shape{(int)((N + kLnWarps - 1) / kLnWarps), kLnWarps};   // one row per warp
#define BT_LN_FWD(V)                                                                                     \
    BT_KERNEL_LAUNCH((ln_fwd_kernel<V>), shape.ctas, shape.warps * 32, 0, s, x, gamma, beta, N, C4, y, y_hi, y_lo, mean, rstd)
    if (vpl <= 1) BT_LN_FWD(1);
    else if (vpl <= 2) BT_LN_FWD(2);
    else if (vpl <= 4) BT_LN_FWD(4);
    else if (vpl <= 6) BT_LN_FWD(6);
    else if (vpl <= 8) BT_LN_FWD(8);
    else return cudaErrorInvalidValue;
#undef BT_LN_FWD
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

// ------------------------------------------------------------------ backward

static inline int ln_bwd_ctas(int64_t N) { return ln_shape(N, 2).ctas; }   // two CTAs per SM, one wave
static inline int ln_bwd_wide_ctas(int64_t N) {
    int64_t g = (N + 1) / 2;   // two rows per round, one CTA per SM
    return (int)(g < 148 ? g : 148);
}
size_t layernorm_bwd_scratch_floats(int64_t N, int C) {
    return (size_t)(C > 1024 ? ln_bwd_wide_ctas(N) : ln_bwd_ctas(N)) * 3 * C;
}

// Column accumulators (dgamma, dbeta and, with CS, the column sums of the dx written: the bias
// gradient of the linear layer whose output this dx is the gradient of) live in shared memory, one
// private array per warp, so the registers hold only the row being processed: x, dy and the
// residual gradient are all requested before anything is consumed (18 128-bit loads in flight per
// lane at C = 768), which is what keeps a two-CTA-per-SM kernel near the memory rate.
template <int VPL, bool CS>
__global__ void __launch_bounds__(kLnWarps * 32, 2) ln_bwd_kernel(
    const float* __restrict__ dy, const float* __restrict__ x, const float* __restrict__ gamma,
    const float* __restrict__ mean, const float* __restrict__ rstd, const float* dres, int64_t N, int C4,
    float* dx, float* dx_hi, float* dx_lo, float* __restrict__ partial) {
    pdl_wait();
    pdl_trigger();
    constexpr int kParts = CS ? 3 : 2;
    extern __shared__ float4 sm[];  // [kLnWarps][kParts][C4]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    float4* acc = sm + (size_t)warp * kParts * C4;
    for (int i = lane; i < kParts * C4; i += 32) acc[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    __syncwarp();
    const float inv_c = 1.0f / (float)(C4 * 4);
    for (int64_t row = (int64_t)blockIdx.x * nwarps + warp; row < N; row += (int64_t)gridDim.x * nwarps) {
        const float mu = mean[row], rs = rstd[row];
        float4 xv[VPL], dv[VPL], rv[VPL];
        float s1 = 0.f, s2 = 0.f;
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            int idx = lane + 32 * k;
            if (idx < C4) {
                xv[k] = ld4(x, row * C4 + idx);
                dv[k] = ld4(dy, row * C4 + idx);
                rv[k] = dres ? ld4(dres, row * C4 + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            int idx = lane + 32 * k;
            if (idx < C4) {
                const float4 gm = ld4(gamma, idx);
                xv[k] = make_float4((xv[k].x - mu) * rs, (xv[k].y - mu) * rs, (xv[k].z - mu) * rs, (xv[k].w - mu) * rs);
                float4 a = acc[idx];
                a.x += dv[k].x * xv[k].x; a.y += dv[k].y * xv[k].y;
                a.z += dv[k].z * xv[k].z; a.w += dv[k].w * xv[k].w;
                acc[idx] = a;
                acc[C4 + idx] = add4(acc[C4 + idx], dv[k]);
                dv[k] = make_float4(dv[k].x * gm.x, dv[k].y * gm.y, dv[k].z * gm.z, dv[k].w * gm.w);
                s1 += (dv[k].x + dv[k].y) + (dv[k].z + dv[k].w);
                s2 += (dv[k].x * xv[k].x + dv[k].y * xv[k].y) + (dv[k].z * xv[k].z + dv[k].w * xv[k].w);
            }
        }
        s1 = warp_sum(s1) * inv_c;
        s2 = warp_sum(s2) * inv_c;
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
            int idx = lane + 32 * k;
            if (idx < C4) {
                float4 r;
                r.x = rs * (dv[k].x - s1 - xv[k].x * s2);
                r.y = rs * (dv[k].y - s1 - xv[k].y * s2);
                r.z = rs * (dv[k].z - s1 - xv[k].z * s2);
                r.w = rs * (dv[k].w - s1 - xv[k].w * s2);
                r = add4(r, rv[k]);
                store_raw_split(r, dx, dx_hi, dx_lo, row * C4 + idx);
                if (CS) acc[2 * C4 + idx] = add4(acc[2 * C4 + idx], r);
            }
        }
    }
    // combine the CTA's warps in warp order and publish the CTA partial
    __syncthreads();
    float4* dst = reinterpret_cast<float4*>(partial) + (int64_t)blockIdx.x * kParts * C4;
    for (int i = threadIdx.x; i < kParts * C4; i += blockDim.x) {
        float4 t = sm[i];
        for (int w = 1; w < nwarps; ++w) t = add4(t, sm[(size_t)w * kParts * C4 + i]);
        dst[i] = t;
    }
}

// Rows wider than the register-resident kernel takes (C > 1024): the whole CTA works on a row.
// Thread i owns float4 column i (C / 4 <= 1024 threads), keeps that column's dgamma, dbeta and
// column-sum accumulators in registers, and the two row sums go through a block reduction; two
// rows are in flight per round (6 128-bit loads per thread, two barriers).  One CTA per SM, rows
// dealt to the CTAs two at a time.
constexpr int kWideRows = 2;
template <bool CS>
__global__ void __launch_bounds__(1024, 1) ln_bwd_wide_kernel(
    const float* __restrict__ dy, const float* __restrict__ x, const float* __restrict__ gamma,
    const float* __restrict__ mean, const float* __restrict__ rstd, const float* dres, int64_t N, int C4,
    float* dx, float* dx_hi, float* dx_lo, float* __restrict__ partial) {
    pdl_wait();
    pdl_trigger();
    constexpr int kParts = CS ? 3 : 2;
    constexpr int R = kWideRows;
    __shared__ float red[32][2 * R];
    __shared__ float tot[2 * R];
    const int idx = threadIdx.x, lane = idx & 31, warp = idx >> 5, nwarps = blockDim.x >> 5;
    const bool active = idx < C4;
    const float inv_c = 1.0f / (float)(C4 * 4);
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    const float4 gm = active ? ld4(gamma, idx) : zero;
    float4 a_g = zero, a_b = zero, a_c = zero;
    for (int64_t row0 = (int64_t)blockIdx.x * R; row0 < N; row0 += (int64_t)gridDim.x * R) {
        float4 xh[R], dg[R], rv[R];
        float rs[R], part[2 * R];
#pragma unroll
        for (int j = 0; j < R; ++j) {
            const int64_t row = row0 + j;
            xh[j] = dg[j] = rv[j] = zero;
            rs[j] = 0.f;
            if (row < N && active) {
                xh[j] = ld4(x, row * C4 + idx);
                dg[j] = ld4(dy, row * C4 + idx);
                if (dres) rv[j] = ld4(dres, row * C4 + idx);
            }
        }
#pragma unroll
        for (int j = 0; j < R; ++j) {
            const int64_t row = row0 + j;
            part[2 * j] = part[2 * j + 1] = 0.f;
            if (row < N) {
                const float mu = mean[row];
                rs[j] = rstd[row];
                if (active) {
                    xh[j] = make_float4((xh[j].x - mu) * rs[j], (xh[j].y - mu) * rs[j], (xh[j].z - mu) * rs[j], (xh[j].w - mu) * rs[j]);
                    a_g.x += dg[j].x * xh[j].x; a_g.y += dg[j].y * xh[j].y; a_g.z += dg[j].z * xh[j].z; a_g.w += dg[j].w * xh[j].w;
                    a_b = add4(a_b, dg[j]);
                    dg[j] = make_float4(dg[j].x * gm.x, dg[j].y * gm.y, dg[j].z * gm.z, dg[j].w * gm.w);
                    part[2 * j] = (dg[j].x + dg[j].y) + (dg[j].z + dg[j].w);
                    part[2 * j + 1] = (dg[j].x * xh[j].x + dg[j].y * xh[j].y) + (dg[j].z * xh[j].z + dg[j].w * xh[j].w);
                }
            }
        }
#pragma unroll
        for (int v = 0; v < 2 * R; ++v) {
            const float w = warp_sum(part[v]);
            if (lane == 0) red[warp][v] = w;
        }
        __syncthreads();
        if (idx < 2 * R) {   // warps are combined in warp order
            float t = 0.f;
            for (int w = 0; w < nwarps; ++w) t += red[w][idx];
            tot[idx] = t * inv_c;
        }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < R; ++j) {
            const int64_t row = row0 + j;
            if (row < N && active) {
                const float s1 = tot[2 * j], s2 = tot[2 * j + 1];
                float4 r;
                r.x = rs[j] * (dg[j].x - s1 - xh[j].x * s2);
                r.y = rs[j] * (dg[j].y - s1 - xh[j].y * s2);
                r.z = rs[j] * (dg[j].z - s1 - xh[j].z * s2);
                r.w = rs[j] * (dg[j].w - s1 - xh[j].w * s2);
                r = add4(r, rv[j]);
                store_raw_split(r, dx, dx_hi, dx_lo, row * C4 + idx);
                if (CS) a_c = add4(a_c, r);
            }
        }
    }
    if (active) {
        float4* dst = reinterpret_cast<float4*>(partial) + (int64_t)blockIdx.x * kParts * C4;
        dst[idx] = a_g;
        dst[C4 + idx] = a_b;
        if (CS) dst[2 * C4 + idx] = a_c;
    }
}

// Sums the per-CTA partials in a fixed order: lane = float4 column, warp w takes partials
// w, w+8, ... (twelve, then four loads in flight), the eight warp sums are combined in warp order.
__global__ void __launch_bounds__(256) ln_bwd_reduce_kernel(const float* __restrict__ partial, int nparts, int C4,
                                                            int kparts, float* __restrict__ dgamma,
                                                            float* __restrict__ dbeta, float* __restrict__ dcolsum) {
    pdl_wait();
    pdl_trigger();
    __shared__ float4 sm[8][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int c = blockIdx.x * 32 + lane;  // float4 column over [kparts*C4): dgamma, dbeta, column sums
    const int W = kparts * C4;
    float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
    if (c < W) {
        int p = warp;
        for (; p + 88 < nparts; p += 96) {   // twelve loads in flight: the grid is small, latency is the cost
            float4 a[12];
#pragma unroll
            for (int j = 0; j < 12; ++j) a[j] = ld4(partial, (int64_t)(p + 8 * j) * W + c);
#pragma unroll
            for (int j = 0; j < 12; ++j) t = add4(t, a[j]);
        }
        for (; p + 24 < nparts; p += 32) {
            float4 a0 = ld4(partial, (int64_t)p * W + c), a1 = ld4(partial, (int64_t)(p + 8) * W + c);
            float4 a2 = ld4(partial, (int64_t)(p + 16) * W + c), a3 = ld4(partial, (int64_t)(p + 24) * W + c);
            t = add4(add4(add4(add4(t, a0), a1), a2), a3);
        }
        for (; p < nparts; p += 8) t = add4(t, ld4(partial, (int64_t)p * W + c));
    }
    sm[warp][lane] = t;
    __syncthreads();
    if (warp == 0 && c < W) {
        float4 r = sm[0][lane];
#pragma unroll
        for (int w = 1; w < 8; ++w) r = add4(r, sm[w][lane]);
        if (c < C4) reinterpret_cast<float4*>(dgamma)[c] = r;
        else if (c < 2 * C4) reinterpret_cast<float4*>(dbeta)[c - C4] = r;
        else reinterpret_cast<float4*>(dcolsum)[c - 2 * C4] = r;
    }
}

template <int V>
static cudaError_t ln_bwd_set_smem_limit() {
    constexpr int kMax = 160 * 1024;
    cudaError_t e = cudaFuncSetAttribute(ln_bwd_kernel<V, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMax);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(ln_bwd_kernel<V, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMax);
    return e;
}
static cudaError_t ln_bwd_set_smem_limits() {
    cudaError_t e = ln_bwd_set_smem_limit<1>();
    if (e == cudaSuccess) e = ln_bwd_set_smem_limit<2>();
    if (e == cudaSuccess) e = ln_bwd_set_smem_limit<4>();
    if (e == cudaSuccess) e = ln_bwd_set_smem_limit<6>();
    if (e == cudaSuccess) e = ln_bwd_set_smem_limit<8>();
    return e;
}

cudaError_t launch_layernorm_bwd(const float* dy, const float* x, const float* gamma, const float* mean,
                                 const float* rstd, const float* dres, int64_t N, int C, float* dx, float* dx_hi,
                                 float* dx_lo, float* dgamma, float* dbeta, float* dx_colsum, float* scratch,
                                 cudaStream_t s) {
    const int C4 = C / 4;
    const int vpl = (C4 + 31) / 32;
    if (vpl > 8) {   // C > 1024: the two-pass kernel
        if (C > 4096) return cudaErrorInvalidValue;
        const int kparts = dx_colsum ? 3 : 2;
        const int wgrid = ln_bwd_wide_ctas(N);
        const int wblock = ((C4 + 31) / 32) * 32;
        if (dx_colsum)
            BT_KERNEL_LAUNCH((ln_bwd_wide_kernel<true>), wgrid, wblock, 0, s, dy, x, gamma, mean, rstd, dres, N, C4, dx, dx_hi, dx_lo, scratch);
        else
            BT_KERNEL_LAUNCH((ln_bwd_wide_kernel<false>), wgrid, wblock, 0, s, dy, x, gamma, mean, rstd, dres, N, C4, dx, dx_hi, dx_lo, scratch);
        BT_COUNT_LAUNCH();
        BT_KERNEL_LAUNCH((ln_bwd_reduce_kernel), (kparts * C4 + 31) / 32, 256, 0, s, scratch, wgrid, C4, kparts, dgamma, dbeta, dx_colsum);
        BT_COUNT_LAUNCH();
        return cudaGetLastError();
    }
    const LnShape shape = ln_shape(N, 2);
    const int grid = shape.ctas;
    const size_t smem = (size_t)shape.warps * (dx_colsum ? 3 : 2) * C4 * sizeof(float4);   // 72 KB at C = 768, 8 warps, with sums
    static const cudaError_t attr = ln_bwd_set_smem_limits();
    if (attr != cudaSuccess) return attr;
#define BT_LN_BWD(V)                                                                                          \
    do {                                                                                                      \
        if (dx_colsum)                                                                                        \
            BT_KERNEL_LAUNCH((ln_bwd_kernel<V, true>), grid, shape.warps * 32, smem, s, dy, x, gamma, mean, rstd, dres, N, C4, dx, \
                                                                     dx_hi, dx_lo, scratch);                  \
        else                                                                                                  \
            BT_KERNEL_LAUNCH((ln_bwd_kernel<V, false>), grid, shape.warps * 32, smem, s, dy, x, gamma, mean, rstd, dres, N, C4, dx, \
                                                                      dx_hi, dx_lo, scratch);                 \
    } while (0)
    if (vpl <= 1) BT_LN_BWD(1);
    else if (vpl <= 2) BT_LN_BWD(2);
    else if (vpl <= 4) BT_LN_BWD(4);
    else if (vpl <= 6) BT_LN_BWD(6);
    else if (vpl <= 8) BT_LN_BWD(8);
    else return cudaErrorInvalidValue;
#undef BT_LN_BWD
    BT_COUNT_LAUNCH();
    const int kparts = dx_colsum ? 3 : 2;
    BT_KERNEL_LAUNCH((ln_bwd_reduce_kernel), (kparts * C4 + 31) / 32, 256, 0, s, scratch, grid, C4, kparts, dgamma, dbeta, dx_colsum);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

}  // namespace bt
