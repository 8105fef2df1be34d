// Causal flash attention, forward and backward, FP32 fidelity on the tensor cores.
//
// Every product (Q K^T, P V, dO V^T, dS K, dS^T Q, P^T dO) is a warp-level m16n8k8 TF32
// tensor-core MMA evaluated three times on hi/lo splits (a_lo*b_hi + a_hi*b_lo + a_hi*b_hi,
// FP32 accumulate).  The streamed tiles (K/V in the forward and dq kernels, Q/dO in the dkv kernel)
// are copied raw into double-buffered shared memory with cp.async while the previous tile is
// being consumed (row stride head_dim + 4 floats: both fragment access patterns are bank-conflict
// free); their fragments are split into hi/lo in registers, as are the per-warp operands.  The softmax is the online (running max / running
// sum) form in base 2 with the 1/sqrt(d) log2(e) factor folded into Q; row reductions are
// warp shuffles inside the 4-lane quad that owns a row.
//
// Forward:  one CTA = 64 query rows of one (sequence, head); 4 warps x 16 rows; KV tiles of 64
//           up to the diagonal; heaviest (last) query tiles are scheduled first.
// Backward: two deterministic kernels that recompute P from (q, k, lse):
//           dq  kernel: same decomposition as the forward (warp owns 16 query rows);
//           dkv kernel: CTA owns 128 keys (8 warps x 16), loops over the query tiles at or
//                       below the diagonal; no atomics, no cross-CTA accumulation.
#include "common.cuh"

namespace bt {

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ void mma_tf32(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// d += a * b with a = a_hi + a_lo, b = b_hi + b_lo (lo*lo dropped), small terms first.
__device__ __forceinline__ void mma3(float (&d)[4], const uint32_t (&a_hi)[4], const uint32_t (&a_lo)[4],
                                     uint32_t bh0, uint32_t bh1, uint32_t bl0, uint32_t bl1) {
    mma_tf32(d, a_lo, bh0, bh1);
    mma_tf32(d, a_hi, bl0, bl1);
    mma_tf32(d, a_hi, bh0, bh1);
}
__device__ __forceinline__ void split_u(float x, uint32_t& hi, uint32_t& lo) {
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(hi) : "f"(x));  // nearest TF32 value (see split_tf32)
    lo = __float_as_uint(x - __uint_as_float(hi));
}

// Stages ROWS rows x HD floats (global row stride `gstride`, rows >= nvalid read as zero),
// multiplied by `mul`, into hi/lo shared tiles with row stride HD + 4.
template <int HD, int ROWS, int NT>
__device__ __forceinline__ void stage_split(const float* __restrict__ src, int64_t gstride, int row0, int nvalid,
                                            float mul, float* __restrict__ s_hi, float* __restrict__ s_lo) {
    constexpr int LDS = HD + 4, V4 = HD / 4;
    for (int idx = threadIdx.x; idx < ROWS * V4; idx += NT) {
        const int r = idx / V4, c4 = idx - r * V4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (row0 + r < nvalid) v = *reinterpret_cast<const float4*>(src + (int64_t)(row0 + r) * gstride + c4 * 4);
        v.x *= mul; v.y *= mul; v.z *= mul; v.w *= mul;
        float4 h, l;
        split_tf32(v, h, l);
        *reinterpret_cast<float4*>(s_hi + r * LDS + c4 * 4) = h;
        *reinterpret_cast<float4*>(s_lo + r * LDS + c4 * 4) = l;
    }
}

// Asynchronously copies ROWS rows x HD floats (global row stride `gstride`; rows past the end are
// clamped to the last valid row, their results are masked or never stored) into a raw FP32
// shared tile with row stride HD + 4.  One cp.async group per call.
template <int HD, int ROWS, int NT>
__device__ __forceinline__ void stage_raw_async(const float* __restrict__ src, int64_t gstride, int row0, int nvalid,
                                                float* __restrict__ dst) {
    constexpr int LDS = HD + 4, V4 = HD / 4;
    for (int idx = threadIdx.x; idx < ROWS * V4; idx += NT) {
        const int r = idx / V4, c4 = idx - r * V4;
        const int gr = min(row0 + r, nvalid - 1);
        const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst + r * LDS + c4 * 4);
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(src + (int64_t)gr * gstride + c4 * 4)
                     : "memory");
    }
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// A fragment (16 rows x 8 k) of a shared hi/lo tile: rows row16 + g (+8), columns k0 + t4 (+4).
template <int LDS>
__device__ __forceinline__ void load_a_frag(const float* s_hi, const float* s_lo, int row16, int k0, int g, int t4,
                                            uint32_t (&a_hi)[4], uint32_t (&a_lo)[4]) {
    const int o0 = (row16 + g) * LDS + k0 + t4, o1 = o0 + 8 * LDS;
    a_hi[0] = __float_as_uint(s_hi[o0]);     a_lo[0] = __float_as_uint(s_lo[o0]);
    a_hi[1] = __float_as_uint(s_hi[o1]);     a_lo[1] = __float_as_uint(s_lo[o1]);
    a_hi[2] = __float_as_uint(s_hi[o0 + 4]); a_lo[2] = __float_as_uint(s_lo[o0 + 4]);
    a_hi[3] = __float_as_uint(s_hi[o1 + 4]); a_lo[3] = __float_as_uint(s_lo[o1 + 4]);
}

// acc[nt] (16 x 8 tiles over the 64 tile rows) += A(16 x 8 k-slice ks) . X^T, X a RAW shared tile
// [64][HD]: B fragment element (k, n) = X[n0 + n][k0 + k], split into hi/lo in registers.  The
// three TF32 terms are issued term-major so that consecutive MMAs hit different accumulators.
template <int HD>
__device__ __forceinline__ void mma_a_xT(float (&acc)[8][4], const uint32_t (&a_hi)[4], const uint32_t (&a_lo)[4],
                                         const float* x, int ks, int g, int t4) {
    constexpr int LDS = HD + 4;
    uint32_t bh0[8], bh1[8], bl0[8], bl1[8];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
        const int o = (nt * 8 + g) * LDS + ks * 8 + t4;
        split_u(x[o], bh0[nt], bl0[nt]);
        split_u(x[o + 4], bh1[nt], bl1[nt]);
    }
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) mma_tf32(acc[nt], a_lo, bh0[nt], bh1[nt]);
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) mma_tf32(acc[nt], a_hi, bl0[nt], bl1[nt]);
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) mma_tf32(acc[nt], a_hi, bh0[nt], bh1[nt]);
}

// acc[dt] (16 x 8 tiles over HD) += P(16 x 8 slice nt of a 16 x 64 C-layout tile) . X, X a RAW
// shared tile [64][HD].  The C-fragment columns 2*t4, 2*t4+1 serve as the A-fragment k indices
// t4, t4+4, so B fragment element (k = t4 | t4+4, n) = X[nt*8 + 2*t4 | 2*t4+1][n0 + n].
template <int HD>
__device__ __forceinline__ void mma_p_x(float (&acc)[HD / 8][4], const float (&p)[4], const float* x, int nt, int g,
                                        int t4) {
    constexpr int LDS = HD + 4, KS = HD / 8;
    uint32_t a_hi[4], a_lo[4];
    split_u(p[0], a_hi[0], a_lo[0]);
    split_u(p[2], a_hi[1], a_lo[1]);
    split_u(p[1], a_hi[2], a_lo[2]);
    split_u(p[3], a_hi[3], a_lo[3]);
    uint32_t bh0[KS], bh1[KS], bl0[KS], bl1[KS];
#pragma unroll
    for (int dt = 0; dt < KS; ++dt) {
        const int o = (nt * 8 + 2 * t4) * LDS + dt * 8 + g;
        split_u(x[o], bh0[dt], bl0[dt]);
        split_u(x[o + LDS], bh1[dt], bl1[dt]);
    }
#pragma unroll
    for (int dt = 0; dt < KS; ++dt) mma_tf32(acc[dt], a_lo, bh0[dt], bh1[dt]);
#pragma unroll
    for (int dt = 0; dt < KS; ++dt) mma_tf32(acc[dt], a_hi, bl0[dt], bl1[dt]);
#pragma unroll
    for (int dt = 0; dt < KS; ++dt) mma_tf32(acc[dt], a_hi, bh0[dt], bh1[dt]);
}

__device__ __forceinline__ float quad_max(float v) {
    v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 1));
    return fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 2));
}
__device__ __forceinline__ float quad_sum(float v) {
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    return v + __shfl_xor_sync(0xffffffffu, v, 2);
}

// Q rows of one warp as pre-split A fragments, multiplied by `mul`.
template <int HD>
__device__ __forceinline__ void load_q_frags(const float* __restrict__ base, int64_t gstride, int r0, int r1, int T,
                                             float mul, int t4, uint32_t (&q_hi)[HD / 8][4],
                                             uint32_t (&q_lo)[HD / 8][4]) {
    const float* p0 = base + (int64_t)min(r0, T - 1) * gstride;
    const float* p1 = base + (int64_t)min(r1, T - 1) * gstride;
#pragma unroll
    for (int ks = 0; ks < HD / 8; ++ks) {
        split_u(p0[ks * 8 + t4] * mul, q_hi[ks][0], q_lo[ks][0]);
        split_u(p1[ks * 8 + t4] * mul, q_hi[ks][1], q_lo[ks][1]);
        split_u(p0[ks * 8 + t4 + 4] * mul, q_hi[ks][2], q_lo[ks][2]);
        split_u(p1[ks * 8 + t4 + 4] * mul, q_hi[ks][3], q_lo[ks][3]);
    }
}

// ------------------------------------------------------------------ forward

template <int HD>
__global__ void __launch_bounds__(128, 2) attn_fwd_mma_kernel(const float* __restrict__ qkv, int T, int C, int H,
                                                              float* o, float* o_hi, float* o_lo,
                                                              float* __restrict__ lse) {
    constexpr int LDS = HD + 4, KS = HD / 8, TILE = 64 * LDS;
    extern __shared__ float sm[];  // K[2], V[2] raw tiles (double buffered)
    const int qt = gridDim.x - 1 - blockIdx.x;
    const int b = blockIdx.y / H, h = blockIdx.y % H;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t4 = lane & 3;
    const int64_t gs = 3 * (int64_t)C;
    const float* base = qkv + (int64_t)b * T * gs + h * HD;
    const int r0 = qt * 64 + warp * 16 + g, r1 = r0 + 8;
    const float qmul = kLog2e / sqrtf((float)HD);

    stage_raw_async<HD, 64, 128>(base + C, gs, 0, T, sm);
    stage_raw_async<HD, 64, 128>(base + 2 * C, gs, 0, T, sm + 2 * TILE);
    cp_async_commit();

    uint32_t q_hi[KS][4], q_lo[KS][4];
    load_q_frags<HD>(base, gs, r0, r1, T, qmul, t4, q_hi, q_lo);

    float acc[KS][4];
#pragma unroll
    for (int dt = 0; dt < KS; ++dt) acc[dt][0] = acc[dt][1] = acc[dt][2] = acc[dt][3] = 0.f;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

    for (int kt = 0; kt <= qt; ++kt) {
        const int buf = kt & 1;
        if (kt < qt) {  // prefetch the next tile into the other buffer
            stage_raw_async<HD, 64, 128>(base + C, gs, (kt + 1) * 64, T, sm + (buf ^ 1) * TILE);
            stage_raw_async<HD, 64, 128>(base + 2 * C, gs, (kt + 1) * 64, T, sm + (2 + (buf ^ 1)) * TILE);
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        const float* k_s = sm + buf * TILE;
        const float* v_s = sm + (2 + buf) * TILE;
        float s[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) mma_a_xT<HD>(s, q_hi[ks], q_lo[ks], k_s, ks, g, t4);
        if (kt == qt) {
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                const int col = kt * 64 + nt * 8 + 2 * t4;
                if (col > r0) s[nt][0] = -INFINITY;
                if (col + 1 > r0) s[nt][1] = -INFINITY;
                if (col > r1) s[nt][2] = -INFINITY;
                if (col + 1 > r1) s[nt][3] = -INFINITY;
            }
        }
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            mx0 = fmaxf(mx0, fmaxf(s[nt][0], s[nt][1]));
            mx1 = fmaxf(mx1, fmaxf(s[nt][2], s[nt][3]));
        }
        const float mn0 = fmaxf(m0, quad_max(mx0)), mn1 = fmaxf(m1, quad_max(mx1));
        const float c0 = exp2f(m0 - mn0), c1 = exp2f(m1 - mn1);
        m0 = mn0; m1 = mn1;
        l0 *= c0; l1 *= c1;
#pragma unroll
        for (int dt = 0; dt < KS; ++dt) {
            acc[dt][0] *= c0; acc[dt][1] *= c0; acc[dt][2] *= c1; acc[dt][3] *= c1;
        }
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            float p[4];
            p[0] = exp2f(s[nt][0] - mn0); p[1] = exp2f(s[nt][1] - mn0);
            p[2] = exp2f(s[nt][2] - mn1); p[3] = exp2f(s[nt][3] - mn1);
            l0 += p[0] + p[1];
            l1 += p[2] + p[3];
            mma_p_x<HD>(acc, p, v_s, nt, g, t4);
        }
        __syncthreads();  // everyone is done with this buffer before it is refilled
    }
    l0 = quad_sum(l0);
    l1 = quad_sum(l1);
    const float i0 = 1.0f / l0, i1 = 1.0f / l1;
    const int64_t ob = ((int64_t)b * T) * C + h * HD;
#pragma unroll
    for (int dt = 0; dt < KS; ++dt) {
        const int col = dt * 8 + 2 * t4;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int r = half ? r1 : r0;
            if (r >= T) continue;
            const float inv = half ? i1 : i0;
            float2 v = make_float2(acc[dt][2 * half] * inv, acc[dt][2 * half + 1] * inv);
            const int64_t off = ob + (int64_t)r * C + col;
            if (o) *reinterpret_cast<float2*>(o + off) = v;
            if (o_hi) {
                float2 hh, ll;
                split_tf32(v.x, hh.x, ll.x);
                split_tf32(v.y, hh.y, ll.y);
                *reinterpret_cast<float2*>(o_hi + off) = hh;
                *reinterpret_cast<float2*>(o_lo + off) = ll;
            }
        }
    }
    if (t4 == 0 && lse) {
        const int64_t lb = ((int64_t)b * H + h) * T;
        if (r0 < T) lse[lb + r0] = (m0 + log2f(l0)) * kLn2;
        if (r1 < T) lse[lb + r1] = (m1 + log2f(l1)) * kLn2;
    }
}

// ------------------------------------------------------------------ backward: dq

template <int HD>
__global__ void __launch_bounds__(128, 2) attn_bwd_dq_mma_kernel(const float* __restrict__ qkv,
                                                                 const float* __restrict__ lse,
                                                                 const float* __restrict__ d_o,
                                                                 const float* __restrict__ dvec, int T, int C, int H,
                                                                 float* dqkv, float* dqkv_hi, float* dqkv_lo) {
    constexpr int LDS = HD + 4, KS = HD / 8, TILE = 64 * LDS;
    extern __shared__ float sm[];  // K[2], V[2] raw (double buffered), dO hi, dO lo
    float *do_hi = sm + 4 * TILE, *do_lo = sm + 5 * TILE;
    const int qt = gridDim.x - 1 - blockIdx.x;
    const int b = blockIdx.y / H, h = blockIdx.y % H;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t4 = lane & 3;
    const int64_t gs = 3 * (int64_t)C;
    const float* base = qkv + (int64_t)b * T * gs + h * HD;
    const int r0 = qt * 64 + warp * 16 + g, r1 = r0 + 8;
    const float scale = 1.0f / sqrtf((float)HD);

    stage_raw_async<HD, 64, 128>(base + C, gs, 0, T, sm);
    stage_raw_async<HD, 64, 128>(base + 2 * C, gs, 0, T, sm + 2 * TILE);
    cp_async_commit();

    uint32_t q_hi[KS][4], q_lo[KS][4];
    load_q_frags<HD>(base, gs, r0, r1, T, scale * kLog2e, t4, q_hi, q_lo);
    stage_split<HD, 64, 128>(d_o + (int64_t)b * T * C + h * HD, C, qt * 64, T, 1.0f, do_hi, do_lo);
    const int64_t lb = ((int64_t)b * H + h) * T;
    const float L0 = lse[lb + min(r0, T - 1)] * kLog2e, L1 = lse[lb + min(r1, T - 1)] * kLog2e;
    const float D0 = dvec[lb + min(r0, T - 1)], D1 = dvec[lb + min(r1, T - 1)];

    float dq[KS][4];
#pragma unroll
    for (int dt = 0; dt < KS; ++dt) dq[dt][0] = dq[dt][1] = dq[dt][2] = dq[dt][3] = 0.f;

    for (int kt = 0; kt <= qt; ++kt) {
        const int buf = kt & 1;
        if (kt < qt) {
            stage_raw_async<HD, 64, 128>(base + C, gs, (kt + 1) * 64, T, sm + (buf ^ 1) * TILE);
            stage_raw_async<HD, 64, 128>(base + 2 * C, gs, (kt + 1) * 64, T, sm + (2 + (buf ^ 1)) * TILE);
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        const float* k_s = sm + buf * TILE;
        const float* v_s = sm + (2 + buf) * TILE;
        float s[8][4], dp[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
            dp[nt][0] = dp[nt][1] = dp[nt][2] = dp[nt][3] = 0.f;
        }
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            mma_a_xT<HD>(s, q_hi[ks], q_lo[ks], k_s, ks, g, t4);
            uint32_t a_hi[4], a_lo[4];
            load_a_frag<LDS>(do_hi, do_lo, warp * 16, ks * 8, g, t4, a_hi, a_lo);
            mma_a_xT<HD>(dp, a_hi, a_lo, v_s, ks, g, t4);
        }
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const int col = kt * 64 + nt * 8 + 2 * t4;
            float p[4];
            p[0] = (col > r0) ? 0.f : exp2f(s[nt][0] - L0);
            p[1] = (col + 1 > r0) ? 0.f : exp2f(s[nt][1] - L0);
            p[2] = (col > r1) ? 0.f : exp2f(s[nt][2] - L1);
            p[3] = (col + 1 > r1) ? 0.f : exp2f(s[nt][3] - L1);
            float ds[4];
            ds[0] = p[0] * (dp[nt][0] - D0);
            ds[1] = p[1] * (dp[nt][1] - D0);
            ds[2] = p[2] * (dp[nt][2] - D1);
            ds[3] = p[3] * (dp[nt][3] - D1);
            mma_p_x<HD>(dq, ds, k_s, nt, g, t4);
        }
        __syncthreads();
    }
    const int64_t ob = ((int64_t)b * T) * gs + h * HD;
#pragma unroll
    for (int dt = 0; dt < KS; ++dt) {
        const int col = dt * 8 + 2 * t4;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int r = half ? r1 : r0;
            if (r >= T) continue;
            float2 v = make_float2(dq[dt][2 * half] * scale, dq[dt][2 * half + 1] * scale);
            const int64_t off = ob + (int64_t)r * gs + col;
            if (dqkv) *reinterpret_cast<float2*>(dqkv + off) = v;
            if (dqkv_hi) {
                float2 hh, ll;
                split_tf32(v.x, hh.x, ll.x);
                split_tf32(v.y, hh.y, ll.y);
                *reinterpret_cast<float2*>(dqkv_hi + off) = hh;
                *reinterpret_cast<float2*>(dqkv_lo + off) = ll;
            }
        }
    }
}

// ------------------------------------------------------------------ backward: dk, dv

template <int HD>
__global__ void __launch_bounds__(256) attn_bwd_dkv_mma_kernel(const float* __restrict__ qkv,
                                                               const float* __restrict__ lse,
                                                               const float* __restrict__ d_o,
                                                               const float* __restrict__ dvec, int T, int C, int H,
                                                               float* dqkv, float* dqkv_hi, float* dqkv_lo) {
    constexpr int LDS = HD + 4, KS = HD / 8, KT = 128 * LDS, QT = 64 * LDS;
    extern __shared__ float sm[];
    // K', V of this CTA's 128 keys as hi/lo (A operands); Q[2], dO[2] raw query tiles (double
    // buffered B operands); lse[2][64], D[2][64].
    float *k_hi = sm, *k_lo = sm + KT, *v_hi = sm + 2 * KT, *v_lo = sm + 3 * KT;
    float *q_raw = sm + 4 * KT, *do_raw = q_raw + 2 * QT;
    float *lse_s = q_raw + 4 * QT, *d_s = lse_s + 128;
    const int j0 = blockIdx.x * 128;
    const int b = blockIdx.y / H, h = blockIdx.y % H;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t4 = lane & 3;
    const int64_t gs = 3 * (int64_t)C;
    const float* base = qkv + (int64_t)b * T * gs + h * HD;
    const float* dob = d_o + (int64_t)b * T * C + h * HD;
    const int64_t lb = ((int64_t)b * H + h) * T;
    const float scale = 1.0f / sqrtf((float)HD);
    const int jw = j0 + warp * 16;             // first key of this warp
    const int jr0 = jw + g, jr1 = jr0 + 8;     // the two key rows of this thread
    const int n_qt = (T + 63) / 64, qt0 = j0 / 64;

    stage_raw_async<HD, 64, 256>(base, gs, qt0 * 64, T, q_raw);
    stage_raw_async<HD, 64, 256>(dob, C, qt0 * 64, T, do_raw);
    cp_async_commit();
    // K is staged pre-multiplied by scale*log2(e) (it only feeds the score recomputation)
    stage_split<HD, 128, 256>(base + C, gs, j0, T, scale * kLog2e, k_hi, k_lo);
    stage_split<HD, 128, 256>(base + 2 * C, gs, j0, T, 1.0f, v_hi, v_lo);

    float dk[KS][4], dv[KS][4];
#pragma unroll
    for (int dt = 0; dt < KS; ++dt) {
        dk[dt][0] = dk[dt][1] = dk[dt][2] = dk[dt][3] = 0.f;
        dv[dt][0] = dv[dt][1] = dv[dt][2] = dv[dt][3] = 0.f;
    }
    for (int qt = qt0; qt < n_qt; ++qt) {
        const int q0 = qt * 64, buf = (qt - qt0) & 1;
        if (threadIdx.x < 64) {
            const int r = q0 + threadIdx.x;
            lse_s[buf * 64 + threadIdx.x] = (r < T) ? lse[lb + r] * kLog2e : INFINITY;
            d_s[buf * 64 + threadIdx.x] = (r < T) ? dvec[lb + r] : 0.f;
        }
        if (qt + 1 < n_qt) {
            stage_raw_async<HD, 64, 256>(base, gs, q0 + 64, T, q_raw + (buf ^ 1) * QT);
            stage_raw_async<HD, 64, 256>(dob, C, q0 + 64, T, do_raw + (buf ^ 1) * QT);
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        if (q0 + 63 >= jw) {  // otherwise every query row of this tile precedes this warp's keys
            const float* q_s = q_raw + buf * QT;
            const float* do_s = do_raw + buf * QT;
            float s[8][4], dp[8][4];
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
                dp[nt][0] = dp[nt][1] = dp[nt][2] = dp[nt][3] = 0.f;
            }
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                uint32_t a_hi[4], a_lo[4];
                load_a_frag<LDS>(k_hi, k_lo, warp * 16, ks * 8, g, t4, a_hi, a_lo);
                mma_a_xT<HD>(s, a_hi, a_lo, q_s, ks, g, t4);       // S^T = K Q^T
                load_a_frag<LDS>(v_hi, v_lo, warp * 16, ks * 8, g, t4, a_hi, a_lo);
                mma_a_xT<HD>(dp, a_hi, a_lo, do_s, ks, g, t4);     // dP^T = V dO^T
            }
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                const int ci = nt * 8 + 2 * t4;      // query row (column of S^T) inside the tile
                const int i = q0 + ci;
                const float La = lse_s[buf * 64 + ci], Lb = lse_s[buf * 64 + ci + 1];
                const float Da = d_s[buf * 64 + ci], Db = d_s[buf * 64 + ci + 1];
                float p[4];
                p[0] = (i < jr0) ? 0.f : exp2f(s[nt][0] - La);
                p[1] = (i + 1 < jr0) ? 0.f : exp2f(s[nt][1] - Lb);
                p[2] = (i < jr1) ? 0.f : exp2f(s[nt][2] - La);
                p[3] = (i + 1 < jr1) ? 0.f : exp2f(s[nt][3] - Lb);
                mma_p_x<HD>(dv, p, do_s, nt, g, t4);               // dV += P^T dO
                float ds[4];
                ds[0] = p[0] * (dp[nt][0] - Da);
                ds[1] = p[1] * (dp[nt][1] - Db);
                ds[2] = p[2] * (dp[nt][2] - Da);
                ds[3] = p[3] * (dp[nt][3] - Db);
                mma_p_x<HD>(dk, ds, q_s, nt, g, t4);               // dK += dS^T Q
            }
        }
        __syncthreads();
    }
    const int64_t ob = ((int64_t)b * T) * gs + h * HD;
#pragma unroll
    for (int dt = 0; dt < KS; ++dt) {
        const int col = dt * 8 + 2 * t4;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int r = half ? jr1 : jr0;
            if (r >= T) continue;
            float2 kk = make_float2(dk[dt][2 * half] * scale, dk[dt][2 * half + 1] * scale);
            float2 vv = make_float2(dv[dt][2 * half], dv[dt][2 * half + 1]);
            const int64_t off = ob + (int64_t)r * gs + col;
            if (dqkv) {
                *reinterpret_cast<float2*>(dqkv + off + C) = kk;
                *reinterpret_cast<float2*>(dqkv + off + 2 * C) = vv;
            }
            if (dqkv_hi) {
                float2 hh, ll;
                split_tf32(kk.x, hh.x, ll.x);
                split_tf32(kk.y, hh.y, ll.y);
                *reinterpret_cast<float2*>(dqkv_hi + off + C) = hh;
                *reinterpret_cast<float2*>(dqkv_lo + off + C) = ll;
                split_tf32(vv.x, hh.x, ll.x);
                split_tf32(vv.y, hh.y, ll.y);
                *reinterpret_cast<float2*>(dqkv_hi + off + 2 * C) = hh;
                *reinterpret_cast<float2*>(dqkv_lo + off + 2 * C) = ll;
            }
        }
    }
}

template <int HD>
constexpr size_t fwd_smem() { return (size_t)4 * 64 * (HD + 4) * sizeof(float); }
template <int HD>
constexpr size_t dq_smem() { return (size_t)6 * 64 * (HD + 4) * sizeof(float); }
template <int HD>
constexpr size_t dkv_smem() { return ((size_t)4 * 128 * (HD + 4) + 4 * 64 * (HD + 4) + 256) * sizeof(float); }

template <int HD>
cudaError_t set_attrs() {
    cudaError_t e = cudaFuncSetAttribute(attn_fwd_mma_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)fwd_smem<HD>());
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(attn_bwd_dq_mma_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)dq_smem<HD>());
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(attn_bwd_dkv_mma_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)dkv_smem<HD>());
    return e;
}
cudaError_t ensure_attrs() {
    static cudaError_t st = []() {
        cudaError_t e = set_attrs<16>();
        if (e == cudaSuccess) e = set_attrs<32>();
        if (e == cudaSuccess) e = set_attrs<64>();
        return e;
    }();
    return st;
}

}  // namespace

bool attention_mma_supports(int head_dim) { return head_dim == 16 || head_dim == 32 || head_dim == 64; }

cudaError_t launch_attention_fwd_mma(const float* qkv, int B, int T, int C, int H, float* o, float* o_hi,
                                     float* o_lo, float* lse, cudaStream_t s) {
    cudaError_t e = ensure_attrs();
    if (e != cudaSuccess) return e;
    const int d = C / H;
    dim3 grid((T + 63) / 64, B * H);
#define BT_FWD(HDV) attn_fwd_mma_kernel<HDV><<<grid, 128, fwd_smem<HDV>(), s>>>(qkv, T, C, H, o, o_hi, o_lo, lse)
    if (d == 16) BT_FWD(16);
    else if (d == 32) BT_FWD(32);
    else BT_FWD(64);
#undef BT_FWD
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

cudaError_t launch_attention_bwd_mma(const float* qkv, const float* lse, const float* d_o, const float* dvec, int B,
                                     int T, int C, int H, float* dqkv, float* dqkv_hi, float* dqkv_lo,
                                     cudaStream_t s) {
    cudaError_t e = ensure_attrs();
    if (e != cudaSuccess) return e;
    const int d = C / H;
    dim3 gq((T + 63) / 64, B * H), gk((T + 127) / 128, B * H);
#define BT_BWD(HDV)                                                                                                \
    attn_bwd_dq_mma_kernel<HDV><<<gq, 128, dq_smem<HDV>(), s>>>(qkv, lse, d_o, dvec, T, C, H, dqkv, dqkv_hi, dqkv_lo); \
    attn_bwd_dkv_mma_kernel<HDV><<<gk, 256, dkv_smem<HDV>(), s>>>(qkv, lse, d_o, dvec, T, C, H, dqkv, dqkv_hi, dqkv_lo)
    if (d == 16) { BT_BWD(16); } else if (d == 32) { BT_BWD(32); } else { BT_BWD(64); }
#undef BT_BWD
    BT_COUNT_LAUNCH();
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

}  // namespace bt
