// Plain FP32 FMA GEMM used as the bring-up reference for the tcgen05 kernel (selected with
// BT_FLAG_GEMM_SIMT).  64x64 output tile, 16-deep K slices staged through shared memory, a
// 4x4 micro-tile per thread.  Operands arrive as TF32 hi/lo planes and are re-joined exactly
// (hi + lo) while being staged, so this kernel computes the same FP32 product the tensor-core
// kernel approximates with three TF32 products.
#include "common.cuh"

namespace bt {

constexpr int kSimtTile = 64, kSimtK = 16;

template <int LAYOUT>
__global__ void __launch_bounds__(256) gemm_simt_kernel(int M, int N, int K, const float* __restrict__ a_hi,
                                                        const float* __restrict__ a_lo, int64_t lda,
                                                        const float* __restrict__ b_hi,
                                                        const float* __restrict__ b_lo, int64_t ldb,
                                                        float* __restrict__ D, int64_t ldd,
                                                        const float* __restrict__ bias,
                                                        const float* __restrict__ residual) {
    __shared__ float As[kSimtK][kSimtTile + 4];
    __shared__ float Bs[kSimtK][kSimtTile + 4];
    const int m0 = blockIdx.y * kSimtTile, n0 = blockIdx.x * kSimtTile;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += kSimtK) {
        // stage: 64 x 16 elements of each operand, 4 per thread
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int e = threadIdx.x + 256 * i;
            int mm, kk;
            if (LAYOUT == kTN) { mm = e & 63; kk = e >> 6; } else { kk = e & 15; mm = e >> 4; }
            int gm = m0 + mm, gk = k0 + kk;
            float v = 0.f;
            if (gm < M && gk < K) {
                int64_t off = (LAYOUT == kTN) ? (int64_t)gk * lda + gm : (int64_t)gm * lda + gk;
                v = a_hi[off];
                if (a_lo) v += a_lo[off];
            }
            As[kk][mm] = v;
            int nn;
            if (LAYOUT == kNT) { kk = e & 15; nn = e >> 4; } else { nn = e & 63; kk = e >> 6; }
            int gn = n0 + nn;
            gk = k0 + kk;
            v = 0.f;
            if (gn < N && gk < K) {
                int64_t off = (LAYOUT == kNT) ? (int64_t)gn * ldb + gk : (int64_t)gk * ldb + gn;
                v = b_hi[off];
                if (b_lo) v += b_lo[off];
            }
            Bs[kk][nn] = v;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kSimtK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int gm = m0 + ty * 4 + i;
        if (gm >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int gn = n0 + tx * 4 + j;
            if (gn >= N) continue;
            float v = acc[i][j];
            if (bias) v += bias[gn];
            if (residual) v += residual[(int64_t)gm * ldd + gn];
            D[(int64_t)gm * ldd + gn] = v;
        }
    }
}

cudaError_t launch_gemm_simt(int layout, int64_t M, int64_t N, int64_t K, SplitMat A, SplitMat B, float* D,
                             int64_t ldd, const float* bias, const float* residual, cudaStream_t s) {
    dim3 grid((unsigned)((N + kSimtTile - 1) / kSimtTile), (unsigned)((M + kSimtTile - 1) / kSimtTile));
    const float* a_lo = A.plane ? A.hi + A.plane : nullptr;
    const float* b_lo = B.plane ? B.hi + B.plane : nullptr;
#define BT_SIMT(L)                                                                                           \
    gemm_simt_kernel<L><<<grid, 256, 0, s>>>((int)M, (int)N, (int)K, A.hi, a_lo, A.ld, B.hi, b_lo, B.ld, D, ldd, \
                                             bias, residual)
    if (layout == kNT) BT_SIMT(kNT);
    else if (layout == kNN) BT_SIMT(kNN);
    else BT_SIMT(kTN);
#undef BT_SIMT
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

}  // namespace bt
