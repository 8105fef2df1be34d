// Self-test of the bounded device-side wait: one CTA of one warp runs the library's own
// mbar_wait_warp on a shared-memory barrier that nothing ever arrives at, with a caller-chosen
// limit.  No TMA, no tensor memory, nothing in flight: the wait runs out, the error word is
// raised with code kSelftestWaitCode, and the kernel returns normally.  This is how the path
// bounded wait -> device error word -> BT_ERR_DEVICE_TIMEOUT is exercised without any kernel
// misbehaving.
#include "tc_common.cuh"

namespace bt {

__global__ void __launch_bounds__(32) bounded_wait_probe_kernel(int* err, unsigned long long limit_ns, int code) {
    pdl_wait();
    pdl_trigger();
    __shared__ __align__(8) unsigned long long bar;
    const uint32_t b = tc::smem_u32(&bar);
    if (threadIdx.x == 0) {
        tc::mbar_init(b, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    // phase 0 of a freshly initialised barrier never completes without an arrival
    (void)tc::mbar_wait_warp(b, 0u, err, code, limit_ns);
}

cudaError_t launch_bounded_wait_probe(int* err, unsigned long long limit_ns, int code, cudaStream_t s) {
    BT_KERNEL_LAUNCH((bounded_wait_probe_kernel), 1, 32, 0, s, err, limit_ns, code);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

}  // namespace bt

// ------------------------------------------------------------------ tensor-pipe rate probe
//
// What one SM's tensor pipe delivers for tcgen05.mma.kind::tf32: every CTA (one per SM when the
// grid is the SM count) issues `iters` dependent-free MMAs of M = 128, N = 256, K = 8 from one
// thread, operands in shared memory (K-major, 128-byte swizzle), alternating between two
// accumulators, and records the SM clocks from the first issue to the completion of the last.
// 128 * 256 * 8 MACs per instruction divided by the clocks per instruction is the dense TF32 rate in
// MAC per clock per SM; times 2 * SMs * the SM clock it is the measured TF32 peak that the 3xTF32
// GEMM's roofline is scaled with (three MMAs per FP32 product).  The operand values are arbitrary
// finite numbers; nothing is read back but the clock counts.
namespace bt {

using namespace tc;

__global__ void __launch_bounds__(128) tf32_rate_probe_kernel(int iters, long long* __restrict__ clocks, int* err) {
    extern __shared__ uint8_t probe_smem[];
    __shared__ uint32_t tmem_base_s;
    __shared__ __align__(8) unsigned long long bar;
    const uint32_t sm0 = (smem_u32(probe_smem) + 1023u) & ~1023u;
    float* smf = reinterpret_cast<float*>(probe_smem + (sm0 - smem_u32(probe_smem)));
    const int tid = threadIdx.x;
    for (int i = tid; i < (48 * 1024) / 4; i += 128) smf[i] = 0.001f * (float)(i & 255);
    if (tid < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tmem_base_s;
    long long dt = -1;
    if (tid == 0) {
        const DescBase ad = kmaj_base(sm0), bd = kmaj_base(sm0 + 16u * 1024u);   // A: 128 rows, B: 256 rows of 128 B
        constexpr uint32_t idesc = make_idesc_tf32(128, 256, false, false);
        const long long t0 = clock64();
        for (int it = 0; it < iters; ++it) {
            const uint32_t koff = (uint32_t)(it & 3) * 32u;          // the four 8-deep k-steps of a 128-byte row
            umma_tf32(tm + (uint32_t)(it & 1) * 256u, ad.at(koff), bd.at(koff), idesc, it >= 2 ? 1u : 0u);
        }
        umma_commit(smem_u32(&bar));
        if (mbar_wait(smem_u32(&bar), 0u, err, 901)) dt = clock64() - t0;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (tid < 32) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tm), "r"(512u) : "memory");
    if (tid == 0) clocks[blockIdx.x] = dt;
}

// The issue-rate probe: `issuers` threads (lane 0 of warps 0 .. issuers - 1) each issue `iters`
// MMAs of M = 128, N, K = 8 -- A from shared memory or (TS) from tensor memory -- into an accumulator
// of their own where the columns allow (N = 64) or a shared one, and record the clocks from their
// first issue to the completion of their last MMA.
template <int N, bool TS>
__global__ void __launch_bounds__(128) mma_issue_probe_kernel(int iters, int issuers, long long* __restrict__ clocks, int* err) {
    extern __shared__ uint8_t probe_smem[];
    __shared__ uint32_t tmem_base_s;
    __shared__ __align__(8) unsigned long long bar[4];
    const uint32_t sm0 = (smem_u32(probe_smem) + 1023u) & ~1023u;
    float* smf = reinterpret_cast<float*>(probe_smem + (sm0 - smem_u32(probe_smem)));
    const int tid = threadIdx.x, w = tid >> 5;
    for (int i = tid; i < (48 * 1024) / 4; i += 128) smf[i] = 0.001f * (float)(i & 255);
    if (tid < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid == 0) {
        for (int i = 0; i < 4; ++i) mbar_init(smem_u32(&bar[i]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tm = tmem_base_s;
    if ((tid & 31) == 0 && w < issuers) {
        const DescBase ad = kmaj_base(sm0), bd = kmaj_base(sm0 + 16u * 1024u);   // A: 128 rows, B: up to 256 rows of 128 B
        constexpr uint32_t idesc = make_idesc_tf32(128, N, false, false);
        const uint32_t d = tm + 256u + (N <= 64 ? (uint32_t)w * 64u : 0u);         // columns 0-63 serve as the TMEM A operand
        long long dt = -1;
        const long long t0 = clock64();
        for (int it = 0; it < iters; ++it) {
            const uint32_t koff = (uint32_t)(it & 3) * 32u;
            if (TS) umma_tf32_ts(d, tm + (uint32_t)(it & 7) * 8u, bd.at(koff), idesc, 1u);
            else umma_tf32(d, ad.at(koff), bd.at(koff), idesc, 1u);
        }
        umma_commit(smem_u32(&bar[w]));
        if (mbar_wait(smem_u32(&bar[w]), 0u, err, 902)) dt = clock64() - t0;
        clocks[blockIdx.x * 4 + w] = dt;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (tid < 32) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tm), "r"(512u) : "memory");
}

template <int N, bool TS>
static cudaError_t launch_issue_probe_t(int n_ctas, int iters, int issuers, long long* clocks, int* err, cudaStream_t s) {
    constexpr int kSmem = 49 * 1024 + 1024;
    cudaError_t e = cudaFuncSetAttribute(mma_issue_probe_kernel<N, TS>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    mma_issue_probe_kernel<N, TS><<<n_ctas, 128, kSmem, s>>>(iters, issuers, clocks, err);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

cudaError_t launch_mma_issue_probe(int n, int a_in_tmem, int issuers, int n_ctas, int iters, long long* clocks, int* err,
                                   cudaStream_t s) {
    if (n == 64) return a_in_tmem ? launch_issue_probe_t<64, true>(n_ctas, iters, issuers, clocks, err, s)
                                  : launch_issue_probe_t<64, false>(n_ctas, iters, issuers, clocks, err, s);
    if (n == 128) return a_in_tmem ? launch_issue_probe_t<128, true>(n_ctas, iters, issuers, clocks, err, s)
                                   : launch_issue_probe_t<128, false>(n_ctas, iters, issuers, clocks, err, s);
    if (n == 256 && !a_in_tmem) return launch_issue_probe_t<256, false>(n_ctas, iters, issuers, clocks, err, s);
    return cudaErrorInvalidValue;
}

cudaError_t launch_tf32_rate_probe(int n_ctas, int iters, long long* clocks, int* err, cudaStream_t s) {
    constexpr int kSmem = 49 * 1024 + 1024;
    static cudaError_t attr =
        cudaFuncSetAttribute(tf32_rate_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (attr != cudaSuccess) return attr;
    tf32_rate_probe_kernel<<<n_ctas, 128, kSmem, s>>>(iters, clocks, err);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

}  // namespace bt
