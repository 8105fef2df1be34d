// Shared device helpers and the internal launcher interface of the bt library.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

// Records the thread-local error string returned by bt_last_error() and passes `status` through
// (defined with the C ABI; status is a bt_status).
extern "C" int bt_internal_fail_int(int status, const char* message);

namespace bt {

// Every launcher bumps this counter once per kernel launch (read by bt_launch_count).
extern std::atomic<long long> g_launches;
#define BT_COUNT_LAUNCH() (::bt::g_launches.fetch_add(1, std::memory_order_relaxed))

constexpr float kLnEps = 1e-5f;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// TF32 split: hi = x rounded to the nearest TF32 value (10 mantissa bits, low 13 bits zero),
// lo = x - hi, which is exact in FP32; x = hi + lo holds bit for bit.  Rounding to nearest
// (instead of clearing the low bits) keeps |lo| <= 2^-11 |x| and, more importantly, gives lo a
// random sign, so the terms the three-product scheme drops (lo*lo, and the low bits of lo the
// tensor core ignores) do not add up to a systematic shrink over a chain of GEMMs.
__device__ __forceinline__ void split_tf32(float x, float& hi, float& lo) {
    uint32_t h;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(h) : "f"(x));
    hi = __uint_as_float(h);
    lo = x - hi;
}
__device__ __forceinline__ void split_tf32(const float4& x, float4& hi, float4& lo) {
    split_tf32(x.x, hi.x, lo.x);
    split_tf32(x.y, hi.y, lo.y);
    split_tf32(x.z, hi.z, lo.z);
    split_tf32(x.w, hi.w, lo.w);
}

// Writes v to the raw array and/or to the hi/lo planes at float4 index i.
__device__ __forceinline__ void store_raw_split(float4 v, float* raw, float* hi, float* lo, int64_t i4) {
    if (raw) reinterpret_cast<float4*>(raw)[i4] = v;
    if (hi) {
        float4 h, l;
        split_tf32(v, h, l);
        reinterpret_cast<float4*>(hi)[i4] = h;
        reinterpret_cast<float4*>(lo)[i4] = l;
    }
}

__device__ __forceinline__ float4 ld4(const float* p, int64_t i4) {
    return reinterpret_cast<const float4*>(p)[i4];
}
__device__ __forceinline__ float4 add4(float4 a, float4 b) {
    return make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w);
}

// A GEMM operand stored as two FP32 planes (hi at `hi`, lo at `hi + plane`), row-major
// with `ld` floats between rows.
struct SplitMat {
    const float* hi;
    int64_t plane;
    int64_t rows, cols, ld;
};

#ifdef __CUDACC__
// GELU and its derivative (erf form, or the tanh form): shared by the GELU kernels and the GEMM
// epilogues, where four warps per SM evaluate them for a whole output tile -- hence branch-free and
// about twenty instructions for both values together.
//   erf form:  GELU(x) = x Phi(x),  GELU'(x) = Phi(x) + x phi(x), with one exponential
//              E = exp(-x^2 / 2) shared by phi and by the complementary error function, which is
//              the five-term rational approximation of Abramowitz & Stegun 7.1.26 (absolute error
//              1.5e-7 on erf: about one FP32 rounding of Phi);
//   tanh form: tanh(u) = 1 - 2 / (1 + exp(2u)),  u = sqrt(2 / pi) (x + 0.044715 x^3).
__device__ __forceinline__ float ex2_fast(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float rcp_fast(float x) {
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void gelu_both_f(float x, bool tanh_form, float& g, float& gp) {
    if (tanh_form) {
        const float x2 = x * x;
        const float u = 0.7978845608028654f * fmaf(0.044715f * x2, x, x);
        const float t = 1.0f - 2.0f * rcp_fast(1.0f + ex2_fast(2.8853900817779268f * u));   // exp(2u) = 2^(2u log2 e)
        const float du = 0.7978845608028654f * fmaf(3.0f * 0.044715f, x2, 1.0f);
        const float half = 0.5f * (1.0f + t);
        g = x * half;
        gp = fmaf(0.5f * x * du, fmaf(-t, t, 1.0f), half);
        return;
    }
    const float E = ex2_fast(-0.7213475204444817f * x * x);                  // exp(-x^2 / 2)
    const float r = rcp_fast(fmaf(0.3275911f * 0.7071067811865476f, fabsf(x), 1.0f));
    float q = fmaf(r, 1.061405429f, -1.453152027f);
    q = fmaf(q, r, 1.421413741f);
    q = fmaf(q, r, -0.284496736f);
    q = fmaf(q, r, 0.254829592f);
    const float half_erfc = 0.5f * q * r * E;                                // erfc(|x| / sqrt 2) / 2
    const float Phi = x >= 0.f ? 1.0f - half_erfc : half_erfc;
    g = x * Phi;
    gp = fmaf(x * 0.3989422804014327f, E, Phi);
}
__device__ __forceinline__ float gelu_f(float x, bool tanh_form) {
    float g, gp;
    gelu_both_f(x, tanh_form, g, gp);
    return g;
}
__device__ __forceinline__ float gelu_grad_f(float x, bool tanh_form) {
    float g, gp;
    gelu_both_f(x, tanh_form, g, gp);
    return gp;
}
#endif

// ---------------------------------------------------------------- programmatic dependent launch
// Every kernel of the step starts with pdl_wait() (returns once the kernels before it in the stream
// have completed and their writes are visible) followed by pdl_trigger() (lets the NEXT launch be
// scheduled), and is launched with the programmatic-stream-serialization attribute: the next
// kernel's launch latency and block scheduling then overlap the tail of the current one instead of
// following it.  BT_PDL=0 in the environment turns the attribute off (plain stream order).
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif
bool pdl_enabled();
template <typename... KArgs, typename... Args>
cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#define BT_KERNEL_LAUNCH(kernel, grid, block, smem, stream, ...) \
    (void)bt::launch_k(kernel, dim3(grid), dim3(block), (size_t)(smem), stream, __VA_ARGS__)

enum GemmLayout { kNT = 0, kNN = 1, kTN = 2 };

// One weight matrix of the parameter arena ([rows, cols] row-major at float offset `off`) and the
// index of its first 64x64 tile in the concatenated tile list of all matrices.
struct MatDesc {
    long long off;
    int rows, cols;
    int tile0, tiles_c;
};
constexpr int kMaxSplitMats = 256;
// For every listed matrix: TF32 hi/lo planes in place (w_hi + off, lo at + plane) AND the hi/lo
// planes of its transpose ([cols, rows] row-major at wt_hi + off), in one pass over the weights.
cudaError_t launch_split_matrices(const float* params, float* w_hi, float* wt_hi, int64_t plane,
                                  const MatDesc* descs_dev, int nmats, int ntiles, cudaStream_t s);

struct AdamParams {
    float lr, beta1, beta2, eps, weight_decay;
    float inv_c1, inv_c2;  // 1 / (1 - beta^t), computed on the host in double
};

// ---------------------------------------------------------------- launchers (host)
// All return cudaGetLastError() of their launches.

cudaError_t launch_split(const float* x, float* hi, float* lo, int64_t n, cudaStream_t s);
// Ids outside [0, V) are treated as id 0; position + 1 of one of them is left in *bad (nullable).
cudaError_t launch_embedding_fwd(const int32_t* tok, const float* wte, const float* wpe, int64_t N, int T,
                                 int C, int V, float* x, int* bad, cudaStream_t s);
// partial: N*C floats (embedding_bwd_partial_bytes); table: Vp bytes per chunk of 128 positions, the rest of
// embedding_bwd_scratch_bytes (both scratch, contents irrelevant on entry).
size_t embedding_bwd_partial_bytes(int64_t N, int C);
size_t embedding_bwd_scratch_bytes(int64_t N, int C, int Vp);
cudaError_t launch_embedding_bwd(const int32_t* tok, const float* dx, int64_t N, int T, int C, int V, int Vp,
                                 float* dwte, float* dwpe, float* partial, uint8_t* table, cudaStream_t s);
cudaError_t launch_layernorm_fwd(const float* x, const float* gamma, const float* beta, int64_t N, int C,
                                 float* y, float* y_hi, float* y_lo, float* mean, float* rstd, cudaStream_t s);
size_t layernorm_bwd_scratch_floats(int64_t N, int C);
cudaError_t launch_layernorm_bwd(const float* dy, const float* x, const float* gamma, const float* mean,
                                 const float* rstd, const float* dres, int64_t N, int C, float* dx, float* dx_hi,
                                 float* dx_lo, float* dgamma, float* dbeta, float* dx_colsum, float* scratch,
                                 cudaStream_t s);   // dx_colsum (nullable): column sums of the dx written
cudaError_t launch_gelu_fwd(const float* x, int64_t n, int tanh_form, float* y, float* y_hi, float* y_lo,
                            cudaStream_t s);
cudaError_t launch_gelu_bwd(const float* x, const float* dy, int64_t n, int tanh_form, float* dx, float* dx_hi,
                            float* dx_lo, cudaStream_t s);
// GELU backward that also writes the column sums of dx (an N x C matrix) into colsum[C];
// scratch as for launch_colsum(N, C).
cudaError_t launch_gelu_bwd_colsum(const float* x, const float* dy, int64_t N, int C, int tanh_form, float* dx,
                                   float* dx_hi, float* dx_lo, float* colsum, float* scratch, cudaStream_t s);
cudaError_t launch_softmax_xent(const float* logits, const int32_t* targets, int64_t N, int Vp, float inv_count,
                                float* losses, float* loss_mean, float* dl, float* dl_hi, float* dl_lo, int V,
                                int* bad, cudaStream_t s);
int softmax_xent_max_in_place_columns();
size_t colsum_scratch_floats(int64_t N, int C);
// x_lo (nullable): second plane added to the first (sums a split array).
cudaError_t launch_colsum_stage2(const float* partial, int groups, int C, float* out, cudaStream_t s);
cudaError_t launch_colsum(const float* x, const float* x_lo, int64_t N, int C, float* out, float* scratch,
                          cudaStream_t s);
// Gradient accumulation over micro-steps (see the kernel): n % 4 == 0.
cudaError_t launch_grad_accumulate(float* acc, float* g, int64_t n, float w, int mode, float* loss_acc, float* loss,
                                   cudaStream_t s);
size_t grad_norm_scratch_bytes(int64_t n);
cudaError_t launch_grad_norm(const float* g, int64_t n, float clip, float* out2, void* scratch, cudaStream_t s);
// Flat-arena AdamW: n floats (multiple of 1024), decay_flags[n / 1024].
cudaError_t launch_adamw_flat(float* p, const float* g, float* m, float* v, int64_t n, const uint8_t* decay_flags,
                              AdamParams hp, const float* d_scale, cudaStream_t s);
struct AdamTensorList {
    enum { kMax = 64 };
    float* p[kMax];
    const float* g[kMax];
    float* m[kMax];
    float* v[kMax];
    long long numel[kMax];
    int decay[kMax];
    int chunk_begin[kMax + 1];
    int n;
};
cudaError_t launch_adamw_multi(const AdamTensorList& tl, AdamParams hp, const float* d_scale, cudaStream_t s);
cudaError_t launch_splitk_reduce(const float* partials, int splits, int64_t n, float* out, cudaStream_t s);
cudaError_t launch_init_normal(float* p, int64_t n, float std, uint64_t seed, uint64_t offset, cudaStream_t s);
cudaError_t launch_fill(float* p, int64_t n, float v, cudaStream_t s);
// One warp waits (bounded by limit_ns) on a barrier nobody arrives at, then raises *err = code.
constexpr int kSelftestWaitCode = 900;
cudaError_t launch_bounded_wait_probe(int* err, unsigned long long limit_ns, int code, cudaStream_t s);
// clocks[cta] = SM clocks that `iters` tcgen05.mma.kind::tf32 (128 x 256 x 8) took on that CTA's SM (-1: wait ran out).
cudaError_t launch_tf32_rate_probe(int n_ctas, int iters, long long* clocks, int* err, cudaStream_t s);
cudaError_t launch_mma_issue_probe(int n, int a_in_tmem, int issuers, int n_ctas, int iters, long long* clocks, int* err,
                                   cudaStream_t s);

// SIMT reference GEMM: D = op(A) op(B) (+bias) (+residual), operands given as split planes
// (lo may be absent: plane == 0 means "hi only").
cudaError_t launch_gemm_simt(int layout, int64_t M, int64_t N, int64_t K, SplitMat A, SplitMat B, float* D,
                             int64_t ldd, const float* bias, const float* residual, cudaStream_t s);

// tcgen05 GEMM.  `partials` (nullable) receives split-K partial sums; max_partial_floats its size.
// D may be null when d_hi is given: the output is then written only as TF32 hi/lo planes
// (d_hi[row*ldd + col], lo plane at d_hi + d_plane).
// err_word: device int set non-zero when a bounded wait ran out.
cudaError_t launch_gemm_tc(int layout, int64_t M, int64_t N, int64_t K, SplitMat A, SplitMat B, float* D,
                           int64_t ldd, const float* bias, const float* residual, float* partials,
                           size_t max_partial_floats, int* err_word, cudaStream_t s, float* d_hi = nullptr,
                           int64_t d_plane = 0, int two_cta_mode = -1, int act = 0, float* col_partial = nullptr);
// act: 1 / 2 = the hi/lo planes receive GELU(output) (erf / tanh form) while D keeps the output itself;
//      3 / 4 = the same planes, and D receives GELU'(output) instead of the output (what the backward
//      pass needs of it);
//      5 / 6 = GELU backward in the epilogue: `residual` holds the pre-activation h [M, N] and the
//      output is (A B) o GELU'(h) (erf / tanh form) -- the input gradient of the GELU whose output
//      fed the product that A B back-propagates through;  7 = the same with GELU'(h) already in
//      `residual`.  In 5 - 7 col_partial (nullable) receives the column sums of the output per 32-row
//      group, [ceil(M / 32)][N]: launch_colsum_stage2 adds the groups in order (the bias gradient of
//      the layer that produced h); no bias, no K-split.
// two_cta_mode: -1 the planner chooses between 128-row tiles on single CTAs and 256-row tiles on
// CTA pairs (cta_group::2); 0 / 1 force the one or the other (1 applies where M >= 256).
size_t gemm_tc_partial_floats_bound();
size_t gemm_tc_partial_floats_for_chain_cap(int64_t M, int64_t N, int64_t K);
// Heads per group in the CTA order of the head_dim-64 tensor-core attention kernels, for a grid of
// `heads` (sequence x head) by `blocks` (query or key blocks) CTAs.
int attn_head_group(int heads, int blocks);
void gemm_tc_plan_info(int64_t M, int64_t N, int64_t K, bool can_split, bool can_tail, int two_cta_mode, int out[7]);
bool gemm_tc_init(char* err, size_t errlen);  // resolves the tensor-map encoder

// Attention.  lo planes are written when the hi pointer is non-null.
cudaError_t launch_attention_fwd(const float* qkv, const float* qkv_hi, int64_t qkv_plane, int B, int T, int C, int H,
                                 float* o, float* o_hi, float* o_lo, float* lse, bool simt, int* err_word,
                                 cudaStream_t s);
cudaError_t attention_tc_default_err(int** out);
// o given raw (o_lo == nullptr) or as hi/lo planes.  dvec: B*H*T floats of scratch.  qkv and d_o may
// be given raw and/or as hi/lo planes (see attention.cu for which kernel then runs).
cudaError_t launch_attention_bwd(const float* qkv, const float* qkv_hi, int64_t qkv_plane, const float* o,
                                 const float* o_lo, const float* lse, const float* d_o, const float* do_hi,
                                 int64_t do_plane, int B, int T, int C, int H, float* dqkv, float* dqkv_hi,
                                 float* dqkv_lo, float* dvec, bool simt, int* err_word, cudaStream_t s,
                                 float* rg_sums = nullptr, bool* rg_sums_written = nullptr);
// rg_sums (nullable): [attention_bwd_rowgroups(B, T)][3C] floats; when the tcgen05 kernels run they
// fill it with the column sums of dqkv per 32-row group (*rg_sums_written = true), so the QKV bias
// gradient is the column sum of this small array.
int64_t attention_bwd_rowgroups(int B, int T);

}  // namespace bt
