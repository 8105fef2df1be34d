// Attention dispatch: tcgen05 kernels for head_dim 64 and 128 when the inputs come as hi/lo
// planes, warp-MMA kernels for head_dim 16 / 32 / 64 on raw inputs, the FP32 FMA reference on request.
#include "common.cuh"

namespace bt {

cudaError_t launch_attention_fwd_simt(const float* qkv, int B, int T, int C, int H, float* o, float* o_hi,
                                      float* o_lo, float* lse, cudaStream_t s);
cudaError_t launch_attention_bwd_simt(const float* qkv, const float* o, const float* o_lo, const float* lse,
                                      const float* d_o, int B, int T, int C, int H, float* dqkv, float* dqkv_hi,
                                      float* dqkv_lo, float* dvec, cudaStream_t s);
cudaError_t launch_attention_dvec(const float* o, const float* o_lo, const float* d_o, const float* d_o_lo, int B,
                                  int T, int C, int H, float* dvec, cudaStream_t s);
cudaError_t launch_attention_bwd_tc(const float* qkv_hi, int64_t qkv_plane, const float* do_hi, int64_t do_plane,
                                    const float* o, const float* o_lo, const float* lse, float* dvec, int B, int T,
                                    int C, int H, float* dqkv_hi, int64_t dqkv_plane, float* rg_sums, int* err_word,
                                    cudaStream_t s);
// Heads per group in the CTA order of the head_dim-64 tensor-core kernels: the smallest divisor of the
// head count whose groups hold at least one and a half times as many CTAs as there are SMs (equal groups:
// a short last group starts its long walks last and becomes the tail).  Measured: 16 - 32 heads at 8
// blocks per head (forward -6 %, backward -1 to -2 %), 2 heads at 128 blocks (-6 % / -3 %), no gain at
// 32 blocks, and groups smaller than the machine lose up to 13 % in the backward kernels.
// BT_ATTN_HEAD_GROUP=n pins it (tuning aid).
int attn_head_group(int heads, int blocks) {
    static const int forced = []() {
        const char* v = getenv("BT_ATTN_HEAD_GROUP");
        return v ? atoi(v) : 0;
    }();
    if (forced > 0) return forced < heads ? forced : heads;
    static const int sms = []() {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        return n;
    }();
    if (blocks < 1) blocks = 1;
    for (int g = 1; g < heads; ++g)
        if (heads % g == 0 && 2 * g * blocks >= 3 * sms) return g;
    return heads;
}

bool attention_mma_supports(int head_dim);
cudaError_t launch_attention_fwd_mma(const float* qkv, int B, int T, int C, int H, float* o, float* o_hi,
                                     float* o_lo, float* lse, cudaStream_t s);
cudaError_t launch_attention_bwd_mma(const float* qkv, const float* lse, const float* d_o, const float* dvec, int B,
                                     int T, int C, int H, float* dqkv, float* dqkv_hi, float* dqkv_lo,
                                     cudaStream_t s);

bool attention_tc_supports(int head_dim, int C);
bool attention_tc128_supports(int head_dim, int C);
cudaError_t launch_attention_fwd_tc128(const float* qkv_hi, int64_t qkv_plane, int B, int T, int C, int H, float* o,
                                       float* o_hi, float* o_lo, float* lse, int* err_word, cudaStream_t s);
cudaError_t launch_attention_bwd_tc128(const float* qkv_hi, int64_t qkv_plane, const float* do_hi, int64_t do_plane,
                                       const float* lse, const float* dvec, int B, int T, int C, int H, float* dqkv_hi,
                                       int64_t dqkv_plane, float* rg_sums, int* err_word, cudaStream_t s);
cudaError_t launch_attention_fwd_tc(const float* qkv_hi, int64_t qkv_plane, int B, int T, int C, int H, float* o,
                                    float* o_hi, float* o_lo, float* lse, int* err_word, cudaStream_t s);

// qkv_hi (nullable): the same qkv as TF32 hi/lo planes (lo at qkv_hi + qkv_plane); with it and
// head_dim 64 or 128 the tcgen05 kernels run, otherwise the warp-MMA kernel on the raw array.
cudaError_t launch_attention_fwd(const float* qkv, const float* qkv_hi, int64_t qkv_plane, int B, int T, int C, int H,
                                 float* o, float* o_hi, float* o_lo, float* lse, bool simt, int* err_word,
                                 cudaStream_t s) {
    if (!simt && qkv_hi && attention_tc_supports(C / H, C))
        return launch_attention_fwd_tc(qkv_hi, qkv_plane, B, T, C, H, o, o_hi, o_lo, lse, err_word, s);
    if (!simt && qkv_hi && lse && attention_tc128_supports(C / H, C))
        return launch_attention_fwd_tc128(qkv_hi, qkv_plane, B, T, C, H, o, o_hi, o_lo, lse, err_word, s);
    if (!qkv) return cudaErrorInvalidValue;
    if (simt || !attention_mma_supports(C / H)) return launch_attention_fwd_simt(qkv, B, T, C, H, o, o_hi, o_lo, lse, s);
    return launch_attention_fwd_mma(qkv, B, T, C, H, o, o_hi, o_lo, lse, s);
}

// Inputs may be given raw and/or as hi/lo planes (qkv_hi, do_hi; lo at +plane).  With head_dim 64 or 128,
// both split inputs and only the split output requested, the tcgen05 kernels run; otherwise the
// warp-MMA kernels run on the raw arrays.
cudaError_t launch_attention_bwd(const float* qkv, const float* qkv_hi, int64_t qkv_plane, const float* o,
                                 const float* o_lo, const float* lse, const float* d_o, const float* do_hi,
                                 int64_t do_plane, int B, int T, int C, int H, float* dqkv, float* dqkv_hi,
                                 float* dqkv_lo, float* dvec, bool simt, int* err_word, cudaStream_t s,
                                 float* rg_sums, bool* rg_sums_written) {
    if (rg_sums_written) *rg_sums_written = false;
    const bool tc128 = attention_tc128_supports(C / H, C);
    const bool tc = !simt && qkv_hi && do_hi && dqkv_hi && !dqkv && (attention_tc_supports(C / H, C) || tc128) &&
                    dqkv_lo == dqkv_hi + (int64_t)B * T * 3 * C;
    if (tc) {
        if (rg_sums_written) *rg_sums_written = rg_sums != nullptr;
        if (!tc128)   // head_dim 64: the dq kernel forms rowsum(dO o O) itself
            return launch_attention_bwd_tc(qkv_hi, qkv_plane, do_hi, do_plane, o, o_lo, lse, dvec, B, T, C, H, dqkv_hi,
                                           (int64_t)B * T * 3 * C, rg_sums, err_word, s);
        cudaError_t e = d_o ? launch_attention_dvec(o, o_lo, d_o, nullptr, B, T, C, H, dvec, s)
                            : launch_attention_dvec(o, o_lo, do_hi, do_hi + do_plane, B, T, C, H, dvec, s);
        if (e != cudaSuccess) return e;
        return launch_attention_bwd_tc128(qkv_hi, qkv_plane, do_hi, do_plane, lse, dvec, B, T, C, H, dqkv_hi,
                                          (int64_t)B * T * 3 * C, rg_sums, err_word, s);
    }
    if (!qkv || !d_o) return cudaErrorInvalidValue;
    if (simt || !attention_mma_supports(C / H))
        return launch_attention_bwd_simt(qkv, o, o_lo, lse, d_o, B, T, C, H, dqkv, dqkv_hi, dqkv_lo, dvec, s);
    cudaError_t e = launch_attention_dvec(o, o_lo, d_o, nullptr, B, T, C, H, dvec, s);
    if (e != cudaSuccess) return e;
    return launch_attention_bwd_mma(qkv, lse, d_o, dvec, B, T, C, H, dqkv, dqkv_hi, dqkv_lo, s);
}

}  // namespace bt
