// Causal flash attention forward on the 5th-generation tensor cores (head_dim 64), FP32 fidelity
// through 3xTF32 split products.
//
// One CTA owns 128 query rows of one (sequence, head) -- one row per TMEM lane -- and walks the
// 64-key tiles up to the diagonal:
//
//   warp 0 (one lane)  TMA producer: Q once, then double-buffered K tiles (K-major, 128-byte
//                      swizzle) and V tiles (MN-major, 128-byte swizzle with 32-byte atoms), each as
//                      hi/lo planes straight from the split qkv array the QKV GEMM wrote.
//   warp 1 (one lane)  MMA issuer.  S = Q K^T: 24 tcgen05.mma.kind::tf32 (8 k-steps x 3 split
//                      terms) with both operands in shared memory, accumulator S[buf] in TMEM.
//                      O_tile = P V: 24 MMAs with A = P (hi/lo) read from TENSOR MEMORY and B = V
//                      from shared memory, accumulator O[buf] in TMEM.  S of tile t+1 is issued
//                      before P V of tile t, so the tensor pipe works while the softmax runs.
//   warps 2-5          softmax / correction: thread i owns query row i.  It reads its 64 scores
//                      with tcgen05.ld (the row maximum and sum need no shuffles), forms
//                      p = exp2((s - m) * scale*log2e), splits p into hi/lo and writes both back to
//                      TMEM with tcgen05.st as the A operand of P V.  The running output is kept in
//                      registers: O_reg = O_reg * corr + O_tile, so no accumulator in TMEM is ever
//                      rescaled.
//
// TMEM map (512 columns): per buffer b in {0,1}: S at 256b, P_hi at 256b+64, P_lo at 256b+128,
// O_tile at 256b+192.  Shared memory: Q 64 KB, K 2 x 32 KB, V 2 x 32 KB.
// Every mbarrier wait is bounded; a wait that runs out raises the device error word and the CTA
// drains, frees its TMEM and exits.  No cluster multicast is used.
#include "common.cuh"
#include "tc_common.cuh"

namespace bt {

using namespace tc;

namespace {

constexpr int HD = 64, BQ = 128, BKV = 64;
constexpr int kThreads = 192;
constexpr uint32_t kQBytes = 2u * 2u * BQ * 128u;      // 2 k-blocks x (hi, lo) x 128 rows x 128 B
constexpr uint32_t kKVBytes = 2u * 2u * BKV * 128u;    // per buffer
constexpr uint32_t kSmemBytes = 1024u + kQBytes + 4u * kKVBytes + 256u;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct AttnArgs {
    int T, C, H;
    float* o;
    float* o_hi;
    float* o_lo;
    float* lse;
    int* err;
};

__global__ void __launch_bounds__(kThreads, 1)
attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmV, const AttnArgs g) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t q_s = smem_base;
    const uint32_t k_s = q_s + kQBytes;            // two buffers
    const uint32_t v_s = k_s + 2u * kKVBytes;      // two buffers
    const uint32_t bars = v_s + 2u * kKVBytes;
    // barrier slots
    const uint32_t q_full = bars;
    auto k_full = [&](int b) { return bars + 8u * (1 + b); };
    auto k_empty = [&](int b) { return bars + 8u * (3 + b); };
    auto v_full = [&](int b) { return bars + 8u * (5 + b); };
    auto v_empty = [&](int b) { return bars + 8u * (7 + b); };
    auto s_full = [&](int b) { return bars + 8u * (9 + b); };
    auto p_full = [&](int b) { return bars + 8u * (11 + b); };
    auto o_full = [&](int b) { return bars + 8u * (13 + b); };
    const uint32_t tmem_slot = bars + 8u * 15;
    volatile uint32_t* tmem_slot_ptr =
        reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - smem_u32(smem_raw)));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int qt = gridDim.x - 1 - blockIdx.x;           // heaviest query tiles first
    const int b = blockIdx.y / g.H, h = blockIdx.y % g.H;
    const int q0 = qt * BQ;
    const int last_row = min(q0 + BQ - 1, g.T - 1);
    const int n_kt = last_row / BKV + 1;
    const int row_base = b * g.T;                         // row of this sequence in the [B*T, 3C] array

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(k_full(i), 1);
            mbar_init(k_empty(i), 1);
            mbar_init(v_full(i), 1);
            mbar_init(v_empty(i), 1);
            mbar_init(s_full(i), 1);
            mbar_init(p_full(i), 4);
            mbar_init(o_full(i), 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(512u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot_ptr;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            mbar_expect_tx(q_full, kQBytes);
            for (int kb = 0; kb < 2; ++kb)
                tma_load_3d(q_s + kb * (kQBytes / 2), &tmQ, q_full, h * HD + kb * 32, row_base + q0, 0);
            bool ok = true;
            for (int kt = 0; kt < n_kt && ok; ++kt) {
                const int buf = kt & 1;
                const uint32_t ph = (kt >> 1) & 1u;
                if (!mbar_wait(k_empty(buf), ph ^ 1u, g.err, 11)) { ok = false; break; }
                mbar_expect_tx(k_full(buf), kKVBytes);
                for (int kb = 0; kb < 2; ++kb)
                    tma_load_3d(k_s + buf * kKVBytes + kb * (kKVBytes / 2), &tmK, k_full(buf),
                                g.C + h * HD + kb * 32, row_base + kt * BKV, 0);
                if (!mbar_wait(v_empty(buf), ph ^ 1u, g.err, 12)) { ok = false; break; }
                mbar_expect_tx(v_full(buf), kKVBytes);
                for (int grp = 0; grp < 2; ++grp)
                    tma_load_3d(v_s + buf * kKVBytes + grp * (kKVBytes / 2), &tmV, v_full(buf),
                                2 * g.C + h * HD + grp * 32, row_base + kt * BKV, 0);
            }
            if (!ok)
                for (int i = 0; i < 2000; ++i) __nanosleep(1000);  // let loads in flight land
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_s = make_idesc_tf32(BQ, BKV, false, false);
            constexpr uint32_t idesc_o = make_idesc_tf32(BQ, HD, false, true);
            bool ok = mbar_wait(q_full, 0, g.err, 13);
            auto issue_s = [&](int kt) -> bool {
                const int buf = kt & 1;
                if (!mbar_wait(k_full(buf), (kt >> 1) & 1u, g.err, 14)) return false;
                tc_fence_after();
                const uint32_t d = tmem_base + (uint32_t)buf * 256u;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const int kb = ks >> 2, j = ks & 3;
                    const uint32_t qa = q_s + kb * (kQBytes / 2) + j * 32u;
                    const uint32_t ka = k_s + buf * kKVBytes + kb * (kKVBytes / 2) + j * 32u;
                    const uint64_t a_hi = make_desc(qa, 16u, 1024u, 2u), a_lo = make_desc(qa + BQ * 128u, 16u, 1024u, 2u);
                    const uint64_t b_hi = make_desc(ka, 16u, 1024u, 2u), b_lo = make_desc(ka + BKV * 128u, 16u, 1024u, 2u);
                    umma_tf32(d, a_lo, b_hi, idesc_s, ks > 0 ? 1u : 0u);
                    umma_tf32(d, a_hi, b_lo, idesc_s, 1u);
                    umma_tf32(d, a_hi, b_hi, idesc_s, 1u);
                }
                umma_commit(k_empty(buf));
                umma_commit(s_full(buf));
                return true;
            };
            auto issue_pv = [&](int kt) -> bool {
                const int buf = kt & 1;
                if (!mbar_wait(p_full(buf), (kt >> 1) & 1u, g.err, 15)) return false;
                if (!mbar_wait(v_full(buf), (kt >> 1) & 1u, g.err, 16)) return false;
                tc_fence_after();
                const uint32_t t0 = tmem_base + (uint32_t)buf * 256u;
                const uint32_t d = t0 + 192u;
                const uint32_t va = v_s + buf * kKVBytes;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint64_t b_hi = make_desc(va + j * 1024u, kKVBytes / 2, 512u, 1u);
                    const uint64_t b_lo = make_desc(va + BKV * 128u + j * 1024u, kKVBytes / 2, 512u, 1u);
                    umma_tf32_ts(d, t0 + 128u + j * 8u, b_hi, idesc_o, j > 0 ? 1u : 0u);  // P_lo V_hi
                    umma_tf32_ts(d, t0 + 64u + j * 8u, b_lo, idesc_o, 1u);                // P_hi V_lo
                    umma_tf32_ts(d, t0 + 64u + j * 8u, b_hi, idesc_o, 1u);                // P_hi V_hi
                }
                umma_commit(v_empty(buf));
                umma_commit(o_full(buf));
                return true;
            };
            if (ok) ok = issue_s(0);
            for (int kt = 0; kt < n_kt && ok; ++kt) {
                if (kt + 1 < n_kt) ok = issue_s(kt + 1);
                if (ok) ok = issue_pv(kt);
            }
        }
    } else {
        // ------------------------------------------------------------ softmax / correction warps
        const int lane_group = warp & 3;
        const int row = q0 + lane_group * 32 + lane;               // query row of this thread
        const uint32_t t_lane = tmem_base + ((uint32_t)(lane_group * 32) << 16);
        const float c = kLog2e / sqrtf((float)HD);
        float m = -INFINITY, l = 0.f, corr_prev = 0.f;
        float o_reg[HD];
#pragma unroll
        for (int i = 0; i < HD; ++i) o_reg[i] = 0.f;
        bool ok = true;

        auto add_output = [&](int kt, float corr) -> bool {
            const int buf = kt & 1;
            if (!mbar_wait_warp(o_full(buf), (kt >> 1) & 1u, g.err, 17)) return false;
            tc_fence_after();
            uint32_t r0[32], r1[32];
            tmem_ld32(t_lane + buf * 256u + 192u, r0);
            tmem_ld32(t_lane + buf * 256u + 224u, r1);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                o_reg[i] = fmaf(o_reg[i], corr, __uint_as_float(r0[i]));
                o_reg[32 + i] = fmaf(o_reg[32 + i], corr, __uint_as_float(r1[i]));
            }
            return true;
        };

        for (int kt = 0; kt < n_kt && ok; ++kt) {
            const int buf = kt & 1;
            if (!mbar_wait_warp(s_full(buf), (kt >> 1) & 1u, g.err, 18)) { ok = false; break; }
            tc_fence_after();
            uint32_t s0[32], s1[32];
            tmem_ld32(t_lane + buf * 256u, s0);
            tmem_ld32(t_lane + buf * 256u + 32u, s1);
            tmem_ld_wait();
            const int key0 = kt * BKV;
            float mx = -INFINITY;
            if (key0 + BKV - 1 > row) {  // this tile crosses the diagonal for this row
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    if (key0 + i > row) s0[i] = 0xff800000u;        // -inf
                    if (key0 + 32 + i > row) s1[i] = 0xff800000u;
                }
            }
#pragma unroll
            for (int i = 0; i < 32; ++i) mx = fmaxf(mx, fmaxf(__uint_as_float(s0[i]), __uint_as_float(s1[i])));
            const float m_new = fmaxf(m, mx);
            // rows of the second half of the tile see no key of a tile that lies wholly above them:
            // m_new may still be -inf only before the first valid key, which tile 0 always holds
            const float corr = exp2f((m - m_new) * c);
            const float mc = m_new * c;
            float sum = 0.f;
            uint32_t hi[32], lo[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const float p = exp2f(fmaf(__uint_as_float(s0[i]), c, -mc));
                sum += p;
                float fh, fl;
                split_tf32(p, fh, fl);
                hi[i] = __float_as_uint(fh);
                lo[i] = __float_as_uint(fl);
            }
            tmem_st32(t_lane + buf * 256u + 64u, hi);
            tmem_st32(t_lane + buf * 256u + 128u, lo);
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const float p = exp2f(fmaf(__uint_as_float(s1[i]), c, -mc));
                sum += p;
                float fh, fl;
                split_tf32(p, fh, fl);
                hi[i] = __float_as_uint(fh);
                lo[i] = __float_as_uint(fl);
            }
            tmem_st32(t_lane + buf * 256u + 96u, hi);
            tmem_st32(t_lane + buf * 256u + 160u, lo);
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(p_full(buf));
            l = fmaf(l, corr, sum);
            m = m_new;
            // fold in the previous tile's P V while the tensor core works on this one
            if (kt > 0) ok = add_output(kt - 1, corr_prev);
            corr_prev = corr;
        }
        if (ok) ok = add_output(n_kt - 1, corr_prev);
        if (ok && row < g.T) {
            const float inv = 1.0f / l;
            const int64_t off = ((int64_t)(row_base + row)) * g.C + h * HD;
#pragma unroll
            for (int i = 0; i < HD; i += 4) {
                float4 v = make_float4(o_reg[i] * inv, o_reg[i + 1] * inv, o_reg[i + 2] * inv, o_reg[i + 3] * inv);
                store_raw_split(v, g.o ? g.o + off : nullptr, g.o_hi ? g.o_hi + off : nullptr,
                                g.o_lo ? g.o_lo + off : nullptr, i / 4);
            }
            if (g.lse) g.lse[((int64_t)b * g.H + h) * g.T + row] = (m * c + log2f(l)) * kLn2;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

__device__ int g_attn_err_word = 0;  // error word for the per-op entry points (no caller buffer)

bool encode3(CUtensorMap* tm, const float* base, int64_t cols, int64_t rows, int64_t ld, int64_t plane,
             uint32_t box_cols, uint32_t box_rows, CUtensorMapSwizzle sw) {
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc) return false;
    cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, 2};
    cuuint64_t strides[2] = {(cuuint64_t)ld * 4, (cuuint64_t)plane * 4};
    cuuint32_t box[3] = {box_cols, box_rows, 2};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, (void*)base, dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool attention_tc_supports(int head_dim, int C) { return head_dim == 64 && (C % 4) == 0; }

// Device address of the built-in error word (per device), for callers without their own.
cudaError_t attention_tc_default_err(int** out) {
    return cudaGetSymbolAddress((void**)out, g_attn_err_word);
}

cudaError_t launch_attention_fwd_tc(const float* qkv_hi, int64_t qkv_plane, int B, int T, int C, int H, float* o,
                                    float* o_hi, float* o_lo, float* lse, int* err_word, cudaStream_t s) {
    static cudaError_t attr = cudaFuncSetAttribute(attn_fwd_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   (int)kSmemBytes);
    if (attr != cudaSuccess) return attr;
    if (!err_word) {
        cudaError_t e = attention_tc_default_err(&err_word);
        if (e != cudaSuccess) return e;
    }
    CUtensorMap tmQ, tmK, tmV;
    const int64_t rows = (int64_t)B * T, cols = 3 * (int64_t)C;
    bool ok = encode3(&tmQ, qkv_hi, cols, rows, cols, qkv_plane, 32, BQ, CU_TENSOR_MAP_SWIZZLE_128B) &&
              encode3(&tmK, qkv_hi, cols, rows, cols, qkv_plane, 32, BKV, CU_TENSOR_MAP_SWIZZLE_128B) &&
              encode3(&tmV, qkv_hi, cols, rows, cols, qkv_plane, 32, BKV, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B);
    if (!ok) return cudaErrorInvalidValue;
    AttnArgs g{T, C, H, o, o_hi, o_lo, lse, err_word};
    dim3 grid((T + BQ - 1) / BQ, B * H);
    attn_fwd_tc_kernel<<<grid, kThreads, kSmemBytes, s>>>(tmQ, tmK, tmV, g);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

}  // namespace bt
