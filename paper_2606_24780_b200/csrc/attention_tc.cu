// Causal flash attention forward on the 5th-generation tensor cores (head_dim 64), FP32 fidelity
// through 3xTF32 split products.
//
// One CTA owns 128 query rows of one (sequence, head) -- one row per TMEM lane -- and walks the
// 64-key tiles up to the diagonal:
//
//   warps 0-3, 4-7     two softmax / correction warpgroups taking alternate key tiles (buffer b
//                      belongs to warpgroup b), merged at the end; in each, thread i owns query row i.  It reads its 64 scores
//                      with tcgen05.ld (the row maximum and sum need no shuffles), forms
//                      p = exp2((s - m) * scale*log2e), splits p into hi/lo and writes both back to
//                      TMEM with tcgen05.st as the A operand of P V.  The running output is kept in
//                      registers: O_reg = O_reg * corr + O_tile, so no accumulator in TMEM is ever
//                      rescaled.
//   warp 8 (one lane)  TMA producer: Q once, then the K tiles (K-major, 128-byte swizzle) and V
//                      tiles (MN-major, 128-byte swizzle with 32-byte atoms) through one ring of five
//                      slots, each as hi/lo planes straight from the split qkv array the QKV GEMM wrote.
//   warp 9 (one lane)  MMA issuer.  S = Q K^T: 24 tcgen05.mma.kind::tf32 (8 k-steps x 3 split
//                      terms) with both operands in shared memory, accumulator S[buf] in TMEM.
//                      S of tile t+1 is issued before P V of tile t, so the tensor pipe works
//                      while the softmax runs.
//   warp 10 (one lane) second MMA issuer.  O_tile = P V: 24 MMAs with A = P (hi/lo) read from
//                      TENSOR MEMORY and B = V from shared memory, accumulator O[buf] in TMEM.
//
// TMEM map (512 columns): per buffer b in {0,1}: S at 256b, P_hi at 256b+64, P_lo at 256b+128,
// O_tile at 256b+192.  Shared memory: Q 64 KB, five 32 KB tile slots.
// Every mbarrier wait is bounded; a wait that runs out raises the device error word and the CTA
// drains, frees its TMEM and exits.  Every TMA load targets this CTA's own shared memory only.
#include "common.cuh"
#include "tc_common.cuh"

namespace bt {

using namespace tc;

namespace {

constexpr int HD = 64, BQ = 128, BKV = 64;
// Warps 0-7: the two softmax warpgroups (a warp's TMEM lane quadrant is its index mod 4); warp 8: TMA
// producer; warps 9, 10: the two MMA issuers.  (Registers are handed out per four warps: eleven warps
// get the 168 registers per thread that twelve would.)
constexpr int kThreads = 352;
constexpr int kWarpProducer = 8, kWarpMmaS = 9, kWarpMmaO = 10;
constexpr uint32_t kQBytes = 2u * 2u * BQ * 128u;      // 2 k-blocks x (hi, lo) x 128 rows x 128 B
constexpr uint32_t kKVBytes = 2u * 2u * BKV * 128u;    // one K or V tile (hi, lo)
// K and V tiles share one ring of five slots, filled in the order K0 K1 V0 K2 V1 K3 V2 ...: the load
// at position p goes to slot p mod 5 once the load at position p - 5 has been consumed.  K(t) then
// takes over the slot of V(t-4) and V(t) the slot of K(t-1), so a K tile is requested three tile
// periods before its product and a V tile more than one period before its own: a tile load takes
// about 1.5 tile periods to arrive, which a two-deep ring per operand cannot cover.
constexpr int kSlots = 5;
constexpr uint32_t kSmemBytes = 1024u + kQBytes + kSlots * kKVBytes + 256u;
static_assert(kSmemBytes <= 232448u, "shared memory");
__device__ __forceinline__ int pos_k(int t) { return t == 0 ? 0 : 2 * t - 1; }
__device__ __forceinline__ int pos_v(int t) { return 2 * t + 2; }
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct AttnArgs {
    int T, C, H;
    int head_group;   // heads per group of the CTA order (grouped_block)
    float* o;
    float* o_hi;
    float* o_lo;
    float* lse;
    int* err;
    unsigned long long* trace;   // optional timing trace of CTA (0,0) (debug aid, normally null)
};

// trace record: (tag, SM clock); only block (0,0) records
__device__ __forceinline__ void trace_mark(unsigned long long* tr, unsigned long long tag) {
    if (tr == nullptr || blockIdx.x != 0 || blockIdx.y != 0) return;
    const unsigned long long i = atomicAdd(tr, 1ull);
    if (i < 2000) {
        tr[2 + 2 * i] = tag;
        tr[3 + 2 * i] = clock64();
    }
}

__global__ void __launch_bounds__(kThreads, 1)
attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                   const __grid_constant__ CUtensorMap tmV, const AttnArgs g) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t q_s = smem_base;
    const uint32_t ring_s = q_s + kQBytes;         // kSlots tiles
    const uint32_t bars = ring_s + kSlots * kKVBytes;
    // barrier slots
    const uint32_t q_full = bars;
    auto slot_full = [&](int i) { return bars + 8u * (1 + i); };
    auto slot_empty = [&](int i) { return bars + 8u * (6 + i); };
    auto s_full = [&](int b) { return bars + 8u * (11 + b); };
    auto p_full = [&](int b) { return bars + 8u * (13 + b); };
    auto o_full = [&](int b) { return bars + 8u * (15 + b); };
    const uint32_t merge_full = bars + 8u * 17;
    const uint32_t all_done = bars + 8u * 18;
    const uint32_t tmem_slot = bars + 8u * 19;
    volatile uint32_t* tmem_slot_ptr =
        reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - smem_u32(smem_raw)));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int bh, yb;
    grouped_block(g.head_group, bh, yb);
    const int qt = gridDim.y - 1 - yb;                   // heaviest query tiles first, over the heads of a group
    const int b = bh / g.H, h = bh % g.H;
    const int q0 = qt * BQ;
    const int last_row = min(q0 + BQ - 1, g.T - 1);
    const int n_kt = last_row / BKV + 1;
    const int row_base = b * g.T;                         // row of this sequence in the [B*T, 3C] array

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int i = 0; i < kSlots; ++i) {
            mbar_init(slot_full(i), 1);
            mbar_init(slot_empty(i), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(s_full(i), 1);
            mbar_init(p_full(i), 4);
            mbar_init(o_full(i), 1);
        }
        mbar_init(merge_full, 4);
        mbar_init(all_done, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kWarpMmaS) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(512u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot_ptr;
    pdl_wait();      // set-up done; global memory is touched from here on
    pdl_trigger();

    if (warp == kWarpProducer) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            mbar_expect_tx(q_full, kQBytes);
            for (int kb = 0; kb < 2; ++kb)
                tma_load_3d(q_s + kb * (kQBytes / 2), &tmQ, q_full, h * HD + kb * 32, row_base + q0, 0);
            bool ok = true;
            const int n_pos = pos_v(n_kt - 1) + 1;
            int slot = 0;
            uint32_t round = 0;                          // p / kSlots
            for (int p = 0; p < n_pos && ok; ++p) {
                const bool is_k = p == 0 || (p & 1);
                const int t = p == 0 ? 0 : (is_k ? (p + 1) >> 1 : (p - 2) >> 1);
                if (t < n_kt) {                          // only K(n_kt) near the end falls outside
                    if (!mbar_wait(slot_empty(slot), (round & 1u) ^ 1u, g.err, is_k ? 11 : 12)) { ok = false; break; }
                    mbar_expect_tx(slot_full(slot), kKVBytes);
                    const uint32_t dst = ring_s + (uint32_t)slot * kKVBytes;
                    for (int kb = 0; kb < 2; ++kb)
                        tma_load_3d(dst + kb * (kKVBytes / 2), is_k ? &tmK : &tmV, slot_full(slot),
                                    (is_k ? g.C : 2 * g.C) + h * HD + kb * 32, row_base + t * BKV, 0);
                }
                if (++slot == kSlots) { slot = 0; ++round; }
            }
            if (!ok)
                for (int i = 0; i < 2000; ++i) __nanosleep(1000);  // let loads in flight land
        }
    } else if (warp == kWarpMmaS) {
        // ------------------------------------------------------------ MMA issuer 1: S = Q K^T
        if (lane == 0) {
            constexpr uint32_t idesc_s = make_idesc_tf32(BQ, BKV, false, false);
            bool ok = mbar_wait(q_full, 0, g.err, 13);
            const DescBase qd = make_desc_base(q_s, 16u, 1024u, 2u);
            for (int kt = 0; kt < n_kt && ok; ++kt) {
                const int buf = kt & 1;
                const int pk = pos_k(kt), slot = pk % kSlots;
                if (!mbar_wait(slot_full(slot), (uint32_t)(pk / kSlots) & 1u, g.err, 14)) { ok = false; break; }
                // S[buf] is free once the softmax of tile kt-2 has read it (it then publishes P)
                if (kt >= 2 && !mbar_wait(p_full(buf), ((kt - 2) >> 1) & 1u, g.err, 20)) { ok = false; break; }
                tc_fence_after();
                trace_mark(g.trace, 100 + kt);
                const uint32_t d = tmem_base + (uint32_t)buf * 256u;
                const DescBase kd = make_desc_base(ring_s + (uint32_t)slot * kKVBytes, 16u, 1024u, 2u);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t qo = (uint32_t)(ks >> 2) * (kQBytes / 2) + (uint32_t)(ks & 3) * 32u;
                    const uint32_t ko = (uint32_t)(ks >> 2) * (kKVBytes / 2) + (uint32_t)(ks & 3) * 32u;
                    const uint64_t a_hi = qd.at(qo), a_lo = qd.at(qo + BQ * 128u);
                    const uint64_t b_hi = kd.at(ko), b_lo = kd.at(ko + BKV * 128u);
                    umma_tf32(d, a_lo, b_hi, idesc_s, ks > 0 ? 1u : 0u);
                    umma_tf32(d, a_hi, b_lo, idesc_s, 1u);
                    umma_tf32(d, a_hi, b_hi, idesc_s, 1u);
                }
                umma_commit(slot_empty(slot));
                umma_commit(s_full(buf));
                trace_mark(g.trace, 200 + kt);
            }
        }
    } else if (warp == kWarpMmaO) {
        // ------------------------------------------------------------ MMA issuer 2: O_tile = P V
        // A second issuing thread: the two products of a tile go to different accumulators and are
        // ordered only through the barriers, so their instruction streams can be issued in parallel.
        if (lane == 0) {
            constexpr uint32_t idesc_o = make_idesc_tf32(BQ, HD, false, true);
            bool ok = true;
            for (int kt = 0; kt < n_kt && ok; ++kt) {
                const int buf = kt & 1;
                // P(kt) published; the softmax warps read O[buf] of tile kt-2 before publishing it
                if (!mbar_wait(p_full(buf), (kt >> 1) & 1u, g.err, 15)) { ok = false; break; }
                const int pv = pos_v(kt), slot = pv % kSlots;
                if (!mbar_wait(slot_full(slot), (uint32_t)(pv / kSlots) & 1u, g.err, 16)) { ok = false; break; }
                tc_fence_after();
                trace_mark(g.trace, 300 + kt);
                const uint32_t t0 = tmem_base + (uint32_t)buf * 256u;
                const uint32_t d = t0 + 192u;
                const DescBase vd = make_desc_base(ring_s + (uint32_t)slot * kKVBytes, kKVBytes / 2, 512u, 1u);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint64_t b_hi = vd.at(j * 1024u), b_lo = vd.at(BKV * 128u + j * 1024u);
                    umma_tf32_ts(d, t0 + 128u + j * 8u, b_hi, idesc_o, j > 0 ? 1u : 0u);  // P_lo V_hi
                    umma_tf32_ts(d, t0 + 64u + j * 8u, b_lo, idesc_o, 1u);                // P_hi V_lo
                    umma_tf32_ts(d, t0 + 64u + j * 8u, b_hi, idesc_o, 1u);                // P_hi V_hi
                }
                umma_commit(slot_empty(slot));
                umma_commit(o_full(buf));
                trace_mark(g.trace, 400 + kt);
            }
            if (ok) umma_commit(all_done);
        }
    } else if (warp < 8) {
        // ------------------------------------------------------------ softmax / correction warps
        // Two warpgroups (warps 0-3 and 4-7) take alternate key tiles, each with its own running
        // maximum, sum and output; they are merged at the end.  Two warps per scheduler hide each
        // other's instruction latencies.
        const int wg = warp >> 2;                                    // 0 or 1; owns TMEM buffer wg
        const int lane_group = warp & 3;
        const int rloc = lane_group * 32 + lane;                    // row inside the CTA
        const int row = q0 + rloc;                                   // query row of this thread
        const uint32_t t_lane = tmem_base + ((uint32_t)(lane_group * 32) << 16) + (uint32_t)wg * 256u;
        const float c = kLog2e / sqrtf((float)HD);
        float m = -INFINITY, l = 0.f, corr_prev = 0.f;
        float o_reg[HD];
#pragma unroll
        for (int i = 0; i < HD; ++i) o_reg[i] = 0.f;
        bool ok = true;

        auto add_output = [&](int kt, float corr) -> bool {
            if (!mbar_wait_warp(o_full(wg), (kt >> 1) & 1u, g.err, 17)) return false;
            tc_fence_after();
            uint32_t r0[32], r1[32];
            tmem_ld32(t_lane + 192u, r0);
            tmem_ld32(t_lane + 224u, r1);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                o_reg[i] = fmaf(o_reg[i], corr, __uint_as_float(r0[i]));
                o_reg[32 + i] = fmaf(o_reg[32 + i], corr, __uint_as_float(r1[i]));
            }
            return true;
        };

        int last = -1;
        for (int kt = wg; kt < n_kt && ok; kt += 2) {
            // fold in this warpgroup's previous tile first: O[wg] must have been read before P of
            // this tile is published (the P V product of this tile overwrites O[wg])
            if (last >= 0 && !add_output(last, corr_prev)) { ok = false; break; }
            if (rloc == 0) trace_mark(g.trace, 500 + kt);
            if (!mbar_wait_warp(s_full(wg), (kt >> 1) & 1u, g.err, 18)) { ok = false; break; }
            tc_fence_after();
            if (rloc == 0) trace_mark(g.trace, 600 + kt);
            uint32_t s0[32], s1[32];
            tmem_ld32(t_lane, s0);
            tmem_ld32(t_lane + 32u, s1);
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
            // a tile that lies wholly above a row leaves its maximum at -inf; keep the arithmetic finite
            const float m_new = fmaxf(m, mx);
            const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
            const float corr = ex2_approx((m - m_use) * c);           // m = -inf -> 0
            const float mc = m_use * c;
            float sum = 0.f;
            uint32_t hi[32], lo[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const float p = ex2_approx(fmaf(__uint_as_float(s0[i]), c, -mc));
                sum += p;
                split_tf32_int(p, hi[i], lo[i]);
            }
            tmem_st32(t_lane + 64u, hi);
            tmem_st32(t_lane + 128u, lo);
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const float p = ex2_approx(fmaf(__uint_as_float(s1[i]), c, -mc));
                sum += p;
                split_tf32_int(p, hi[i], lo[i]);
            }
            tmem_st32(t_lane + 96u, hi);
            tmem_st32(t_lane + 160u, lo);
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(p_full(wg));
            if (rloc == 0) trace_mark(g.trace, 700 + kt);
            l = fmaf(l, corr, sum);
            m = m_new;
            corr_prev = corr;
            last = kt;
        }
        if (ok && last >= 0) ok = add_output(last, corr_prev);

        // merge: warpgroup 1 hands (m, l, O) of its rows to warpgroup 0 through the first ring slots,
        // which are idle once every tile's products have completed
        float* xch = reinterpret_cast<float*>(smem_raw + (ring_s - smem_u32(smem_raw)));   // [128][66]
        if (wg == 1) {
            if (ok) ok = mbar_wait_warp(all_done, 0, g.err, 21);   // no product still reads the K buffers
            float* dst = xch + rloc * 66;
            dst[64] = m;
            dst[65] = l;
#pragma unroll
            for (int i = 0; i < HD; ++i) dst[i] = o_reg[i];
            __threadfence_block();
            __syncwarp();
            if (lane == 0) mbar_arrive(merge_full);
        } else {
            if (ok) ok = mbar_wait_warp(merge_full, 0, g.err, 19);
            if (ok) {
                const float* src = xch + rloc * 66;
                const float m1 = src[64], l1 = src[65];
                const float mm = fmaxf(m, m1);                      // finite: tile 0 belongs to warpgroup 0
                const float f0 = ex2_approx((m - mm) * c), f1 = ex2_approx((m1 - mm) * c);
                l = l * f0 + l1 * f1;
                m = mm;
#pragma unroll
                for (int i = 0; i < HD; ++i) o_reg[i] = o_reg[i] * f0 + src[i] * f1;
                // the rows leave in full 128-byte segments through a slice of the idle third ring slot
                const float inv = 1.0f / l;
                const int wrow0 = q0 + lane_group * 32;                 // first query row of this warp
                const int nvalid = max(0, min(32, g.T - wrow0));
                const int64_t off0 = ((int64_t)(row_base + wrow0)) * g.C + h * HD;
                float* tile = reinterpret_cast<float*>(smem_raw + (ring_s + 2u * kKVBytes - smem_u32(smem_raw)) + (uint32_t)lane_group * kRowTileBytes);
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    float v[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = o_reg[half * 32 + i] * inv;
                    warp_rows_store(v, tile, lane, nvalid, g.o ? g.o + off0 + half * 32 : nullptr,
                                    g.o_hi ? g.o_hi + off0 + half * 32 : nullptr, g.o_lo ? g.o_lo + off0 + half * 32 : nullptr,
                                    g.C, nullptr);
                }
                if (row < g.T && g.lse) g.lse[((int64_t)b * g.H + h) * g.T + row] = (m * c + log2f(l)) * kLn2;
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kWarpMmaS) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

unsigned long long* g_trace_ptr = nullptr;   // set through bt_debug_set_attention_trace
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

void attention_tc_set_trace(unsigned long long* p) { g_trace_ptr = p; }
unsigned long long* attention_tc_get_trace() { return g_trace_ptr; }

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
    AttnArgs g{T, C, H, attn_head_group(B * H, (T + BQ - 1) / BQ), o, o_hi, o_lo, lse, err_word, g_trace_ptr};
    dim3 grid(B * H, (T + BQ - 1) / BQ);
    BT_KERNEL_LAUNCH((attn_fwd_tc_kernel), grid, kThreads, kSmemBytes, s, tmQ, tmK, tmV, g);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

}  // namespace bt
