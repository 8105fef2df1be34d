// Causal flash attention backward on the 5th-generation tensor cores (head_dim 64), 3xTF32.
//
// Two deterministic kernels (no atomics) that recompute the probabilities from (q, k, lse):
//
//   dkv kernel  one CTA owns 128 keys (one per TMEM lane) of one (sequence, head) and walks the
//               64-row query tiles at or below the diagonal:
//                 S^T  = K' Q^T      A = K' (pre-scaled, hi/lo) held in TENSOR MEMORY, B = Q tile (smem)
//                 dP^T = V  dO^T     A = V (smem, resident),                           B = dO tile
//                 P^T  = exp2(S^T - lse),  dS^T = P^T o (dP^T - D)       (thread = key row)
//                 dV  += P^T  dO     A = P^T  (hi/lo written back to tensor memory),   B = dO tile
//                 dK  += dS^T Q      A = dS^T (tensor memory),                          B = Q tile
//               dK and dV accumulate in tensor memory over the whole walk (the backward needs no
//               running-max rescaling).  The walk runs from the LAST query tile down to the diagonal:
//               the tensor core adds into its FP32 accumulator with truncation, so a long chain of
//               small additions to an already large sum drifts toward zero (about n * 2^-25 after
//               n MMAs); probabilities of a key usually decay with the query's distance, and adding
//               the small far-away terms first keeps that drift relative to a small sum.
//   dq kernel   one CTA owns 128 query rows and walks the 64-key tiles up to the diagonal:
//                 S  = Q' K^T (A = Q' in tensor memory),  dP = dO V^T (A = dO resident in smem),
//                 dS = P o (dP - D),  dQ += dS K (A = dS in tensor memory).
//
// Streamed tiles arrive by TMA as hi/lo planes in the two shared-memory layouts the tensor core
// needs: K-major (128-byte swizzle) where the tile is the B operand of a "row . row" product, and
// MN-major (128-byte swizzle, 32-byte atoms) where its rows are the contraction index.  The two
// layouts have their own full/empty barriers, so a tile's K-major half is refilled as soon as the
// first pair of products has consumed it.
//
// Issuing threads.  One thread issues a tcgen05.mma about every 57 clocks whatever its shape, while
// an N = 64 product occupies the pipe for 32 clocks when its A operand comes from tensor memory
// (48 from shared memory).  The products are therefore spread over several issuing threads, each
// owning whole products and a chain of tensor-memory regions of its own: in the dkv kernel warp 1
// issues S^T(t+1) right behind dV(t) (same regions: the pipe runs one thread's MMAs in order) and
// warp 10 dP^T(t+1) behind dK(t); in the dq kernel warps 1, 10 and 11 issue S, dP and dQ, and the
// two score products of tile t + 2 wait on a barrier for the dQ product of tile t to have read the
// buffer they overwrite.  The chains meet only in mbarriers.
// Every mbarrier wait is bounded and reports through the device error word; the polling loop is
// out of line and the long run-once sequences have one copy each, because these kernels are
// large (90 and 101 KB of code) and every CTA start runs through them with a cold instruction cache.
#include "common.cuh"
#include "tc_common.cuh"

namespace bt {

using namespace tc;

unsigned long long* attention_tc_get_trace();

namespace {

constexpr int HD = 64, BR = 128, BT_ = 32;  // head dim, rows owned by the CTA, streamed tile rows
constexpr int kThreads = 320;   // TMA warp, MMA warp, two element-wise warpgroups (alternate tiles)
// One thread issues a tcgen05.mma about every 55-59 clocks, whatever its shape; an N = 64 product
// whose A operand comes from tensor memory occupies the pipe for 32.  The kernels below therefore
// spread their products over several issuing threads (one lane each of warps 1, 10 and, in the dq
// kernel, 11), every thread owning whole products and a chain of regions of its own, ordered
// against the others only through mbarriers.
constexpr int kThreadsDkv = 352, kThreadsDq = 384;
constexpr int kWarpMma2 = 10, kWarpMma3 = 11;
constexpr float kLog2e = 1.4426950408889634f;
constexpr uint32_t kResBytes = 2u * 2u * BR * 128u;   // resident 128-row operand: 2 k-blocks x (hi,lo)
constexpr uint32_t kTileBytes = 2u * 2u * BT_ * 128u; // one streamed 32-row tile in one layout (16 KB)

// Per-CTA (start, end, SM, tiles) record behind the mark regions of the trace buffer (debug aid).
__device__ __forceinline__ void trace_cta(unsigned long long* tr, int kernel_index, int slot, unsigned long long v) {
    if (tr == nullptr) return;
    const unsigned long long n = (unsigned long long)gridDim.x * gridDim.y;
    const unsigned long long id = (unsigned long long)blockIdx.y * gridDim.x + blockIdx.x;
    tr[4002 + 4 * (kernel_index * n + id) + slot] = v;
}
__device__ __forceinline__ unsigned smid() {
    unsigned r;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(r));
    return r;
}

// The 64 accumulator columns of the warp's 32 rows (times mul) -> hi/lo planes in global memory,
// in full 128-byte row segments (see warp_rows_store).  The tensor-memory loads are .sync.aligned:
// EVERY lane of the warp must call this.  hi0 / lo0: row 0 of the warp, column 0 of the head;
// nvalid: rows of the warp inside the sequence; sums (nullable): 64 column sums over those rows.
// PAIRS: the accumulator is 128 columns wide and output columns 32 h .. 32 h + 31 are the sum of its
// columns 64 h .. 64 h + 31 and 64 h + 32 .. 64 h + 63 (the halves of a split product, see the dq kernel).
template <bool PAIRS = false>
__device__ __forceinline__ void tmem_rows_to_split(uint32_t t_row, float mul, float* hi0, float* lo0,
                                                   long long row_stride, int nvalid, float* sums, float* tile,
                                                   int lane) {
#pragma unroll 1   // the body is long and runs once per CTA: keep one copy of it
    for (int half = 0; half < 2; ++half) {
        uint32_t r[32];
        float v[32];
        if (PAIRS) {
            uint32_t r2[32];
            tmem_ld32(t_row + half * 64, r);
            tmem_ld32(t_row + half * 64 + 32, r2);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = (__uint_as_float(r[i]) + __uint_as_float(r2[i])) * mul;
        } else {
            tmem_ld32(t_row + half * 32, r);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]) * mul;
        }
        warp_rows_store(v, tile, lane, nvalid, nullptr, hi0 + half * 32, lo0 + half * 32, row_stride,
                        sums ? sums + half * 32 : nullptr);
    }
}

// Byte offsets of one 8-deep k-step inside an operand tile (compile-time after unrolling).
//  MN-major 32-row tile (2 column groups of [hi|lo][32 rows][128 B]), contraction over the rows.
__device__ __forceinline__ constexpr uint32_t mnmaj_off(int ks, bool lo) {
    return (lo ? BT_ * 128u : 0u) + (uint32_t)ks * 1024u;
}
__device__ __forceinline__ DescBase mnmaj_base(uint32_t tile) { return make_desc_base(tile, 2u * BT_ * 128u, 512u, 1u); }

// D = rowsum(dO o O) over one head's 64 columns for the warp's 32 rows; lane r returns row r's value.
// The rows are read as they lie in memory (8 lanes x 16 bytes = one 128-byte segment), four rows of
// all planes in flight per lane; a 3-step butterfly adds the 8 column slices of a row, 8 shuffles
// bring row r's sum to lane r.  a = O (a_lo nullable), b = dO as hi/lo planes; rows >= nvalid read
// the last valid row.
__device__ __forceinline__ float warp_rows_dot64(const float* a_hi, const float* a_lo, const float* b_hi,
                                                 const float* b_lo, long long row_stride, int nvalid, int lane) {
    const int sub = lane >> 3, cq = lane & 7;
    float acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
#pragma unroll
        for (int g4 = 0; g4 < 2; ++g4) {
            float4 x[4], y[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int r = max(0, min(sub + 4 * (4 * g4 + j), nvalid - 1));
                const long long off = (long long)r * row_stride + half * 32 + 4 * cq;
                x[j] = *reinterpret_cast<const float4*>(a_hi + off);
                if (a_lo) x[j] = add4(x[j], *reinterpret_cast<const float4*>(a_lo + off));
                y[j] = add4(*reinterpret_cast<const float4*>(b_hi + off), *reinterpret_cast<const float4*>(b_lo + off));
            }
#pragma unroll
            for (int j = 0; j < 4; ++j)
                acc[4 * g4 + j] += (x[j].x * y[j].x + x[j].y * y[j].y) + (x[j].z * y[j].z + x[j].w * y[j].w);
        }
    }
    float d = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float v = acc[i];
        v += __shfl_xor_sync(0xffffffffu, v, 1);
        v += __shfl_xor_sync(0xffffffffu, v, 2);
        v += __shfl_xor_sync(0xffffffffu, v, 4);
        v = __shfl_sync(0xffffffffu, v, 8 * (lane & 3));     // row sub + 4 i lives in the lanes of slice `sub`
        if ((lane >> 2) == i) d = v;                          // lane r wants row r = (r & 3) + 4 (r >> 2)
    }
    return d;
}

struct BwdArgs {
    int T, C, H;
    int head_group;           // heads per group of the CTA order (grouped_block)
    const float* qkv_hi;      // split qkv [2][B*T][3C]
    long long qkv_plane;
    const float* lse;
    const float* dvec;        // [B, H, T] rowsum(dO o O): written by the dq kernel, read by the dkv kernel
    float* dvec_out;          // the same array, for the dq kernel
    const float* o_hi;        // attention output [B*T][C] (raw, or the hi plane with o_lo the lo plane)
    const float* o_lo;        // nullable
    const float* do_hi;       // split output gradient [2][B*T][C]
    long long do_plane;
    float* dqkv_hi;           // split output [2][B*T][3C]
    long long dqkv_plane;
    int* err;
    unsigned long long* trace;   // optional timing trace of CTA (0,0) (debug aid, normally null)
    float* rg_sums;           // optional [B * nrg][3C]: column sums of dqkv over each 32-row group
    int nrg;                  // 32-row groups per sequence (4 per 128-row block)
};

// trace record: (tag, SM clock) in the recording role's own region (no atomics, so a mark costs
// a few instructions); only block (0,0) records
constexpr int kTraceRegion = 500;
static __device__ __noinline__ void trace_mark(unsigned long long* tr, int role, int& n, unsigned long long tag) {
    if (tr == nullptr || blockIdx.x != 0 || blockIdx.y != 0) return;
    if (n < kTraceRegion) {
        unsigned long long* p = tr + 2 + 2 * (role * kTraceRegion + n);
        p[0] = tag;
        p[1] = clock64();
        ++n;
    }
}

// Shared prologue: barriers + TMEM allocation.  Returns the TMEM base address.
__device__ __forceinline__ uint32_t setup(uint32_t bars, int n_bars_count1, uint32_t p_bar0, int n_p_bars,
                                          uint32_t tmem_slot, uint8_t* smem_raw, int warp, uint32_t two_mask = 0u) {
    if (threadIdx.x == 0) {
        for (int i = 0; i < n_bars_count1; ++i) mbar_init(bars + 8u * i, ((two_mask >> i) & 1u) ? 2 : 1);
        for (int i = 0; i < n_p_bars; ++i) mbar_init(p_bar0 + 8u * i, 4);
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
    return *reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - smem_u32(smem_raw)));
}

// ------------------------------------------------------------------------------------------ dkv
//
// 64-row query tiles, single score buffers, and an issue order that still keeps the tensor pipe fed:
//     ... dV(t) | S^T(t+1) | dK(t) | dP^T(t+1) | dV(t+1) | S^T(t+2) | ...
// S^T/P^T live in one pair of tensor-memory regions, dP^T/dS^T in another; the group that
// overwrites a region is issued right after the group that last read it, and while the pipe
// runs the two groups of the other region the 256 element-wise threads turn S^T into P^T (or
// dP^T into dS^T).  N = 64 for every product (an MMA costs the same ~50 clocks for N = 32), so a
// 64 x 128 tile takes 96 MMAs where two 32-row tiles took 144.
//   tensor memory: K' hi|lo 0-127, dK 128-191, dV 192-255, S^T -> P^T_hi 256-319, P^T_lo 320-383,
//                  dP^T -> dS^T_hi 384-447, dS^T_lo 448-511
//   shared memory: V (128 keys, K-major, resident) 64 KB; one 32 KB buffer each for the query
//                  tile's Q and dO in the K-major layout (B of S^T, dP^T) and in the MN-major layout
//                  (B of dK, dV); every buffer has its own full/empty barriers and is refilled as
//                  soon as the one product that reads it has completed.
constexpr int BT64 = 64;
constexpr uint32_t kTile64 = 2u * 2u * BT64 * 128u;   // one 64-row tile in one layout (32 KB)
constexpr uint32_t kDkvSmem = 1024u + kResBytes + 4u * kTile64 + 256u + 4u * kRowTileBytes + 1024u;   // + K' staging tiles, + row statistics
__device__ __forceinline__ constexpr uint32_t mn64_off(int ks, bool lo) { return (lo ? BT64 * 128u : 0u) + (uint32_t)ks * 1024u; }
__device__ __forceinline__ DescBase mn64_base(uint32_t tile) { return make_desc_base(tile, 2u * BT64 * 128u, 512u, 1u); }

__global__ void __launch_bounds__(kThreadsDkv, 1)
attn_bwd_dkv_tc_kernel(const __grid_constant__ CUtensorMap tmQk, const __grid_constant__ CUtensorMap tmQm,
                       const __grid_constant__ CUtensorMap tmDOk, const __grid_constant__ CUtensorMap tmDOm,
                       const __grid_constant__ CUtensorMap tmVres, const BwdArgs g) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t v_s = base;                                  // resident V (A operand of dP^T)
    const uint32_t qk_s = base + kResBytes, dok_s = qk_s + kTile64, dom_s = dok_s + kTile64, qm_s = dom_s + kTile64;
    const uint32_t bars = qm_s + kTile64;
    enum { V_FULL = 0, QK_FULL, QK_EMPTY, DOK_FULL, DOK_EMPTY, DOM_FULL, DOM_EMPTY, QM_FULL, QM_EMPTY, S_FULL,
           DP_FULL, ACC_FULL, P_READY, DS_READY, K_READY, STAT_READY, N_BARS };
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
    const uint32_t tmem_slot = bars + 8u * N_BARS;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // grid = (sequence x head, key block): blocks are dispatched x-fastest, so all the key blocks
    // with the longest walks (low j0) start first and the short ones fill the tail
    int bh, yb;
    grouped_block(g.head_group, bh, yb);
    const int b = bh / g.H, h = bh % g.H;
    const int j0 = yb * BR;
    const int row_base = b * g.T;
    const int n_qt = (g.T + BT64 - 1) / BT64, qt0 = j0 / BT64;
    const int n_t = n_qt - qt0;
    if (threadIdx.x == 0) {
        trace_cta(g.trace, 0, 0, globaltimer_ns());
        trace_cta(g.trace, 0, 2, smid());
        trace_cta(g.trace, 0, 3, n_t);
    }

    if (threadIdx.x == 0) {
        for (int i = 0; i < P_READY; ++i) mbar_init(bar(i), i == ACC_FULL ? 2 : 1);   // both issuing threads commit at the end
        mbar_init(bar(P_READY), 8);      // both element-wise warpgroups (8 warps) write every tile
        mbar_init(bar(DS_READY), 8);
        mbar_init(bar(K_READY), 4);
        mbar_init(bar(STAT_READY), 4);
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
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - smem_u32(smem_raw)));
    pdl_wait();      // set-up done; global memory is touched from here on
    pdl_trigger();
    const uint32_t tK_hi = tmem, tK_lo = tmem + 64, tdK = tmem + 128, tdV = tmem + 192;
    const uint32_t tS = tmem + 256, tPlo = tmem + 320, tdP = tmem + 384, tdSlo = tmem + 448;
    // tile t of the walk is query tile n_qt - 1 - t: from the last query tile down to the diagonal
    // (the tensor core adds into its FP32 accumulator with truncation; adding the small far-away
    // terms first keeps the drift of a long accumulation relative to a small sum)
    auto q_row0 = [&](int t) { return (n_qt - 1 - t) * BT64; };

    if (warp == 0) {
        if (lane == 0) {
            mbar_expect_tx(bar(V_FULL), kResBytes);
            for (int kb = 0; kb < 2; ++kb)
                tma_load_3d(v_s + kb * (kResBytes / 2), &tmVres, bar(V_FULL), 2 * g.C + h * HD + kb * 32, row_base + j0, 0);
            bool ok = true;
            // one buffer per (tensor, layout); t = the tile whose data goes in
            auto load = [&](uint32_t dst, const CUtensorMap* tm, int full, int empty, int t) -> bool {
                if (!mbar_wait_ool(bar(empty), (uint32_t)(t & 1) ^ 1u, g.err, 21)) return false;
                mbar_expect_tx(bar(full), kTile64);
                for (int part = 0; part < 2; ++part)
                    tma_load_3d(dst + part * (kTile64 / 2), tm, bar(full), h * HD + part * 32, row_base + q_row0(t), 0);
                return true;
            };
            // in the order the products consume them: S^T(0), dP^T(0), then per tile dV(t), S^T(t+1), dK(t),
            // dP^T(t+1) -- as a schedule walked by one loop, so that the load sequence exists once
            for (int i = 0; i < 4 * n_t + 2 && ok; ++i) {
                // j: 0 dO MN-major (t), 1 Q K-major (t+1), 2 Q MN-major (t), 3 dO K-major (t+1); first Q(0), dO(0) K-major
                const int j = i == 0 ? 1 : i == 1 ? 3 : (i - 2) & 3;
                const int tt = i < 2 ? 0 : ((i - 2) >> 2) + (j & 1);
                if (tt >= n_t) continue;
                const uint32_t dst = j == 0 ? dom_s : j == 1 ? qk_s : j == 2 ? qm_s : dok_s;
                const CUtensorMap* tm = j == 0 ? &tmDOm : j == 1 ? &tmQk : j == 2 ? &tmQm : &tmDOk;
                const int full = j == 0 ? DOM_FULL : j == 1 ? QK_FULL : j == 2 ? QM_FULL : DOK_FULL;
                ok = load(dst, tm, full, full + 1, tt);      // every EMPTY barrier follows its FULL barrier
            }
            if (!ok)
                for (int i = 0; i < 2000; ++i) __nanosleep(1000);
        }
    } else if (warp == 1 || warp == kWarpMma2) {
        if (lane == 0) {
            constexpr uint32_t idesc_a = make_idesc_tf32(BR, BT64, false, false);  // 128 x 64, B K-major
            constexpr uint32_t idesc_a2 = make_idesc_tf32(BR, 2 * BT64, false, false);  // 128 x 128: B = [hi rows | lo rows]
            constexpr uint32_t idesc_b = make_idesc_tf32(BR, HD, false, true);     // 128 x 64, B MN-major
            // warp 1: the S^T -> P^T -> dV chain (regions tS, tPlo, tdV); warp 10: dP^T -> dS^T -> dK
            const bool score_chain = warp == 1;
            const int trole = score_chain ? 0 : 3;   // region of the debug trace
            bool ok = score_chain ? mbar_wait_ool(bar(K_READY), 0, g.err, 24) : mbar_wait_ool(bar(V_FULL), 0, g.err, 23);
            int tn = 0;
            const DescBase vd = kmaj_base(v_s), qd = kmaj_base(qk_s), od = kmaj_base(dok_s);
            const DescBase omd = mn64_base(dom_s), qmd = mn64_base(qm_s);
            auto issue_s = [&](int t) -> bool {      // S^T(t) = K' Q^T
                if (!mbar_wait_ool(bar(QK_FULL), (uint32_t)(t & 1), g.err, 25)) return false;
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    // the tile's lo rows follow its hi rows: [Q_hi | Q_lo] is one 128-row operand, and the
                    // product's two halves land in the S^T and the P^T_lo columns (added when they are read)
                    const uint64_t q_hl = qd.at(kmaj_off(BT64, ks, false));
                    umma_tf32_ts(tS, tK_hi + ks * 8, q_hl, idesc_a2, ks > 0 ? 1u : 0u);   // K'_hi Q_hi | K'_hi Q_lo
                    umma_tf32_ts(tS, tK_lo + ks * 8, q_hl, idesc_a, 1u);                  // + K'_lo Q_hi
                }
                umma_commit(bar(QK_EMPTY));
                umma_commit(bar(S_FULL));
                trace_mark(g.trace, trole, tn, 100 + t);
                return true;
            };
            auto issue_dp = [&](int t) -> bool {     // dP^T(t) = V dO^T
                if (!mbar_wait_ool(bar(DOK_FULL), (uint32_t)(t & 1), g.err, 26)) return false;
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t v_hi = vd.at(kmaj_off(BR, ks, false)), v_lo = vd.at(kmaj_off(BR, ks, true));
                    const uint64_t o_hl = od.at(kmaj_off(BT64, ks, false));
                    umma_tf32(tdP, v_hi, o_hl, idesc_a2, ks > 0 ? 1u : 0u);   // V_hi dO_hi | V_hi dO_lo
                    umma_tf32(tdP, v_lo, o_hl, idesc_a, 1u);                  // + V_lo dO_hi
                }
                umma_commit(bar(DOK_EMPTY));
                umma_commit(bar(DP_FULL));
                trace_mark(g.trace, trole, tn, 200 + t);
                return true;
            };
            auto issue_dv = [&](int t) -> bool {     // dV += P^T(t) dO
                if (!mbar_wait_ool(bar(P_READY), (uint32_t)(t & 1), g.err, 27)) return false;
                if (!mbar_wait_ool(bar(DOM_FULL), (uint32_t)(t & 1), g.err, 28)) return false;
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t o_hi = omd.at(mn64_off(ks, false)), o_lo = omd.at(mn64_off(ks, true));
                    const uint32_t acc = (t > 0 || ks > 0) ? 1u : 0u;
                    umma_tf32_ts(tdV, tPlo + ks * 8, o_hi, idesc_b, acc);
                    umma_tf32_ts(tdV, tS + ks * 8, o_lo, idesc_b, 1u);
                    umma_tf32_ts(tdV, tS + ks * 8, o_hi, idesc_b, 1u);
                }
                umma_commit(bar(DOM_EMPTY));
                trace_mark(g.trace, trole, tn, 300 + t);
                return true;
            };
            auto issue_dk = [&](int t) -> bool {     // dK += dS^T(t) Q
                if (!mbar_wait_ool(bar(DS_READY), (uint32_t)(t & 1), g.err, 29)) return false;
                if (!mbar_wait_ool(bar(QM_FULL), (uint32_t)(t & 1), g.err, 30)) return false;
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t q_hi = qmd.at(mn64_off(ks, false)), q_lo = qmd.at(mn64_off(ks, true));
                    const uint32_t acc = (t > 0 || ks > 0) ? 1u : 0u;
                    umma_tf32_ts(tdK, tdSlo + ks * 8, q_hi, idesc_b, acc);
                    umma_tf32_ts(tdK, tdP + ks * 8, q_lo, idesc_b, 1u);
                    umma_tf32_ts(tdK, tdP + ks * 8, q_hi, idesc_b, 1u);
                }
                umma_commit(bar(QM_EMPTY));
                trace_mark(g.trace, trole, tn, 400 + t);
                return true;
            };
            // Within a chain the product that overwrites a region follows the product that last read it
            // in this thread's own program order (the pipe executes a thread's MMAs in order); the two
            // chains share no region.
            // (one call site per product: the unrolled issue sequences are large)
            if (score_chain) {
                for (int t = 0; t <= n_t && ok; ++t) {
                    if (t > 0) ok = issue_dv(t - 1);               // frees the S^T / P^T regions ...
                    if (ok && t < n_t) ok = issue_s(t);            // ... which the next scores overwrite
                }
            } else {
                for (int t = 0; t <= n_t && ok; ++t) {
                    if (t > 0) ok = issue_dk(t - 1);               // frees the dP^T / dS^T regions ...
                    if (ok && t < n_t) ok = issue_dp(t);           // ... which the next dP^T overwrites
                }
            }
            if (ok) umma_commit(bar(ACC_FULL));
        }
    } else if (warp < kWarpMma2) {
        const int wg = (warp - 2) >> 2;                   // 0 or 1: columns (query rows) 32 wg .. 32 wg + 31 of every tile
        const int lane_group = warp & 3;
        const int etid = lane_group * 32 + lane;          // 0..127: key row owned inside the CTA
        const int key = j0 + etid;
        const uint32_t t_lane = ((uint32_t)(lane_group * 32) << 16);
        const float scale = 1.0f / sqrtf((float)HD);
        const int64_t gs = 3 * (int64_t)g.C;
        const int64_t lb = ((int64_t)b * g.H + h) * g.T;
        if (wg == 0) {   // K' = K * scale * log2(e) into tensor memory
            const int wrow0 = min(j0 + lane_group * 32, g.T - 1);
            const int64_t off = (int64_t)(row_base + wrow0) * gs + g.C + h * HD;
            float* tile = reinterpret_cast<float*>(smem_raw + (bars + 256u - smem_u32(smem_raw)) + (uint32_t)lane_group * kRowTileBytes);
            rows_to_tmem(g.qkv_hi + off, g.qkv_hi + g.qkv_plane + off, gs, max(1, min(32, g.T - wrow0)), scale * kLog2e,
                         tK_hi + t_lane, tK_lo + t_lane, tile, lane);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(K_READY));
        }
        bool ok = true;
        int tn = 0;
        const uint32_t c0 = 32u * (uint32_t)wg;
        // Softmax statistics of a tile's 64 query rows (log-sum-exp in base-2 units, D = rowsum(dO o O)):
        // every thread needs the 32 values of its warpgroup's columns.  128 threads fetch one value each
        // for the NEXT tile while the current one is worked on and leave it in shared memory
        // ([2][L 0-63 | D 64-127], double-buffered by tile parity), from where it is read with
        // 128-bit broadcast loads.  (Each thread loading its 64 values itself -- 512 load instructions
        // per tile and SM -- took 3,000 of a tile's 7,000 clocks.)  A buffer is rewritten at the end of
        // tile t for tile t + 1: every warp read tile t - 1's values before the products of tile t could start.
        float* stat = reinterpret_cast<float*>(smem_raw + (bars + 256u + 4u * kRowTileBytes - smem_u32(smem_raw)));
        const int sidx = (warp - 2) * 32 + lane;          // 0..255; the first 128 threads stage values
        auto fetch_stat = [&](int t) -> float {
            const int r = min(q_row0(t) + (sidx & 63), g.T - 1);   // clamped: rows past the end are masked below
            return sidx < 64 ? __ldg(g.lse + lb + r) * kLog2e : __ldg(g.dvec + lb + r);
        };
        auto publish_stat = [&](int t, float v) {          // warps 2-5: value of tile t into its buffer
            if (sidx < 128) {
                stat[(t & 1) * 128 + sidx] = v;
                __threadfence_block();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(STAT_READY));
            }
        };
        if (n_t > 0) publish_stat(0, sidx < 128 ? fetch_stat(0) : 0.f);
        for (int t = 0; t < n_t && ok; ++t) {
            const int q0 = q_row0(t) + 32 * wg;
            const int nvalid = min(32, g.T - q0);
            float next_stat = 0.f;
            if (sidx < 128 && t + 1 < n_t) next_stat = fetch_stat(t + 1);   // in flight during this tile
            if (!mbar_wait_warp_ool(bar(STAT_READY), (uint32_t)(t & 1), g.err, 42)) { ok = false; break; }
            float Lc[32], Dc[32];
            {
                const float4* Ls = reinterpret_cast<const float4*>(stat + (t & 1) * 128 + 32 * wg);
                const float4* Ds = reinterpret_cast<const float4*>(stat + (t & 1) * 128 + 64 + 32 * wg);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float4 l4 = Ls[i], d4 = Ds[i];
                    Lc[4 * i] = l4.x; Lc[4 * i + 1] = l4.y; Lc[4 * i + 2] = l4.z; Lc[4 * i + 3] = l4.w;
                    Dc[4 * i] = d4.x; Dc[4 * i + 1] = d4.y; Dc[4 * i + 2] = d4.z; Dc[4 * i + 3] = d4.w;
                }
            }
            if (etid == 0) trace_mark(g.trace, 1 + wg, tn, 700 + t);
            if (!mbar_wait_warp_ool(bar(S_FULL), (uint32_t)(t & 1), g.err, 31)) { ok = false; break; }
            tc_fence_after();
            uint32_t s[32];
            float p[32];
            uint32_t lo[32];
            tmem_ld32(tS + t_lane + c0, s);
            tmem_ld32(tPlo + t_lane + c0, lo);        // the second half of the split score product
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const bool live = (i < nvalid) && (q0 + i >= key);   // in the sequence and not before this key
                p[i] = live ? ex2_approx((__uint_as_float(s[i]) + __uint_as_float(lo[i])) - Lc[i]) : 0.f;
                split_tf32_int(p[i], s[i], lo[i]);
            }
            tmem_st32(tS + t_lane + c0, s);          // P^T hi over S^T
            tmem_st32(tPlo + t_lane + c0, lo);
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(P_READY));
            if (etid == 0) trace_mark(g.trace, 1 + wg, tn, 800 + t);
            if (!mbar_wait_warp_ool(bar(DP_FULL), (uint32_t)(t & 1), g.err, 32)) { ok = false; break; }
            tc_fence_after();
            tmem_ld32(tdP + t_lane + c0, s);
            tmem_ld32(tdSlo + t_lane + c0, lo);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const float ds = p[i] * ((__uint_as_float(s[i]) + __uint_as_float(lo[i])) - Dc[i]);
                split_tf32_int(ds, s[i], lo[i]);
            }
            tmem_st32(tdP + t_lane + c0, s);         // dS^T hi over dP^T
            tmem_st32(tdSlo + t_lane + c0, lo);
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(DS_READY));
            if (etid == 0) trace_mark(g.trace, 1 + wg, tn, 900 + t);
            if (t + 1 < n_t) publish_stat(t + 1, next_stat);
        }
        if (ok) ok = mbar_wait_warp_ool(bar(ACC_FULL), 0, g.err, 33);
        if (ok) {   // warp-uniform: the tensor-memory loads below need the whole warp
            tc_fence_after();
            const int wrow0 = j0 + lane_group * 32;                    // first key row of this warp
            const int nvalid = max(0, min(32, g.T - wrow0));
            float* hi = g.dqkv_hi + (int64_t)(row_base + wrow0) * gs + h * HD;   // dereferenced for valid rows only
            float* lo = hi + g.dqkv_plane;
            float* sums = g.rg_sums
                              ? g.rg_sums + ((int64_t)b * g.nrg + (j0 >> 5) + lane_group) * gs + h * HD
                              : nullptr;
            // the streamed-tile buffers are idle by now: each warp stages its rows in a slice of them
            float* tile = reinterpret_cast<float*>(smem_raw + (qk_s - smem_u32(smem_raw)) + (uint32_t)(warp - 2) * kRowTileBytes);
            // warpgroup 0 writes dK (columns C .. 2C of the row), warpgroup 1 dV (2C .. 3C): one call site
            const int64_t col = (int64_t)(1 + wg) * g.C;
            tmem_rows_to_split((wg == 0 ? tdK : tdV) + t_lane, wg == 0 ? scale : 1.0f, hi + col, lo + col, gs, nvalid,
                               sums ? sums + col : nullptr, tile, lane);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
    if (threadIdx.x == 0) trace_cta(g.trace, 0, 1, globaltimer_ns());
}

// ------------------------------------------------------------------------------------------- dq

// The dq kernel streams 64-key tiles: its score products then run with N = 64 (an MMA costs the
// same ~50 clocks for N = 32 and N = 64), and dS hi/lo overwrite S and dP in place, so two
// 128-column buffers fit beside Q' and dQ.  Shared memory holds dO (64 KB), two stages of the
// K-major K and V tiles (4 x 32 KB) and ONE stage of the MN-major K tile (32 KB): 224 KB.
constexpr int BKT = 64;
constexpr uint32_t kTileQ = 2u * 2u * BKT * 128u;   // one streamed 64-row tile in one layout (32 KB)
constexpr uint32_t kDqSmem = 1024u + kResBytes + 5u * kTileQ + 256u + 512u;   // + the 128 row sums D
//  MN-major 64-row tile (2 column groups of [hi|lo][64 rows][128 B]), contraction over the rows.
__device__ __forceinline__ constexpr uint32_t mnmaj64_off(int ks, bool lo) {
    return (lo ? BKT * 128u : 0u) + (uint32_t)ks * 1024u;
}
__device__ __forceinline__ DescBase mnmaj64_base(uint32_t tile) { return make_desc_base(tile, 2u * BKT * 128u, 512u, 1u); }

__global__ void __launch_bounds__(kThreadsDq, 1)
attn_bwd_dq_tc_kernel(const __grid_constant__ CUtensorMap tmKk, const __grid_constant__ CUtensorMap tmKm,
                      const __grid_constant__ CUtensorMap tmVk, const __grid_constant__ CUtensorMap tmDOres,
                      const BwdArgs g) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t do_s = base;                                 // resident dO (A operand of dP)
    auto kk_s = [&](int st) { return base + kResBytes + (uint32_t)st * 2u * kTileQ; };
    auto vk_s = [&](int st) { return kk_s(st) + kTileQ; };
    const uint32_t km_s = base + kResBytes + 4u * kTileQ;       // single stage
    const uint32_t qstage = km_s;                               // staging of the query rows before the first fill
    const uint32_t bars = base + kResBytes + 5u * kTileQ;
    // count-1: 0 do_full, 1-2 kfull, 5 mfull, 6 / 8 dq_done, 7 mempty, 11 acc_full; count-2 (the S and the dP
    // issuing threads both commit): 3-4 kempty, 9-10 sdp_full
    const uint32_t do_full = bars;
    auto kfull = [&](int s) { return bars + 8u * (1 + s); };
    auto kempty = [&](int s) { return bars + 8u * (3 + s); };
    const uint32_t mfull = bars + 8u * 5;
    const uint32_t mempty = bars + 8u * 7;
    auto sdp_full = [&](int b) { return bars + 8u * (9 + b); };
    auto dq_done = [&](int b) { return bars + 8u * (6 + 2 * b); };   // dQ(t) has read buffer b: it may be overwritten
    const uint32_t acc_full = bars + 8u * 11;
    // count-4: 12-13 ds_full, 14 q_ready
    auto ds_full = [&](int b) { return bars + 8u * (12 + b); };
    const uint32_t q_ready = bars + 8u * 14;
    const uint32_t tmem_slot = bars + 8u * 15;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int bh, yb;
    grouped_block(g.head_group, bh, yb);
    const int qt = gridDim.y - 1 - yb;                          // heaviest query tiles first, over the heads of a group
    const int b = bh / g.H, h = bh % g.H;
    const int q0 = qt * BR;
    const int row_base = b * g.T;
    const int n_t = min(q0 + BR - 1, g.T - 1) / BKT + 1;         // key tiles up to the diagonal
    if (threadIdx.x == 0) {
        trace_cta(g.trace, 1, 0, globaltimer_ns());
        trace_cta(g.trace, 1, 2, smid());
        trace_cta(g.trace, 1, 3, n_t);
    }

    const uint32_t tmem = setup(bars, 12, bars + 8u * 12, 3, tmem_slot, smem_raw, warp, 0x618u);   // bars 3, 4, 9, 10: two arrivals
    pdl_wait();      // set-up done; global memory is touched from here on
    pdl_trigger();
    // dQ is 128 columns: the halves of the split product dS . [K_hi | K_lo] by 32-column groups (see issue_b)
    const uint32_t tQ_hi = tmem, tQ_lo = tmem + 64, tdQ = tmem + 128;
    auto tbuf = [&](int bb) { return tmem + 256u + 128u * (uint32_t)bb; };   // +0 S -> dS_hi, +64 dP -> dS_lo

    if (warp == 0) {
        if (lane == 0) {
            mbar_expect_tx(do_full, kResBytes);
            for (int kb = 0; kb < 2; ++kb)
                tma_load_3d(do_s + kb * (kResBytes / 2), &tmDOres, do_full, h * HD + kb * 32, row_base + q0, 0);
            bool ok = true;
            auto load_kmajor = [&](int t) -> bool {
                const int st = t & 1, k0 = t * BKT;
                if (!mbar_wait_ool(kempty(st), ((t >> 1) & 1u) ^ 1u, g.err, 31)) return false;
                mbar_expect_tx(kfull(st), 2u * kTileQ);
                for (int kb = 0; kb < 2; ++kb) {
                    tma_load_3d(kk_s(st) + kb * (kTileQ / 2), &tmKk, kfull(st), g.C + h * HD + kb * 32, row_base + k0, 0);
                    tma_load_3d(vk_s(st) + kb * (kTileQ / 2), &tmVk, kfull(st), 2 * g.C + h * HD + kb * 32, row_base + k0, 0);
                }
                return true;
            };
            // The K-major tiles of tile t+1 go out before the wait for the single MN-major buffer:
            // the score products of t+1 are issued ahead of the dQ product of t.
            ok = load_kmajor(0);
            for (int t = 0; t < n_t && ok; ++t) {
                if (t + 1 < n_t) ok = load_kmajor(t + 1);
                if (!ok) break;
                // the MN-major buffer doubles as the staging area of the query rows: first fill after that
                if (t == 0 && !mbar_wait_ool(q_ready, 0, g.err, 40)) { ok = false; break; }
                if (!mbar_wait_ool(mempty, (t & 1u) ^ 1u, g.err, 32)) { ok = false; break; }
                mbar_expect_tx(mfull, kTileQ);
                for (int grp = 0; grp < 2; ++grp)
                    tma_load_3d(km_s + grp * (kTileQ / 2), &tmKm, mfull, g.C + h * HD + grp * 32, row_base + t * BKT, 0);
            }
            if (!ok)
                for (int i = 0; i < 2000; ++i) __nanosleep(1000);
        }
    } else if (warp == 1 || warp == kWarpMma2) {
        // ---- the two score products, one issuing thread each: warp 1 S = Q' K^T (A in tensor memory),
        // warp 10 dP = dO V^T (A resident in shared memory).  Both write into buffer t & 1, which the
        // dQ product of tile t - 2 must have read.
        if (lane == 0) {
            constexpr uint32_t idesc_a = make_idesc_tf32(BR, BKT, false, false);   // 128 x 64, B K-major
            const bool s_product = warp == 1;
            bool ok = s_product ? mbar_wait_ool(q_ready, 0, g.err, 34) : mbar_wait_ool(do_full, 0, g.err, 33);
            int tn = 0;
            const DescBase dod = kmaj_base(do_s);
            for (int t = 0; t < n_t && ok; ++t) {
                const int st = t & 1, bb = t & 1;
                trace_mark(g.trace, 0, tn, 100 + t);
                if (!mbar_wait_ool(kfull(st), (t >> 1) & 1u, g.err, 35)) { ok = false; break; }
                if (t >= 2 && !mbar_wait_ool(dq_done(bb), ((t - 2) >> 1) & 1u, g.err, 41)) { ok = false; break; }
                trace_mark(g.trace, 0, tn, 200 + t);
                tc_fence_after();
                if (s_product) {
                    const uint32_t dS = tbuf(bb);
                    const DescBase kd = kmaj_base(kk_s(st));
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint64_t k_hi = kd.at(kmaj_off(BKT, ks, false)), k_lo = kd.at(kmaj_off(BKT, ks, true));
                        umma_tf32_ts(dS, tQ_lo + ks * 8, k_hi, idesc_a, ks > 0 ? 1u : 0u);
                        umma_tf32_ts(dS, tQ_hi + ks * 8, k_lo, idesc_a, 1u);
                        umma_tf32_ts(dS, tQ_hi + ks * 8, k_hi, idesc_a, 1u);
                    }
                } else {
                    const uint32_t dP = tbuf(bb) + 64u;
                    const DescBase vkd = kmaj_base(vk_s(st));
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint64_t o_hi = dod.at(kmaj_off(BR, ks, false)), o_lo = dod.at(kmaj_off(BR, ks, true));
                        const uint64_t v_hi = vkd.at(kmaj_off(BKT, ks, false)), v_lo = vkd.at(kmaj_off(BKT, ks, true));
                        umma_tf32(dP, o_lo, v_hi, idesc_a, ks > 0 ? 1u : 0u);
                        umma_tf32(dP, o_hi, v_lo, idesc_a, 1u);
                        umma_tf32(dP, o_hi, v_hi, idesc_a, 1u);
                    }
                }
                umma_commit(kempty(st));
                umma_commit(sdp_full(bb));
                trace_mark(g.trace, 0, tn, 300 + t);
            }
        }
    } else if (warp == kWarpMma3) {
        // ---- the accumulating product dQ += dS K, a third issuing thread
        if (lane == 0) {
            constexpr uint32_t idesc_b = make_idesc_tf32(BR, HD, false, true);     // 128 x 64, B MN-major
            constexpr uint32_t idesc_b2 = make_idesc_tf32(BR, 2 * HD, false, true);   // 128 x 128, B = four column groups
            bool ok = true;
            int tn = 0;
            // Two instructions per k-step.  The MN-major K tile lies in shared memory as the column
            // groups [K_hi g0 | K_lo g0 | K_hi g1 | K_lo g1] (g = 32 head columns), 8 KB apart: seen
            // with that stride it is one operand of N = 128, and dS_hi times it fills the four
            // 32-column groups of dQ in that order.  dS_lo . K_hi (groups g0, g1, 16 KB apart, N = 64)
            // is accumulated 32 columns further, so that its halves land on the second and third group:
            // head columns 0-31 = dQ[0:32) + dQ[32:64), 32-63 = dQ[64:96) + dQ[96:128).
            const DescBase kmd = mnmaj64_base(km_s);
            const DescBase kmd4 = make_desc_base(km_s, BKT * 128u, 512u, 1u);
            for (int t = 0; t < n_t && ok; ++t) {
                const int bb = t & 1;
                if (!mbar_wait_ool(ds_full(bb), (t >> 1) & 1u, g.err, 36)) { ok = false; break; }
                trace_mark(g.trace, 0, tn, 400 + t);
                if (!mbar_wait_ool(mfull, t & 1u, g.err, 37)) { ok = false; break; }
                trace_mark(g.trace, 0, tn, 500 + t);
                tc_fence_after();
                const uint32_t s_hi = tbuf(bb), s_lo = tbuf(bb) + 64u;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t acc = (t > 0 || ks > 0) ? 1u : 0u;
                    umma_tf32_ts(tdQ, s_hi + ks * 8, kmd4.at(mnmaj64_off(ks, false)), idesc_b2, acc);
                    umma_tf32_ts(tdQ + 32u, s_lo + ks * 8, kmd.at(mnmaj64_off(ks, false)), idesc_b, 1u);
                }
                umma_commit(mempty);
                umma_commit(dq_done(bb));
                trace_mark(g.trace, 0, tn, 600 + t);
            }
            if (ok) umma_commit(acc_full);
        }
    } else if (warp < kWarpMma2) {
        const int wg = (warp - 2) >> 2;
        const int lane_group = warp & 3;
        const int row = q0 + lane_group * 32 + lane;
        const uint32_t t_lane = ((uint32_t)(lane_group * 32) << 16);
        const float scale = 1.0f / sqrtf((float)HD);
        const int64_t gs = 3 * (int64_t)g.C;
        const int64_t lb = ((int64_t)b * g.H + h) * g.T;
        const int rc = min(row, g.T - 1);
        if (wg == 0) {
            // the MN-major K buffer is not filled before the first score products are under way: its
            // first 18 KB stage the query rows on their way into tensor memory
            const int wrow0 = min(q0 + lane_group * 32, g.T - 1);
            const int64_t off = (int64_t)(row_base + wrow0) * gs + h * HD;
            float* tile = reinterpret_cast<float*>(smem_raw + (qstage - smem_u32(smem_raw)) + (uint32_t)lane_group * kRowTileBytes);
            rows_to_tmem(g.qkv_hi + off, g.qkv_hi + g.qkv_plane + off, gs, max(1, min(32, g.T - wrow0)), scale * kLog2e,
                         tQ_hi + t_lane, tQ_lo + t_lane, tile, lane);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tile is next written by TMA
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(q_ready);
        }
        // D = rowsum(dO o O) of the CTA's 128 rows: formed here by warpgroup 1, which has nothing
        // else to do until its first tile, handed to warpgroup 0 through shared memory and left in
        // global memory for the dkv kernel
        float* dsm = reinterpret_cast<float*>(smem_raw + (bars + 256u - smem_u32(smem_raw)));
        if (wg == 1) {
            const int wrow0 = min(q0 + lane_group * 32, g.T - 1);
            const long long off = (long long)(row_base + wrow0) * g.C + h * HD;
            const float d = warp_rows_dot64(g.o_hi + off, g.o_lo ? g.o_lo + off : nullptr, g.do_hi + off,
                                            g.do_hi + g.do_plane + off, g.C, max(1, min(32, g.T - wrow0)), lane);
            dsm[lane_group * 32 + lane] = d;
            if (row < g.T) g.dvec_out[lb + row] = d;
        }
        asm volatile("bar.sync 2, 256;" ::: "memory");    // the eight element-wise warps, exactly once
        const float L = g.lse[lb + rc] * kLog2e, D = dsm[lane_group * 32 + lane];
        bool ok = true;
        int tn = 0;
        const uint32_t tb = tbuf(wg) + t_lane;
        for (int t = wg; t < n_t && ok; t += 2) {
            const int k0 = t * BKT;
            if (lane_group == 0 && lane == 0) trace_mark(g.trace, 1 + wg, tn, 700 + t);
            if (!mbar_wait_warp_ool(sdp_full(wg), (t >> 1) & 1u, g.err, 38)) { ok = false; break; }
            if (lane_group == 0 && lane == 0) trace_mark(g.trace, 1 + wg, tn, 800 + t);
            tc_fence_after();
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t s[32], dp[32];
                tmem_ld32(tb + half * 32u, s);
                tmem_ld32(tb + 64u + half * 32u, dp);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    float p = ex2_approx(__uint_as_float(s[i]) - L);
                    if (k0 + half * 32 + i > row) p = 0.f;          // key follows this query: masked
                    const float ds = p * (__uint_as_float(dp[i]) - D);
                    split_tf32_int(ds, s[i], dp[i]);
                }
                tmem_st32(tb + half * 32u, s);                      // dS hi over S
                tmem_st32(tb + 64u + half * 32u, dp);               // dS lo over dP
            }
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(ds_full(wg));
            if (lane_group == 0 && lane == 0) trace_mark(g.trace, 1 + wg, tn, 1000 + t);
        }
        if (wg == 0) {
            if (ok) ok = mbar_wait_warp_ool(acc_full, 0, g.err, 39);
            if (ok) {   // warp-uniform: the tensor-memory loads below need the whole warp
                tc_fence_after();
                const int wrow0 = q0 + lane_group * 32;                // first query row of this warp
                const int nvalid = max(0, min(32, g.T - wrow0));
                float* hi = g.dqkv_hi + (int64_t)(row_base + wrow0) * gs + h * HD;
                float* sums = g.rg_sums
                                  ? g.rg_sums + ((int64_t)b * g.nrg + (q0 >> 5) + lane_group) * gs + h * HD
                                  : nullptr;
                float* tile = reinterpret_cast<float*>(smem_raw + (kk_s(0) - smem_u32(smem_raw)) + (uint32_t)(warp - 2) * kRowTileBytes);
                tmem_rows_to_split<true>(tdQ + t_lane, scale, hi, hi + g.dqkv_plane, gs, nvalid, sums, tile, lane);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
    if (threadIdx.x == 0) trace_cta(g.trace, 1, 1, globaltimer_ns());
}

bool enc3(CUtensorMap* tm, const float* base, int64_t cols, int64_t rows, int64_t plane, uint32_t box_rows,
          bool mn_major) {
    EncodeTiledFn enc = tensor_map_encoder();
    if (!enc) return false;
    cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, 2};
    cuuint64_t strides[2] = {(cuuint64_t)cols * 4, (cuuint64_t)plane * 4};
    cuuint32_t box[3] = {32, box_rows, 2};
    cuuint32_t estr[3] = {1, 1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, (void*)base, dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE,
               mn_major ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

cudaError_t attention_tc_default_err(int** out);

// Rows of the optional row-group sums array: one per 32 rows of every 128-row block.
int64_t attention_bwd_rowgroups(int B, int T) { return (int64_t)B * 4 * ((T + BR - 1) / BR); }

// dqkv (hi/lo planes) from qkv (hi/lo planes), dO (hi/lo planes), O (raw, or hi/lo planes) and lse;
// dvec [B, H, T] receives rowsum(dO o O) on the way.
// rg_sums (nullable, [attention_bwd_rowgroups][3C]): column sums of dqkv per 32-row group; summing
// its rows gives the gradient of the QKV bias without another pass over dqkv.
cudaError_t launch_attention_bwd_tc(const float* qkv_hi, int64_t qkv_plane, const float* do_hi, int64_t do_plane,
                                    const float* o, const float* o_lo, const float* lse, float* dvec, int B, int T,
                                    int C, int H, float* dqkv_hi, int64_t dqkv_plane, float* rg_sums, int* err_word,
                                    cudaStream_t s) {
    static cudaError_t attr = []() {
        cudaError_t e = cudaFuncSetAttribute(attn_bwd_dkv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)kDkvSmem);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attn_bwd_dq_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDqSmem);
        return e;
    }();
    if (attr != cudaSuccess) return attr;
    if (!err_word) {
        cudaError_t e = attention_tc_default_err(&err_word);
        if (e != cudaSuccess) return e;
    }
    const int64_t rows = (int64_t)B * T;
    CUtensorMap dok64, dom64, vres, dores;
    bool ok = enc3(&dok64, do_hi, C, rows, do_plane, BT64, false) &&                // 64-row K-major / MN-major tiles of dO
              enc3(&dom64, do_hi, C, rows, do_plane, BT64, true) &&
              enc3(&vres, qkv_hi, 3 * (int64_t)C, rows, qkv_plane, BR, false) &&    // 128-row resident tiles
              enc3(&dores, do_hi, C, rows, do_plane, BR, false);
    CUtensorMap qk64, qm64;
    ok = ok && enc3(&qk64, qkv_hi, 3 * (int64_t)C, rows, qkv_plane, BKT, false) &&  // 64-row K-major / MN-major tiles of qkv
         enc3(&qm64, qkv_hi, 3 * (int64_t)C, rows, qkv_plane, BKT, true);
    if (!ok) return cudaErrorInvalidValue;
    BwdArgs g{T, C, H, attn_head_group(B * H, (T + BR - 1) / BR), qkv_hi, qkv_plane, lse, dvec, dvec, o, o_lo, do_hi, do_plane, dqkv_hi, dqkv_plane, err_word,
              attention_tc_get_trace(), rg_sums, 4 * ((T + BR - 1) / BR)};
    dim3 gk(B * H, (T + BR - 1) / BR);
    // the dq kernel goes first: it also forms D = rowsum(dO o O), which the dkv kernel reads
    BT_KERNEL_LAUNCH((attn_bwd_dq_tc_kernel), gk, kThreadsDq, kDqSmem, s, qk64, qm64, qk64, dores, g);
    BT_COUNT_LAUNCH();
    BT_KERNEL_LAUNCH((attn_bwd_dkv_tc_kernel), gk, kThreadsDkv, kDkvSmem, s, qk64, qm64, dok64, dom64, vres, g);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

}  // namespace bt
