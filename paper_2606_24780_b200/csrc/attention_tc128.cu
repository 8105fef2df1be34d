// Causal flash attention for head_dim 128 on the 5th-generation tensor cores, forward and
// backward, FP32 fidelity through 3xTF32 split products.
//
// With 128-wide heads a 128-row operand in hi/lo planes takes 128 KB, so only ONE such operand
// fits in shared memory and one more in tensor memory (256 columns).  Every pass of the method is
// therefore the same small pipeline, instantiated five times:
//
//     X   = A1 B1^T          A1: the CTA's own 128 rows, pre-scaled, hi/lo in TENSOR MEMORY
//     Y   = A2 B2^T          A2: the CTA's own 128 rows of a second tensor, resident in shared memory
//     Z   = f(X, Y)          element-wise, thread = row (tensor-memory lane)
//     Out += Z B3            Z hi/lo written back to tensor memory, Out accumulates there
//
//   pass   rows (lanes)  A1   B1  A2   B2   f                          B3   Out
//   MAX    queries       Q'   K   -    -    row maximum m (X in 1xTF32) -    -
//   FWD    queries       Q'   K   -    -    P = exp2(X - m), l = sum P V    O = (P V) / l, lse = m + log l
//   DQ     queries       Q'   K   dO   V    dS = P o (Y - D)           K    dQ (x 1/sqrt d)
//   DK     keys          K'   Q   V    dO   dS^T = P^T o (Y - D)       Q    dK (x 1/sqrt d)
//   DV     keys          K'   Q   -    -    P^T                        dO   dV
//
// (Q' = Q log2(e)/sqrt(d), K' likewise: X is the score in base-2 units.)  The forward runs MAX and
// then FWD.  MAX only has to find a reference value near each row's maximum, so it forms the scores
// from the hi planes alone (one MMA per k-step instead of three); FWD then uses that reference for
// every tile -- P needs no running-maximum rescaling, O accumulates in tensor memory like the
// backward's outputs -- and normalises with the sum of the P it actually formed, so the result does
// not depend on how exact the reference is.  The streamed
// tiles B1, B2 (K-major, 128-byte swizzle) and B3 (MN-major, 128-byte swizzle with 32-byte atoms)
// are 32 rows x 128 columns x (hi, lo) = 32 KB each.  With A2 resident (DQ, DK) every stream has
// one buffer, refilled as soon as the one product that reads it has completed; the passes without
// A2 spend its 128 KB on three B1 stages and two B3 stages.  X / Y live in two tensor-memory
// buffers that the two element-wise warpgroups take alternately, and Z overwrites X / Y in place.
//
//   warp 0 (one lane)   TMA producer
//   warp 1 (one lane)   MMA issuer: X(0) Y(0), then per tile t: X(t+1) Y(t+1) | Out(t)
//   warps 2-5, 6-9      element-wise warpgroups (tile t belongs to warpgroup t & 1)
//
//   tensor memory: A1 hi 0-127, A1 lo 128-255, Out 256-383, buffer b: X -> Z_hi at 384 + 64 b,
//                  Y -> Z_lo at 416 + 64 b
//   shared memory: A2 128 KB (or stream stages), B1 / B2 / B3 32 KB each
// Every mbarrier wait is bounded and reports through the device error word; a CTA whose wait ran
// out stops issuing, lets loads in flight land, frees its tensor memory and exits.
#include "common.cuh"
#include "tc_common.cuh"

namespace bt {

using namespace tc;

namespace {

constexpr int HD = 128, BR = 128, BT_ = 32;
constexpr int kThreads = 320;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr uint32_t kRes = 4u * 2u * BR * 128u;     // resident operand: 4 k-blocks x (hi, lo) x 128 rows x 128 B
constexpr uint32_t kTile = 4u * 2u * BT_ * 128u;   // streamed tile: 4 blocks x (hi, lo) x 32 rows x 128 B
constexpr uint32_t kSmem = 1024u + kRes + 3u * kTile + 256u;

enum Pass { P_LSE = 0, P_FWD = 1, P_DQ = 2, P_DK = 3, P_DV = 4 };

struct Args128 {
    int T, C, H;
    const float* a1_hi;       // hi plane of the array the CTA's own rows come from (lo at + a1_plane)
    long long a1_plane;
    long long a1_stride;      // row stride of that array in floats
    int a1_col;               // column of head 0 in it
    int a2_col, b1_col, b2_col, b3_col;   // column of head 0 in the arrays behind the tensor maps
    const float* lse;         // [B, H, T], natural log (backward passes); FWD reads the MAX pass's reference
    const float* dvec;        // [B, H, T] rowsum(dO o O) (DQ, DK)
    float* lse_out;           // MAX: the row reference (base-2 units); FWD: the log-sum-exp
    float* out_raw;           // row-major outputs [B*T][out_stride], any may be null
    float* out_hi;
    float* out_lo;
    long long out_stride;
    int out_col;              // column of head 0 in the output
    float out_mul;
    float* rg_sums;           // optional column sums of the output per 32-row group: [B * nrg][out_stride]
    int nrg;
    int* err;
    int head_group;           // heads per group of the CTA order (grouped_block)
};

// MN-major 32-row tile: 4 column groups of [hi | lo][32 rows][128 B]; k-step = 8 rows.
__device__ __forceinline__ constexpr uint32_t mnmaj_off(int ks, bool lo) {
    return (lo ? BT_ * 128u : 0u) + (uint32_t)ks * 1024u;
}
__device__ __forceinline__ DescBase mnmaj_base(uint32_t tile) { return make_desc_base(tile, 2u * BT_ * 128u, 512u, 1u); }

template <int PASS>
__global__ void __launch_bounds__(kThreads, 1)
attn128_kernel(const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmB1,
               const __grid_constant__ CUtensorMap tmB2, const __grid_constant__ CUtensorMap tmB3, const Args128 g) {
    constexpr bool kKeys = (PASS == P_DK || PASS == P_DV);    // lanes are keys, streamed rows are queries
    constexpr bool kHasY = (PASS == P_DQ || PASS == P_DK);
    constexpr bool kHasOut = (PASS != P_LSE);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t a2_s = base;
    const uint32_t b1_s = base + kRes, b2_s = b1_s + kTile, b3_s = b2_s + kTile;
    const uint32_t bars = b3_s + kTile;
    // Passes without a resident A2 spend its 128 KB on the streams: B1 three stages deep (its own
    // buffer and two A2 slots), B3 two stages (the other two A2 slots); the B2 / B3 buffers then only
    // stage the CTA's own rows on their way into tensor memory.
    constexpr int S1 = kHasY ? 1 : 3, S3 = kHasY ? 1 : 2;
    enum { A2_FULL = 0, B1_FULL, B1_EMPTY = B1_FULL + 3, B2_FULL = B1_EMPTY + 3, B2_EMPTY, B3_FULL, B3_EMPTY = B3_FULL + 2,
           XY_FULL0 = B3_EMPTY + 2, XY_FULL1, ACC_FULL, Z_READY0, Z_READY1, A1_READY, N_BARS };
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
    auto b1_stage = [&](int st) { return (kHasY || st == 0) ? b1_s : a2_s + (uint32_t)(st - 1) * kTile; };
    auto b3_stage = [&](int st) { return kHasY ? b3_s : a2_s + (uint32_t)(2 + st) * kTile; };
    const uint32_t tmem_slot = bars + 8u * N_BARS;
    auto smem_ptr = [&](uint32_t addr) { return smem_raw + (addr - smem_u32(smem_raw)); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int bh, yb;
    grouped_block(g.head_group, bh, yb);
    const int b = bh / g.H, h = bh % g.H;
    // query passes: heaviest (last) query blocks first; key passes: block 0 has the longest walk
    const int blk = kKeys ? yb : (int)gridDim.y - 1 - yb;
    const int r0 = blk * BR;                              // first own row inside the sequence
    const int row_base = b * g.T;
    const int n_tiles_seq = (g.T + BT_ - 1) / BT_;
    const int n_t = kKeys ? n_tiles_seq - r0 / BT_ : min(r0 + BR - 1, g.T - 1) / BT_ + 1;
    // first streamed row of tile t: keys walk up from 0; queries walk from the LAST tile down to the
    // diagonal (the tensor core truncates when it adds into its accumulator: small far terms first)
    auto o0 = [&](int t) { return kKeys ? (n_tiles_seq - 1 - t) * BT_ : t * BT_; };

    if (threadIdx.x == 0) {
        for (int i = 0; i < Z_READY0; ++i) mbar_init(bar(i), 1);
        mbar_init(bar(Z_READY0), 4);
        mbar_init(bar(Z_READY1), 4);
        mbar_init(bar(A1_READY), 8);
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
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(smem_ptr(tmem_slot));
    pdl_wait();      // set-up done; global memory is touched from here on
    pdl_trigger();
    const uint32_t tA1_hi = tmem, tA1_lo = tmem + 128, tOut = tmem + 256;
    auto tbuf = [&](int bb) { return tmem + 384u + 64u * (uint32_t)bb; };   // +0 X -> Z_hi, +32 Y -> Z_lo

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            if (kHasY) {
                mbar_expect_tx(bar(A2_FULL), kRes);
                for (int kb = 0; kb < 4; ++kb)
                    tma_load_3d(a2_s + kb * (kRes / 4), &tmA2, bar(A2_FULL), g.a2_col + h * HD + kb * 32, row_base + r0, 0);
            }
            bool ok = true;
            // t = the tile whose rows go in; a stream of S stages keeps tile t in stage t % S
            auto load = [&](uint32_t dst, const CUtensorMap* tm, int full, int empty, int col, int t, int stages) -> bool {
                const int st = t % stages;
                const uint32_t round = (uint32_t)(t / stages);
                if (!mbar_wait(bar(empty + st), (round & 1u) ^ 1u, g.err, 51)) return false;
                mbar_expect_tx(bar(full + st), kTile);
                for (int part = 0; part < 4; ++part)
                    tma_load_3d(dst + part * (kTile / 4), tm, bar(full + st), col + h * HD + part * 32, row_base + o0(t), 0);
                return true;
            };
            ok = load(b1_stage(0), &tmB1, B1_FULL, B1_EMPTY, g.b1_col, 0, S1);
            if (kHasY) {
                // here the B2 / B3 buffers stage the CTA's own rows on their way into tensor memory first
                if (ok) ok = mbar_wait(bar(A1_READY), 0, g.err, 52);
                if (ok) ok = load(b2_s, &tmB2, B2_FULL, B2_EMPTY, g.b2_col, 0, 1);
            }
            for (int t = 0; t < n_t && ok; ++t) {
                if (t + 1 < n_t) {
                    ok = load(b1_stage((t + 1) % S1), &tmB1, B1_FULL, B1_EMPTY, g.b1_col, t + 1, S1);
                    if (ok && kHasY) ok = load(b2_s, &tmB2, B2_FULL, B2_EMPTY, g.b2_col, t + 1, 1);
                }
                if (ok && kHasOut) ok = load(b3_stage(t % S3), &tmB3, B3_FULL, B3_EMPTY, g.b3_col, t, S3);
            }
            if (!ok)
                for (int i = 0; i < 2000; ++i) __nanosleep(1000);   // let loads in flight land
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_x = make_idesc_tf32(BR, BT_, false, false);   // 128 x 32, B K-major
            constexpr uint32_t idesc_o = make_idesc_tf32(BR, HD, false, true);     // 128 x 128, B MN-major
            bool ok = mbar_wait(bar(A1_READY), 0, g.err, 53);
            if (ok && kHasY) ok = mbar_wait(bar(A2_FULL), 0, g.err, 54);
            const DescBase a2d = kmaj_base(a2_s), b2d = kmaj_base(b2_s);
            auto issue_xy = [&](int t) -> bool {
                const uint32_t tX = tbuf(t & 1), tY = tX + 32u;
                const int st1 = t % S1;
                if (!mbar_wait(bar(B1_FULL + st1), (uint32_t)((t / S1) & 1), g.err, 55)) return false;
                tc_fence_after();
                const DescBase b1d = kmaj_base(b1_stage(st1));
#pragma unroll
                for (int ks = 0; ks < 16; ++ks) {
                    const uint64_t b_hi = b1d.at(kmaj_off(BT_, ks, false)), b_lo = b1d.at(kmaj_off(BT_, ks, true));
                    if (PASS == P_LSE) {   // a reference near the row maximum: the hi planes suffice
                        umma_tf32_ts(tX, tA1_hi + ks * 8, b_hi, idesc_x, ks > 0 ? 1u : 0u);
                    } else {
                        umma_tf32_ts(tX, tA1_lo + ks * 8, b_hi, idesc_x, ks > 0 ? 1u : 0u);
                        umma_tf32_ts(tX, tA1_hi + ks * 8, b_lo, idesc_x, 1u);
                        umma_tf32_ts(tX, tA1_hi + ks * 8, b_hi, idesc_x, 1u);
                    }
                }
                umma_commit(bar(B1_EMPTY + st1));
                if (kHasY) {
                    if (!mbar_wait(bar(B2_FULL), (uint32_t)(t & 1), g.err, 56)) return false;
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < 16; ++ks) {
                        const uint64_t a_hi = a2d.at(kmaj_off(BR, ks, false)), a_lo = a2d.at(kmaj_off(BR, ks, true));
                        const uint64_t b_hi = b2d.at(kmaj_off(BT_, ks, false)), b_lo = b2d.at(kmaj_off(BT_, ks, true));
                        umma_tf32(tY, a_lo, b_hi, idesc_x, ks > 0 ? 1u : 0u);
                        umma_tf32(tY, a_hi, b_lo, idesc_x, 1u);
                        umma_tf32(tY, a_hi, b_hi, idesc_x, 1u);
                    }
                    umma_commit(bar(B2_EMPTY));
                }
                umma_commit(bar(XY_FULL0 + (t & 1)));
                return true;
            };
            // waits until the element-wise threads are done with tile t's buffer (Z written, or, in the
            // LSE pass, X read), then accumulates Out += Z B3
            auto issue_out = [&](int t) -> bool {
                if (!mbar_wait(bar(Z_READY0 + (t & 1)), (uint32_t)((t >> 1) & 1), g.err, 57)) return false;
                if (kHasOut) {
                    const int st3 = t % S3;
                    if (!mbar_wait(bar(B3_FULL + st3), (uint32_t)((t / S3) & 1), g.err, 58)) return false;
                    tc_fence_after();
                    const DescBase b3d = mnmaj_base(b3_stage(st3));
                    const uint32_t z_hi = tbuf(t & 1), z_lo = z_hi + 32u;
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {
                        const uint64_t b_hi = b3d.at(mnmaj_off(ks, false)), b_lo = b3d.at(mnmaj_off(ks, true));
                        const uint32_t acc = (t > 0 || ks > 0) ? 1u : 0u;
                        umma_tf32_ts(tOut, z_lo + ks * 8, b_hi, idesc_o, acc);
                        umma_tf32_ts(tOut, z_hi + ks * 8, b_lo, idesc_o, 1u);
                        umma_tf32_ts(tOut, z_hi + ks * 8, b_hi, idesc_o, 1u);
                    }
                    umma_commit(bar(B3_EMPTY + st3));
                }
                return true;
            };
            if (ok) {
                tc_fence_after();
                ok = issue_xy(0);
            }
            for (int t = 0; t < n_t && ok; ++t) {
                // X / Y of tile t+1 overwrite the buffer of tile t-1, whose Out product was issued in
                // the previous round: products issued by one thread execute in order
                if (t + 1 < n_t) ok = issue_xy(t + 1);
                if (ok) ok = issue_out(t);
            }
            if (ok) umma_commit(bar(ACC_FULL));
        }
    } else {
        // ---------------------------------------------------------------- element-wise warpgroups
        const int wg = (warp - 2) >> 2;                   // 0 or 1: owns buffer wg, tiles wg, wg + 2, ...
        const int lane_group = warp & 3;                  // the warp's tensor-memory lane quadrant
        const int rloc = lane_group * 32 + lane;
        const int own = r0 + rloc;                        // this thread's row inside the sequence
        const uint32_t t_lane = ((uint32_t)(lane_group * 32) << 16);
        const int64_t lb = ((int64_t)b * g.H + h) * g.T;
        {   // own rows -> tensor memory (pre-scaled): warpgroup 0 takes columns 0-63, warpgroup 1 64-127
            const int wrow0 = min(r0 + lane_group * 32, g.T - 1);
            const long long off = (long long)(row_base + wrow0) * g.a1_stride + g.a1_col + h * HD + 64 * wg;
            float* tile = reinterpret_cast<float*>(smem_ptr(b2_s) + (uint32_t)(warp - 2) * kRowTileBytes);
            rows_to_tmem(g.a1_hi + off, g.a1_hi + g.a1_plane + off, g.a1_stride, max(1, min(32, g.T - wrow0)),
                           kLog2e / sqrtf((float)HD), tA1_hi + t_lane + 64u * wg, tA1_lo + t_lane + 64u * wg, tile, lane);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the staging tiles are next written by TMA
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(A1_READY));
        }
        const int rc = min(own, g.T - 1);
        float L = 0.f, D = 0.f;                           // query passes: this row's statistics
        if (PASS == P_FWD) L = g.lse[lb + rc];            // the MAX pass left the reference there, in base-2 units
        if (PASS == P_DQ) L = g.lse[lb + rc] * kLog2e;
        if (PASS == P_DQ) D = g.dvec[lb + rc];
        float m_run = -INFINITY, l_run = 0.f;             // MAX: maximum, FWD: sum of P, over this warpgroup's tiles
        bool ok = true;
        const uint32_t tb = tbuf(wg) + t_lane;
        for (int t = wg; t < n_t && ok; t += 2) {
            const int s0 = o0(t);                         // first streamed row of the tile
            float Lc[32], Dc[32];
            if (kKeys) {   // the tile's 32 queries: same addresses in every thread (broadcast loads)
                if (s0 + 32 <= g.T && ((lb + s0) & 3) == 0) {   // whole tile inside the sequence, 16-byte aligned: 128-bit loads
                    const float4* lp = reinterpret_cast<const float4*>(g.lse + lb + s0);
                    const float4* dp = reinterpret_cast<const float4*>(g.dvec + lb + s0);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float4 l4 = __ldg(lp + i);
                        Lc[4 * i] = l4.x * kLog2e; Lc[4 * i + 1] = l4.y * kLog2e;
                        Lc[4 * i + 2] = l4.z * kLog2e; Lc[4 * i + 3] = l4.w * kLog2e;
                        if (PASS == P_DK) {
                            const float4 d4 = __ldg(dp + i);
                            Dc[4 * i] = d4.x; Dc[4 * i + 1] = d4.y; Dc[4 * i + 2] = d4.z; Dc[4 * i + 3] = d4.w;
                        }
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int r = min(s0 + i, g.T - 1);   // rows past the end are masked below
                        Lc[i] = __ldg(g.lse + lb + r) * kLog2e;
                        if (PASS == P_DK) Dc[i] = __ldg(g.dvec + lb + r);
                    }
                }
            }
            if (!mbar_wait_warp(bar(XY_FULL0 + wg), (uint32_t)((t >> 1) & 1), g.err, 59)) { ok = false; break; }
            tc_fence_after();
            uint32_t x[32], y[32];
            tmem_ld32(tb, x);
            if (kHasY) tmem_ld32(tb + 32u, y);
            tmem_ld_wait();
            if (PASS == P_LSE) {
                float mx = -INFINITY;
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    if (s0 + i > own) x[i] = 0xff800000u;            // key follows this query: -inf
                    mx = fmaxf(mx, __uint_as_float(x[i]));
                }
                m_run = fmaxf(m_run, mx);
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    bool live;
                    float p;
                    if (kKeys) {
                        live = (s0 + i < g.T) && (s0 + i >= own);     // query in the sequence and not before this key
                        p = live ? ex2_approx(__uint_as_float(x[i]) - Lc[i]) : 0.f;
                    } else {
                        live = (s0 + i <= own);                        // key not after this query
                        p = live ? ex2_approx(__uint_as_float(x[i]) - L) : 0.f;
                    }
                    float z = p;
                    if (PASS == P_FWD) l_run += p;
                    if (PASS == P_DQ) z = p * (__uint_as_float(y[i]) - D);
                    if (PASS == P_DK) z = p * (__uint_as_float(y[i]) - Dc[i]);
                    split_tf32_int(z, x[i], y[i]);
                }
                tmem_st32(tb, x);              // Z hi over X
                tmem_st32(tb + 32u, y);        // Z lo over Y
                tmem_st_wait();
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(Z_READY0 + wg));
        }
        // every product has completed, every load has landed: the stream buffers are free
        if (ok) ok = mbar_wait_warp(bar(ACC_FULL), 0, g.err, 60);
        float out_mul = g.out_mul;
        if (PASS == P_LSE || PASS == P_FWD) {
            // the two warpgroups combine their maxima (MAX) or their sums of P (FWD) through shared memory
            float* xch = reinterpret_cast<float*>(smem_ptr(b3_s));
            xch[wg * BR + rloc] = (PASS == P_LSE) ? m_run : l_run;
            asm volatile("bar.sync 1, 256;" ::: "memory");             // all eight element-wise warps, exactly once
            const float v0 = xch[rloc], v1 = xch[BR + rloc];
            if (PASS == P_LSE) {
                // finite: tile 0 (key 0) belongs to warpgroup 0
                if (wg == 0 && ok && own < g.T) g.lse_out[lb + own] = fmaxf(v0, v1);
            } else {
                const float l = v0 + v1;                               // > 0: the diagonal term
                out_mul *= 1.0f / l;
                if (wg == 0 && ok && own < g.T) g.lse_out[lb + own] = (L + log2f(l)) * kLn2;
            }
        }
        if (PASS != P_LSE && ok) {   // warp-uniform: the tensor-memory loads below need the whole warp
            tc_fence_after();
            const int wrow0 = r0 + lane_group * 32;                    // first row of this warp
            const int nvalid = max(0, min(32, g.T - wrow0));
            const long long off0 = (long long)(row_base + wrow0) * g.out_stride + g.out_col + h * HD + 64 * wg;
            float* sums = g.rg_sums ? g.rg_sums + ((long long)b * g.nrg + (r0 >> 5) + lane_group) * g.out_stride +
                                          g.out_col + h * HD + 64 * wg
                                    : nullptr;
            float* tile = reinterpret_cast<float*>(smem_ptr(b1_s) + (uint32_t)(warp - 2) * kRowTileBytes);
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t r[32];
                tmem_ld32(tOut + t_lane + 64u * wg + 32u * half, r);
                tmem_ld_wait();
                float v[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]) * out_mul;
                warp_rows_store(v, tile, lane, nvalid, g.out_raw ? g.out_raw + off0 + 32 * half : nullptr,
                                g.out_hi ? g.out_hi + off0 + 32 * half : nullptr,
                                g.out_lo ? g.out_lo + off0 + 32 * half : nullptr, g.out_stride,
                                sums ? sums + 32 * half : nullptr);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
}

// Tensor map over a row-major [rows][cols] array given as hi/lo planes: boxes of 32 columns x
// box_rows rows x both planes, in the K-major or the MN-major shared-memory layout.
bool enc128(CUtensorMap* tm, const float* base, int64_t cols, int64_t rows, int64_t plane, uint32_t box_rows,
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

cudaError_t set_attrs() {
    static cudaError_t attr = []() {
        cudaError_t e = cudaFuncSetAttribute(attn128_kernel<P_LSE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attn128_kernel<P_FWD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attn128_kernel<P_DQ>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attn128_kernel<P_DK>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attn128_kernel<P_DV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
        return e;
    }();
    return attr;
}

}  // namespace

cudaError_t attention_tc_default_err(int** out);

bool attention_tc128_supports(int head_dim, int C) { return head_dim == HD && (C % 4) == 0; }

// o (raw and/or hi/lo planes) and lse from the split qkv array.  lse is required: the second pass
// reads what the first one wrote.
cudaError_t launch_attention_fwd_tc128(const float* qkv_hi, int64_t qkv_plane, int B, int T, int C, int H, float* o,
                                       float* o_hi, float* o_lo, float* lse, int* err_word, cudaStream_t s) {
    if (!lse) return cudaErrorInvalidValue;
    cudaError_t e = set_attrs();
    if (e != cudaSuccess) return e;
    if (!err_word && (e = attention_tc_default_err(&err_word)) != cudaSuccess) return e;
    const int64_t rows = (int64_t)B * T, cols = 3 * (int64_t)C;
    CUtensorMap kk, vm;
    if (!enc128(&kk, qkv_hi, cols, rows, qkv_plane, BT_, false) || !enc128(&vm, qkv_hi, cols, rows, qkv_plane, BT_, true))
        return cudaErrorInvalidValue;
    Args128 g{};
    g.T = T; g.C = C; g.H = H;
    g.a1_hi = qkv_hi; g.a1_plane = qkv_plane; g.a1_stride = cols; g.a1_col = 0;
    g.b1_col = C; g.b3_col = 2 * C;
    g.lse_out = lse;
    g.err = err_word;
    g.head_group = B * H;   // one group: groups of heads measured 5 - 10 % slower for these kernels
    dim3 grid(B * H, (T + BR - 1) / BR);
    BT_KERNEL_LAUNCH((attn128_kernel<P_LSE>), grid, kThreads, kSmem, s, kk, kk, kk, vm, g);
    BT_COUNT_LAUNCH();
    g.lse = lse;   // read (the reference) when a CTA starts, overwritten with the log-sum-exp when it ends
    g.out_raw = o; g.out_hi = o_hi; g.out_lo = o_lo; g.out_stride = C; g.out_col = 0; g.out_mul = 1.0f;
    BT_KERNEL_LAUNCH((attn128_kernel<P_FWD>), grid, kThreads, kSmem, s, kk, kk, kk, vm, g);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

// dqkv (hi/lo planes) from qkv (hi/lo planes), dO (hi/lo planes), lse and dvec = rowsum(dO o O);
// rg_sums as in the head_dim-64 kernels (column sums of dqkv per 32-row group, nullable).
cudaError_t launch_attention_bwd_tc128(const float* qkv_hi, int64_t qkv_plane, const float* do_hi, int64_t do_plane,
                                       const float* lse, const float* dvec, int B, int T, int C, int H, float* dqkv_hi,
                                       int64_t dqkv_plane, float* rg_sums, int* err_word, cudaStream_t s) {
    cudaError_t e = set_attrs();
    if (e != cudaSuccess) return e;
    if (!err_word && (e = attention_tc_default_err(&err_word)) != cudaSuccess) return e;
    const int64_t rows = (int64_t)B * T, cols = 3 * (int64_t)C;
    CUtensorMap qkv_k, qkv_m, qkv_res, do_k, do_m, do_res;
    bool ok = enc128(&qkv_k, qkv_hi, cols, rows, qkv_plane, BT_, false) &&
              enc128(&qkv_m, qkv_hi, cols, rows, qkv_plane, BT_, true) &&
              enc128(&qkv_res, qkv_hi, cols, rows, qkv_plane, BR, false) &&
              enc128(&do_k, do_hi, C, rows, do_plane, BT_, false) && enc128(&do_m, do_hi, C, rows, do_plane, BT_, true) &&
              enc128(&do_res, do_hi, C, rows, do_plane, BR, false);
    if (!ok) return cudaErrorInvalidValue;
    Args128 g{};
    g.T = T; g.C = C; g.H = H;
    g.a1_hi = qkv_hi; g.a1_plane = qkv_plane; g.a1_stride = cols;
    g.lse = lse; g.dvec = dvec;
    g.out_hi = dqkv_hi; g.out_lo = dqkv_hi + dqkv_plane; g.out_stride = cols;
    g.rg_sums = rg_sums; g.nrg = 4 * ((T + BR - 1) / BR);
    g.err = err_word;
    g.head_group = B * H;   // one group: groups of heads measured 5 - 10 % slower for these kernels
    const float scale = 1.0f / sqrtf((float)HD);
    dim3 grid(B * H, (T + BR - 1) / BR);
    // dQ: own rows Q (tensor memory) and dO (shared memory); streams K, V, K
    g.a1_col = 0; g.a2_col = 0; g.b1_col = C; g.b2_col = 2 * C; g.b3_col = C; g.out_col = 0; g.out_mul = scale;
    BT_KERNEL_LAUNCH((attn128_kernel<P_DQ>), grid, kThreads, kSmem, s, do_res, qkv_k, qkv_k, qkv_m, g);
    BT_COUNT_LAUNCH();
    // dK: own rows K (tensor memory) and V (shared memory); streams Q, dO, Q
    g.a1_col = C; g.a2_col = 2 * C; g.b1_col = 0; g.b2_col = 0; g.b3_col = 0; g.out_col = C; g.out_mul = scale;
    BT_KERNEL_LAUNCH((attn128_kernel<P_DK>), grid, kThreads, kSmem, s, qkv_res, qkv_k, do_k, qkv_m, g);
    BT_COUNT_LAUNCH();
    // dV: own rows K (tensor memory); streams Q and dO
    g.a1_col = C; g.b1_col = 0; g.b3_col = 0; g.out_col = 2 * C; g.out_mul = 1.0f;
    BT_KERNEL_LAUNCH((attn128_kernel<P_DV>), grid, kThreads, kSmem, s, qkv_res, qkv_k, do_k, do_m, g);
    BT_COUNT_LAUNCH();
    return cudaGetLastError();
}

}  // namespace bt
