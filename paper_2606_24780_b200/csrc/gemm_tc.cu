// FP32 GEMM on the 5th-generation tensor cores with 3xTF32 split accumulation.
//
//   D[M,N] = op(A) op(B) (+ bias) (+ residual),   x*y ~= x_hi*y_hi + x_hi*y_lo + x_lo*y_hi
//
// Operands live in HBM as two FP32 planes (hi = top 19 bits, lo = exact remainder); their
// producers write them that way, so this kernel is a pure TMA -> shared memory -> tcgen05.mma
// -> TMEM pipeline with no conversion work on the SM:
//
//   warp 0 (one lane)  TMA producer: 3-D tiled loads (k, row, plane) of the hi and lo tiles of A
//                      and B into a ring of shared-memory stages, completion on mbarriers.
//   warp 1 (one lane)  MMA issuer: per 8-deep k-step three tcgen05.mma.kind::tf32 (lo*hi, hi*lo,
//                      hi*hi; small terms first) into a 128 x BN FP32 accumulator in TMEM;
//                      tcgen05.commit releases the stage / publishes the accumulator.
//   warps 2-5          epilogue: tcgen05.ld the accumulator (one row per thread), add bias and
//                      residual, store.  Two accumulators alternate so the epilogue of tile i
//                      overlaps the main loop of tile i+1.
//
// The kernel is persistent (one CTA per SM, work units = output tiles x K-splits, tile-row index
// fastest so concurrently running CTAs share the B tile and keep A resident in L2).
//
// Operand layouts.  "K-major" operands (rows of K contiguous: A of NT/NN, B of NT) use the
// 128-byte swizzle; "MN-major" operands (K rows of M or N contiguous: A of TN, B of NN/TN) use
// the 128-byte swizzle with 32-byte atoms, the only shared-memory layout the tensor core accepts
// for transposed 32-bit operands.  Every TMA load targets the issuing CTA's own shared memory only.
//
// Every mbarrier wait is bounded: a wait that runs out raises a device error word and the CTA
// drains and exits, still releasing its TMEM.
#include <cuda.h>

#include <cstdio>
#include <cstdlib>
#include <mutex>

#include "common.cuh"
#include "tc_common.cuh"

namespace bt {

using namespace tc;

namespace {

constexpr int BM = 128;
constexpr int kThreads = 192;
constexpr int kEpiWarps = 4;
constexpr uint32_t kSmemBudget = 227u * 1024u;
// Epilogue staging: each epilogue warp owns a 32 x 32 float tile with a 144-byte row pitch (both the
// row-wise 128-bit writes and the transposed 128-bit reads are then bank-conflict free).
constexpr uint32_t kEpiPitch = 144u;
constexpr uint32_t kEpiStageBytes = kEpiWarps * 32u * kEpiPitch;

// BN: tile width (128, 192 or 256).  BK: floats per k-block; 32 = one 128-byte swizzle row,
// 16 = one 64-byte swizzle row (smaller stages, deeper ring).
template <int BN, int BK>
struct Cfg {
    static constexpr uint32_t kATileBytes = 2u * BM * BK * 4u;  // hi + lo
    static constexpr uint32_t kBTileBytes = 2u * BN * BK * 4u;
    static constexpr uint32_t kStageBytes = kATileBytes + kBTileBytes;
    static constexpr int kStagesFit = (int)((kSmemBudget - 2048u - kEpiStageBytes) / kStageBytes);
    static constexpr int kStages = kStagesFit > 8 ? 8 : kStagesFit;
    static constexpr uint32_t kAccStride = (BN <= 128) ? 128u : 256u;  // TMEM columns per accumulator
    static constexpr uint32_t kTmemCols = 2u * kAccStride;             // 256 or 512 (power of two)
    static constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + kEpiStageBytes + 256;
};

struct GemmArgs {
    int M, N, K;
    float* D;
    long long ldd;
    const float* bias;
    const float* residual;
    int tiles_m, tiles_n, splits, kb_per_split, kb_total;
    // Raster of the tiles: groups of group_m row tiles; inside a group the row tiles run fastest, then the
    // column tiles, then the next group.  The units that run at the same time then cover group_m row tiles
    // by (slots / group_m) column tiles: each A and B tile among them is fetched from HBM once and served
    // from L2 to the other CTAs.  group_m >= tiles_m is the plain row-fastest order, 1 column-fastest.
    int group_m;
    float* partials;
    // Tail split (pair kernel, splits == 1): the tiles of the complete rounds run with the whole K; the
    // tail_tiles tiles of the last, partly filled round are cut into tail_splits K ranges, so that this
    // round costs 1 / tail_splits of a tile's time.  Their partial tiles go to `partials`, compact,
    // [split][tail tile][256 x BN]; a second kernel adds them in split order and runs the output path.
    int full_units, tail_tiles, tail_splits, tail_kbps;
    int* err;
    float* d_hi;        // optional TF32 hi/lo planes of the output (lo = d_hi + d_plane)
    long long d_plane;
    int act;            // 0: the planes hold the output; 1 / 2: they hold GELU(output), erf / tanh form;
                        // 3 / 4: as 1 / 2, and D holds GELU'(output) instead of the output;
                        // 5 / 6: `residual` is a pre-activation h and the output is (A B) o GELU'(h);
                        // 7: `residual` holds GELU'(h) itself and the output is (A B) o residual
    float* col_partial; // act 5 - 7: column sums of the output per 32-row group, [ceil(M / 32)][N] (nullable)
};

// Tile and K range of work unit u (K-split launches: all tiles' first range, then all second ranges, ...).
__host__ __device__ __forceinline__ void raster_tile(int t, int tiles_m, int tiles_n, int group_m, int& tm, int& tn) {
    const int per_group = group_m * tiles_n;
    const int grp = t / per_group, rem = t - grp * per_group;
    const int first = grp * group_m;
    const int rows = min(group_m, tiles_m - first);   // the last group may be shorter
    tn = rem / rows;
    tm = first + (rem - tn * rows);
}
__device__ __forceinline__ void decode_unit(const GemmArgs& g, int u, int& tm, int& tn, int& sp) {
    const int tiles = g.tiles_m * g.tiles_n;
    sp = u / tiles;
    raster_tile(u - sp * tiles, g.tiles_m, g.tiles_n, g.group_m, tm, tn);
}

// One work unit of the pair kernel: its tile, its k-block range and, for a partial result, the slot of
// its partial tile (-1: the unit produces the output itself).
struct PairUnit {
    int tm, tn, kb0, kb1, partial;
};
__device__ __forceinline__ PairUnit decode_pair_unit(const GemmArgs& g, int u) {
    PairUnit w;
    if (g.tail_splits > 1) {
        int tile = u, sp = 0;
        w.partial = -1;
        w.kb0 = 0;
        w.kb1 = g.kb_total;
        if (u >= g.full_units) {
            const int v = u - g.full_units;
            sp = v / g.tail_tiles;                       // all tiles' first range, then all second ranges, ...
            tile = g.full_units + v % g.tail_tiles;
            w.kb0 = sp * g.tail_kbps;
            w.kb1 = min(g.kb_total, w.kb0 + g.tail_kbps);
            w.partial = sp * g.tail_tiles + v % g.tail_tiles;
        }
        int sp_unused;
        decode_unit(g, tile, w.tm, w.tn, sp_unused);
        return w;
    }
    int sp;
    decode_unit(g, u, w.tm, w.tn, sp);
    w.kb0 = sp * g.kb_per_split;
    w.kb1 = min(g.kb_total, w.kb0 + g.kb_per_split);
    w.partial = g.splits > 1 ? sp : -1;
    return w;
}

// Descriptor of one 8-deep k-step of an operand tile.
//   K-major (rows of BK floats): [plane][rows][BK]; BK = 32 -> 128B swizzle (mode 2, SBO 1024),
//                                BK = 16 -> 64B swizzle (mode 4, SBO 512); a k-step advances 32 B.
//   MN-major: per 32-wide column group [plane][BK k-rows][128 B], 128B swizzle with 32B atoms
//             (mode 1, SBO = 512: four k-rows; LBO = distance between column groups); a k-step
//             advances 8 k-rows = 1024 B.
template <bool MN, int BK>
__device__ __forceinline__ uint64_t operand_desc(uint32_t tile_base, int rows, bool lo_plane, int kstep) {
    if (MN) {
        constexpr uint32_t kAtom = 2u * BK * 128u;
        uint32_t addr = tile_base + (lo_plane ? BK * 128u : 0u) + (uint32_t)kstep * 8u * 128u;
        return make_desc(addr, kAtom, 512u, 1u);
    } else {
        uint32_t addr = tile_base + (lo_plane ? (uint32_t)rows * BK * 4u : 0u) + (uint32_t)kstep * 32u;
        return (BK == 32) ? make_desc(addr, 16u, 1024u, 2u) : make_desc(addr, 16u, 512u, 4u);
    }
}

template <bool A_MN, bool B_MN, int BN, int BK>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmArgs g) {
    using C = Cfg<BN, BK>;
    constexpr uint32_t kMnAtomBytes = 2u * BK * 128u;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t epi_stage = smem_base + C::kStages * C::kStageBytes;
    const uint32_t bars = epi_stage + kEpiStageBytes;  // 8-byte barriers
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (C::kStages + s); };
    auto tfull_bar = [&](int a) { return bars + 8u * (2 * C::kStages + a); };
    auto tempty_bar = [&](int a) { return bars + 8u * (2 * C::kStages + 2 + a); };
    const uint32_t tmem_slot = bars + 8u * (2 * C::kStages + 4);
    volatile uint32_t* tmem_slot_ptr =
        reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - smem_u32(smem_raw)));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmB);
        for (int s = 0; s < C::kStages; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), kEpiWarps);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot),
                     "r"(C::kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot_ptr;
    // barriers and tensor memory are set up; from here on global memory is read and written
    pdl_wait();
    pdl_trigger();

    const int units = g.tiles_m * g.tiles_n * g.splits;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
                int tm, tn, sp;
                decode_unit(g, u, tm, tn, sp);
                const int kb0 = sp * g.kb_per_split;
                const int kb1 = min(g.kb_total, kb0 + g.kb_per_split);
                for (int kb = kb0; kb < kb1; ++kb, ++it) {
                    const int s = it % C::kStages;
                    const uint32_t ph = (it / C::kStages) & 1u;
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, g.err, 1)) { ok = false; break; }
                    const uint32_t a_dst = smem_base + s * C::kStageBytes;
                    const uint32_t b_dst = a_dst + C::kATileBytes;
                    mbar_expect_tx(full_bar(s), C::kStageBytes);
                    if (A_MN) {
#pragma unroll
                        for (int a = 0; a < BM / 32; ++a)
                            tma_load_3d(a_dst + a * kMnAtomBytes, &tmA, full_bar(s), tm * BM + 32 * a, kb * BK, 0);
                    } else {
                        tma_load_3d(a_dst, &tmA, full_bar(s), kb * BK, tm * BM, 0);
                    }
                    if (B_MN) {
#pragma unroll
                        for (int a = 0; a < BN / 32; ++a)
                            tma_load_3d(b_dst + a * kMnAtomBytes, &tmB, full_bar(s), tn * BN + 32 * a, kb * BK, 0);
                    } else {
                        tma_load_3d(b_dst, &tmB, full_bar(s), kb * BK, tn * BN, 0);
                    }
                }
            }
            if (!ok) {
                // let loads already in flight land before the CTA's shared memory is released
                for (int i = 0; i < 2000; ++i) __nanosleep(1000);
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_tf32(BM, BN, A_MN, B_MN);
            uint32_t it = 0, ut = 0;
            bool ok = true;
            for (int u = blockIdx.x; u < units && ok; u += gridDim.x, ++ut) {
                int tm, tn, sp;
                decode_unit(g, u, tm, tn, sp);
                const int kb0 = sp * g.kb_per_split;
                const int kb1 = min(g.kb_total, kb0 + g.kb_per_split);
                const int acc = ut & 1;
                const uint32_t aph = (ut >> 1) & 1u;
                if (!mbar_wait(tempty_bar(acc), aph ^ 1u, g.err, 2)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)acc * C::kAccStride;
                for (int kb = kb0; kb < kb1; ++kb, ++it) {
                    const int s = it % C::kStages;
                    const uint32_t ph = (it / C::kStages) & 1u;
                    if (!mbar_wait(full_bar(s), ph, g.err, 3)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_base = smem_base + s * C::kStageBytes;
                    const uint32_t b_base = a_base + C::kATileBytes;
#pragma unroll
                    for (int j = 0; j < BK / 8; ++j) {
                        const uint64_t a_hi = operand_desc<A_MN, BK>(a_base, BM, false, j);
                        const uint64_t a_lo = operand_desc<A_MN, BK>(a_base, BM, true, j);
                        const uint64_t b_hi = operand_desc<B_MN, BK>(b_base, BN, false, j);
                        const uint64_t b_lo = operand_desc<B_MN, BK>(b_base, BN, true, j);
                        umma_tf32(d_tmem, a_lo, b_hi, idesc, (kb > kb0 || j > 0) ? 1u : 0u);
                        umma_tf32(d_tmem, a_hi, b_lo, idesc, 1u);
                        umma_tf32(d_tmem, a_hi, b_hi, idesc, 1u);
                    }
                    umma_commit(empty_bar(s));  // stage free once these MMAs have read it
                }
                if (ok) umma_commit(tfull_bar(acc));  // accumulator complete
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue warps
        const int lane_group = warp & 3;  // TMEM lanes 32*lane_group .. +31 belong to this warp
        uint32_t ut = 0;
        bool ok = true;
        for (int u = blockIdx.x; u < units && ok; u += gridDim.x, ++ut) {
            int tm, tn, sp;
            decode_unit(g, u, tm, tn, sp);
            const int acc = ut & 1;
            const uint32_t aph = (ut >> 1) & 1u;
            if (!mbar_wait_warp(tfull_bar(acc), aph, g.err, 4)) { ok = false; break; }
            tc_fence_after();
            float* Dp = g.D;
            long long ldd = g.ldd;
            if (g.splits > 1) {
                Dp = g.partials + (long long)sp * g.M * g.N;
                ldd = g.N;
            }
            const uint32_t t_row = tmem_base + ((uint32_t)(lane_group * 32) << 16) + (uint32_t)acc * C::kAccStride;
            // A thread reads its accumulator row from tensor memory; the warp's 32 x 32 chunk goes
            // through shared memory so that global memory is then touched a full 128-byte row
            // segment at a time (8 lanes x 16 B): lane -> rows sub + 4i, columns 4*cq .. 4*cq+3.
            float* my_stage = reinterpret_cast<float*>(smem_raw + (epi_stage - smem_u32(smem_raw)) +
                                                       (uint32_t)(warp - 2) * 32u * kEpiPitch);
            const int sub = lane >> 3, cq = lane & 7;
            const int row0 = tm * BM + lane_group * 32;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                const int col0 = tn * BN + c * 32;
                if (col0 >= g.N) break;  // warp-uniform
                uint32_t rr[32];
                tmem_ld32(t_row + c * 32, rr);
                tmem_ld_wait();
                float4* wr = reinterpret_cast<float4*>(reinterpret_cast<uint8_t*>(my_stage) + lane * kEpiPitch);
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    wr[q] = make_float4(__uint_as_float(rr[4 * q]), __uint_as_float(rr[4 * q + 1]),
                                        __uint_as_float(rr[4 * q + 2]), __uint_as_float(rr[4 * q + 3]));
                __syncwarp();
                const int col = col0 + 4 * cq;
                float4 csum = make_float4(0.f, 0.f, 0.f, 0.f);   // this lane's 8 rows of its 4 columns (act 3 / 4)
                if (col < g.N) {
                    float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (g.bias) bv = *reinterpret_cast<const float4*>(g.bias + col);
                    // all residual rows of the chunk are requested before the first store (the output
                    // may alias the residual, so the compiler cannot hoist these loads itself)
                    float4 rv[8];
                    if (g.residual) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const int row = row0 + sub + 4 * i;
                            rv[i] = (row < g.M) ? *reinterpret_cast<const float4*>(g.residual + (long long)row * g.ldd + col)
                                                : make_float4(0.f, 0.f, 0.f, 0.f);
                        }
                        if (g.act == 5 || g.act == 6) {   // h -> GELU'(h): 32 independent evaluations, none behind a store
                            const bool th = g.act == 6;
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                rv[i] = make_float4(gelu_grad_f(rv[i].x, th), gelu_grad_f(rv[i].y, th),
                                                    gelu_grad_f(rv[i].z, th), gelu_grad_f(rv[i].w, th));
                        }
                    }
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int r = sub + 4 * i, row = row0 + r;
                        if (row < g.M) {
                            float4 v = *reinterpret_cast<const float4*>(reinterpret_cast<const uint8_t*>(my_stage) +
                                                                        r * kEpiPitch + cq * 16);
                            v = add4(v, bv);
                            if (g.act >= 5) {   // GELU backward: the product times GELU'(h), and its column sums
                                v = make_float4(v.x * rv[i].x, v.y * rv[i].y, v.z * rv[i].z, v.w * rv[i].w);
                                csum = add4(csum, v);
                            } else if (g.residual) {
                                v = add4(v, rv[i]);
                            }
                            float4 pv = v;      // what the hi/lo planes receive
                            if (g.act >= 1 && g.act <= 4) {   // GELU forward: the planes hold GELU(output) ...
                                const bool th = !(g.act & 1);
                                float4 gp;
                                gelu_both_f(v.x, th, pv.x, gp.x);
                                gelu_both_f(v.y, th, pv.y, gp.y);
                                gelu_both_f(v.z, th, pv.z, gp.z);
                                gelu_both_f(v.w, th, pv.w, gp.w);
                                if (g.act >= 3) v = gp;       // ... and D holds GELU'(output) instead of the output
                            }
                            if (Dp) *reinterpret_cast<float4*>(Dp + (long long)row * ldd + col) = v;
                            if (g.d_hi) {
                                float4 hh, ll;
                                split_tf32(pv, hh, ll);
                                float* hrow = g.d_hi + (long long)row * g.ldd + col;
                                *reinterpret_cast<float4*>(hrow) = hh;
                                *reinterpret_cast<float4*>(hrow + g.d_plane) = ll;
                            }
                        }
                    }
                }
                if (g.act >= 5 && g.col_partial) {   // warp-uniform: the 32 rows of this warp, rows sub + 4 i in lane order
                    csum.x += __shfl_xor_sync(0xffffffffu, csum.x, 8);  csum.y += __shfl_xor_sync(0xffffffffu, csum.y, 8);
                    csum.z += __shfl_xor_sync(0xffffffffu, csum.z, 8);  csum.w += __shfl_xor_sync(0xffffffffu, csum.w, 8);
                    csum.x += __shfl_xor_sync(0xffffffffu, csum.x, 16); csum.y += __shfl_xor_sync(0xffffffffu, csum.y, 16);
                    csum.z += __shfl_xor_sync(0xffffffffu, csum.z, 16); csum.w += __shfl_xor_sync(0xffffffffu, csum.w, 16);
                    if (sub == 0 && col < g.N && row0 < g.M)
                        *reinterpret_cast<float4*>(g.col_partial + (long long)(row0 >> 5) * g.N + col) = csum;
                }
                __syncwarp();   // the staging tile is rewritten by the next chunk
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(acc));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::kTmemCols)
                     : "memory");
    }
}

// ------------------------------------------------------------------ CTA-pair variant
//
// The same GEMM on pairs of CTAs (a cluster of two on neighbouring SMs): the pair owns a 256 x BN
// tile, one tcgen05.mma.cta_group::2 of M = 256 covers it, each CTA streams its own 128 rows of A
// and only HALF of the B tile, so a third less operand data enters shared memory per MMA and the
// ring gets deeper (32 KB stages instead of 48 KB).  The even CTA (leader) issues the MMAs and
// owns the "stage full" and "accumulator drained" barriers; completion is broadcast to both CTAs'
// "stage free" / "accumulator full" barriers by the commit.
// The pair kernel has eight epilogue warps (two per tensor-memory lane quadrant, alternate 32-column
// chunks): its main loop is math bound with stages to spare, so the staging tiles of four more warps
// cost it nothing, while the epilogue of a CTA's last tile -- which nothing overlaps -- halves.
constexpr int kEpiWarps2 = 8;
constexpr int kThreads2 = 64 + 32 * kEpiWarps2;
constexpr uint32_t kEpiStageBytes2 = kEpiWarps2 * 32u * kEpiPitch;
template <int BN, int BK>
struct Cfg2 {
    static constexpr uint32_t kATileBytes = 2u * BM * BK * 4u;          // this CTA's 128 rows, hi + lo
    static constexpr uint32_t kBTileBytes = 2u * (BN / 2) * BK * 4u;    // this CTA's half of the columns
    static constexpr uint32_t kStageBytes = kATileBytes + kBTileBytes;
    static constexpr int kStagesFit = (int)((kSmemBudget - 2048u - kEpiStageBytes2) / kStageBytes);
    static constexpr int kStages = kStagesFit > 8 ? 8 : kStagesFit;
    static constexpr uint32_t kAccStride = 256u;
    static constexpr uint32_t kTmemCols = 512u;
    static constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + kEpiStageBytes2 + 256;
};

template <bool A_MN, bool B_MN, int BN, int BK>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads2, 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmArgs g) {
    using C = Cfg2<BN, BK>;
    constexpr int BH = BN / 2;                         // B columns held by one CTA
    constexpr uint32_t kMnAtomBytes = 2u * BK * 128u;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t epi_stage = smem_base + C::kStages * C::kStageBytes;
    const uint32_t bars = epi_stage + kEpiStageBytes2;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (C::kStages + s); };
    auto tfull_bar = [&](int a) { return bars + 8u * (2 * C::kStages + a); };
    auto tempty_bar = [&](int a) { return bars + 8u * (2 * C::kStages + 2 + a); };
    const uint32_t tmem_slot = bars + 8u * (2 * C::kStages + 4);
    volatile uint32_t* tmem_slot_ptr =
        reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_slot - smem_u32(smem_raw)));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();          // 0 = leader
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmB);
        for (int s = 0; s < C::kStages; ++s) {
            mbar_init(full_bar(s), 1);                 // used in the leader: its producer's expect_tx arrival
            mbar_init(empty_bar(s), 1);                // one commit per use, delivered to both CTAs
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull_bar(a), 1);
            mbar_init(tempty_bar(a), 2 * kEpiWarps2);   // used in the leader: both CTAs' epilogue warps
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot),
                     "r"(C::kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();      // the partner's barriers exist before anything is signalled across the pair
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot_ptr;
    pdl_wait();
    pdl_trigger();

    // tiles_m counts 256-row tiles here
    const int units = g.tail_splits > 1 ? g.full_units + g.tail_tiles * g.tail_splits : g.tiles_m * g.tiles_n * g.splits;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer (both CTAs)
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int u = pair; u < units && ok; u += n_pairs) {
                const PairUnit w = decode_pair_unit(g, u);
                const int kb0 = w.kb0, kb1 = w.kb1;
                const int a_row = w.tm * 2 * BM + (int)rank * BM;    // first A row (or column, if MN-major) of this CTA
                const int b_col = w.tn * BN + (int)rank * BH;        // first B column of this CTA
                for (int kb = kb0; kb < kb1; ++kb, ++it) {
                    const int s = it % C::kStages;
                    const uint32_t ph = (it / C::kStages) & 1u;
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, g.err, 5)) { ok = false; break; }
                    const uint32_t a_dst = smem_base + s * C::kStageBytes;
                    const uint32_t b_dst = a_dst + C::kATileBytes;
                    const uint32_t lbar = mapa_shared(full_bar(s), 0);   // the leader's barrier collects both halves
                    if (rank == 0) mbar_expect_tx(full_bar(s), 2u * C::kStageBytes);
                    if (A_MN) {
#pragma unroll
                        for (int a = 0; a < BM / 32; ++a)
                            tma_load_3d_pair(a_dst + a * kMnAtomBytes, &tmA, lbar, a_row + 32 * a, kb * BK, 0);
                    } else {
                        tma_load_3d_pair(a_dst, &tmA, lbar, kb * BK, a_row, 0);
                    }
                    if (B_MN) {
#pragma unroll
                        for (int a = 0; a < BH / 32; ++a)
                            tma_load_3d_pair(b_dst + a * kMnAtomBytes, &tmB, lbar, b_col + 32 * a, kb * BK, 0);
                    } else {
                        tma_load_3d_pair(b_dst, &tmB, lbar, kb * BK, b_col, 0);
                    }
                }
            }
            if (!ok)
                for (int i = 0; i < 2000; ++i) __nanosleep(1000);
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer (leader only)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = make_idesc_tf32(2 * BM, BN, A_MN, B_MN);
            uint32_t it = 0, ut = 0;
            bool ok = true;
            for (int u = pair; u < units && ok; u += n_pairs, ++ut) {
                const PairUnit w = decode_pair_unit(g, u);
                const int kb0 = w.kb0, kb1 = w.kb1;
                const int acc = ut & 1;
                const uint32_t aph = (ut >> 1) & 1u;
                if (!mbar_wait(tempty_bar(acc), aph ^ 1u, g.err, 6)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)acc * C::kAccStride;
                for (int kb = kb0; kb < kb1; ++kb, ++it) {
                    const int s = it % C::kStages;
                    const uint32_t ph = (it / C::kStages) & 1u;
                    if (!mbar_wait(full_bar(s), ph, g.err, 7)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_base = smem_base + s * C::kStageBytes;
                    const uint32_t b_base = a_base + C::kATileBytes;
#pragma unroll
                    for (int j = 0; j < BK / 8; ++j) {
                        const uint64_t a_hi = operand_desc<A_MN, BK>(a_base, BM, false, j);
                        const uint64_t a_lo = operand_desc<A_MN, BK>(a_base, BM, true, j);
                        const uint64_t b_hi = operand_desc<B_MN, BK>(b_base, BH, false, j);
                        const uint64_t b_lo = operand_desc<B_MN, BK>(b_base, BH, true, j);
                        umma2_tf32(d_tmem, a_lo, b_hi, idesc, (kb > kb0 || j > 0) ? 1u : 0u);
                        umma2_tf32(d_tmem, a_hi, b_lo, idesc, 1u);
                        umma2_tf32(d_tmem, a_hi, b_hi, idesc, 1u);
                    }
                    umma2_commit(empty_bar(s), (uint16_t)3);   // both CTAs may refill this stage
                }
                if (ok) umma2_commit(tfull_bar(acc), (uint16_t)3);
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue warps (both CTAs)
        const int lane_group = warp & 3;
        uint32_t ut = 0;
        bool ok = true;
        const uint32_t my_tempty0 = mapa_shared(tempty_bar(0), 0), my_tempty1 = mapa_shared(tempty_bar(1), 0);
        for (int u = pair; u < units && ok; u += n_pairs, ++ut) {
            const PairUnit w = decode_pair_unit(g, u);
            const int tm = w.tm, tn = w.tn;
            const int acc = ut & 1;
            const uint32_t aph = (ut >> 1) & 1u;
            if (!mbar_wait_warp(tfull_bar(acc), aph, g.err, 8)) { ok = false; break; }
            tc_fence_after();
            float* Dp = g.D;
            long long ldd = g.ldd;
            if (g.splits > 1) {
                Dp = g.partials + (long long)w.partial * g.M * g.N;
                ldd = g.N;
            }
            // a K range of a tail tile: the raw sums go to the tile's compact partial slot (addressed so
            // that the global row / column arithmetic below lands inside it); no bias, residual or planes
            const bool tail_partial = g.tail_splits > 1 && w.partial >= 0;
            if (tail_partial) {
                ldd = BN;
                Dp = g.partials + ((long long)w.partial * (2 * BM) - (long long)tm * (2 * BM)) * BN - (long long)tn * BN;
            }
            const uint32_t t_row = tmem_base + ((uint32_t)(lane_group * 32) << 16) + (uint32_t)acc * C::kAccStride;
            float* my_stage = reinterpret_cast<float*>(smem_raw + (epi_stage - smem_u32(smem_raw)) +
                                                       (uint32_t)(warp - 2) * 32u * kEpiPitch);
            const int sub = lane >> 3, cq = lane & 7;
            const int row0 = tm * 2 * BM + (int)rank * BM + lane_group * 32;
#pragma unroll 1
            for (int c = (warp - 2) >> 2; c < BN / 32; c += 2) {   // the quadrant's two warps take alternate chunks
                const int col0 = tn * BN + c * 32;
                if (col0 >= g.N) break;  // warp-uniform
                uint32_t rr[32];
                tmem_ld32(t_row + c * 32, rr);
                tmem_ld_wait();
                float4* wr = reinterpret_cast<float4*>(reinterpret_cast<uint8_t*>(my_stage) + lane * kEpiPitch);
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    wr[q] = make_float4(__uint_as_float(rr[4 * q]), __uint_as_float(rr[4 * q + 1]),
                                        __uint_as_float(rr[4 * q + 2]), __uint_as_float(rr[4 * q + 3]));
                __syncwarp();
                const int col = col0 + 4 * cq;
                float4 csum = make_float4(0.f, 0.f, 0.f, 0.f);   // this lane's 8 rows of its 4 columns (act 3 / 4)
                if (col < g.N) {
                    float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (g.bias && !tail_partial) bv = *reinterpret_cast<const float4*>(g.bias + col);
                    float4 rv[8];
                    if (g.residual && !tail_partial) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const int row = row0 + sub + 4 * i;
                            rv[i] = (row < g.M) ? *reinterpret_cast<const float4*>(g.residual + (long long)row * g.ldd + col)
                                                : make_float4(0.f, 0.f, 0.f, 0.f);
                        }
                        if ((g.act == 5 || g.act == 6) && !tail_partial) {   // h -> GELU'(h): 32 independent evaluations, none behind a store
                            const bool th = g.act == 6;
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                rv[i] = make_float4(gelu_grad_f(rv[i].x, th), gelu_grad_f(rv[i].y, th),
                                                    gelu_grad_f(rv[i].z, th), gelu_grad_f(rv[i].w, th));
                        }
                    }
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int rr_ = sub + 4 * i, row = row0 + rr_;
                        if (row < g.M) {
                            float4 v = *reinterpret_cast<const float4*>(reinterpret_cast<const uint8_t*>(my_stage) +
                                                                        rr_ * kEpiPitch + cq * 16);
                            v = add4(v, bv);
                            if (g.act >= 5 && !tail_partial) {   // GELU backward: the product times GELU'(h), and its column sums
                                v = make_float4(v.x * rv[i].x, v.y * rv[i].y, v.z * rv[i].z, v.w * rv[i].w);
                                csum = add4(csum, v);
                            } else if (g.residual && !tail_partial) {
                                v = add4(v, rv[i]);
                            }
                            float4 pv = v;      // what the hi/lo planes receive
                            if (g.act >= 1 && g.act <= 4 && !tail_partial) {   // GELU forward: the planes hold GELU(output) ...
                                const bool th = !(g.act & 1);
                                float4 gp;
                                gelu_both_f(v.x, th, pv.x, gp.x);
                                gelu_both_f(v.y, th, pv.y, gp.y);
                                gelu_both_f(v.z, th, pv.z, gp.z);
                                gelu_both_f(v.w, th, pv.w, gp.w);
                                if (g.act >= 3) v = gp;       // ... and D holds GELU'(output) instead of the output
                            }
                            if (Dp) *reinterpret_cast<float4*>(Dp + (long long)row * ldd + col) = v;
                            if (g.d_hi && !tail_partial) {
                                float4 hh, ll;
                                split_tf32(pv, hh, ll);
                                float* hrow = g.d_hi + (long long)row * g.ldd + col;
                                *reinterpret_cast<float4*>(hrow) = hh;
                                *reinterpret_cast<float4*>(hrow + g.d_plane) = ll;
                            }
                        }
                    }
                }
                if (g.act >= 5 && g.col_partial && !tail_partial) {   // warp-uniform: the 32 rows of this warp, rows sub + 4 i in lane order
                    csum.x += __shfl_xor_sync(0xffffffffu, csum.x, 8);  csum.y += __shfl_xor_sync(0xffffffffu, csum.y, 8);
                    csum.z += __shfl_xor_sync(0xffffffffu, csum.z, 8);  csum.w += __shfl_xor_sync(0xffffffffu, csum.w, 8);
                    csum.x += __shfl_xor_sync(0xffffffffu, csum.x, 16); csum.y += __shfl_xor_sync(0xffffffffu, csum.y, 16);
                    csum.z += __shfl_xor_sync(0xffffffffu, csum.z, 16); csum.w += __shfl_xor_sync(0xffffffffu, csum.w, 16);
                    if (sub == 0 && col < g.N && row0 < g.M)
                        *reinterpret_cast<float4*>(g.col_partial + (long long)(row0 >> 5) * g.N + col) = csum;
                }
                __syncwarp();
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(acc ? my_tempty1 : my_tempty0);   // on the leader's barrier
        }
    }

    // The partner's shared and tensor memory stay in use by the pair's MMAs until both CTAs are done.
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::kTmemCols)
                     : "memory");
    }
}

// ------------------------------------------------------------------ host side

EncodeTiledFn g_encode = nullptr;
int g_num_sms = 0;
int g_bk = 16;       // k-block depth in use (BT_GEMM_BK=32 selects the 128-byte-row variant)
int g_force_bn = 0;  // BT_GEMM_BN=128|192|256 pins the tile width (tuning aid)
// Measured time of a CTA-pair tile relative to two single-CTA tiles of the same width: 256-wide pair
// tiles run about 5 % faster (a third less operand data into shared memory), 192-wide ones slower.
int g_group_m = 0;      // BT_GEMM_GROUPM=n pins the raster's group height (tuning aid); 0: chosen per GEMM
int g_tail_split = 1;   // BT_GEMM_TAIL=0 turns the tail split off (tuning aid)
double kTwoCtaFactor256 = 0.95, kTwoCtaFactor192 = 1.03;   // BT_GEMM_F256 / BT_GEMM_F192 override (tuning aid)
int g_two_cta = -1;  // BT_GEMM_2CTA=0 never / 1 always (where the shape allows) / unset: the planner decides
std::once_flag g_once;
char g_init_err[256] = {0};

template <bool A_MN, bool B_MN, int BN, int BK>
cudaError_t set_attr() {
    return cudaFuncSetAttribute(gemm_tc_kernel<A_MN, B_MN, BN, BK>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)Cfg<BN, BK>::kSmemBytes);
}
template <bool A_MN, bool B_MN, int BN, int BK>
cudaError_t set_attr2() {
    return cudaFuncSetAttribute(gemm_tc2_kernel<A_MN, B_MN, BN, BK>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)Cfg2<BN, BK>::kSmemBytes);
}
template <bool A_MN, bool B_MN>
cudaError_t set_attr_layout() {
    {
        cudaError_t b = set_attr2<A_MN, B_MN, 256, 16>();
        if (b == cudaSuccess) b = set_attr2<A_MN, B_MN, 192, 16>();
        if (b == cudaSuccess) b = set_attr2<A_MN, B_MN, 256, 32>();
        if (b == cudaSuccess) b = set_attr2<A_MN, B_MN, 192, 32>();
        if (b != cudaSuccess) return b;
    }
    cudaError_t a = set_attr<A_MN, B_MN, 256, 16>();
    if (a == cudaSuccess) a = set_attr<A_MN, B_MN, 192, 16>();
    if (a == cudaSuccess) a = set_attr<A_MN, B_MN, 128, 16>();
    if (a == cudaSuccess) a = set_attr<A_MN, B_MN, 256, 32>();
    if (a == cudaSuccess) a = set_attr<A_MN, B_MN, 192, 32>();
    if (a == cudaSuccess) a = set_attr<A_MN, B_MN, 128, 32>();
    return a;
}

void init_once() {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
    if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !fn) {
        snprintf(g_init_err, sizeof(g_init_err), "cuTensorMapEncodeTiled not available: %s", cudaGetErrorString(e));
        return;
    }
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&g_num_sms, cudaDevAttrMultiProcessorCount, dev);
    if (const char* v = getenv("BT_GEMM_BK")) g_bk = (atoi(v) == 32) ? 32 : 16;
    if (const char* v = getenv("BT_GEMM_2CTA")) g_two_cta = atoi(v) ? 1 : 0;
    if (const char* v = getenv("BT_GEMM_TAIL")) g_tail_split = atoi(v) ? 1 : 0;
    if (const char* v = getenv("BT_GEMM_GROUPM")) g_group_m = atoi(v) > 0 ? atoi(v) : 0;
    if (const char* v = getenv("BT_GEMM_F256")) kTwoCtaFactor256 = atof(v);
    if (const char* v = getenv("BT_GEMM_F192")) kTwoCtaFactor192 = atof(v);
    if (const char* v = getenv("BT_GEMM_BN")) {
        int bn = atoi(v);
        if (bn == 128 || bn == 192 || bn == 256) g_force_bn = bn;
    }
    cudaError_t a = set_attr_layout<false, false>();
    if (a == cudaSuccess) a = set_attr_layout<false, true>();
    if (a == cudaSuccess) a = set_attr_layout<true, true>();
    if (a != cudaSuccess) {
        snprintf(g_init_err, sizeof(g_init_err), "cudaFuncSetAttribute(smem) failed: %s", cudaGetErrorString(a));
        return;
    }
    g_encode = (EncodeTiledFn)fn;
}

// 3-D map over a split matrix: (contiguous cols, rows, plane).
bool encode_map(CUtensorMap* tm, const SplitMat& m, uint32_t box_cols, uint32_t box_rows, CUtensorMapSwizzle sw) {
    cuuint64_t dims[3] = {(cuuint64_t)m.cols, (cuuint64_t)m.rows, 2};
    cuuint64_t strides[2] = {(cuuint64_t)m.ld * 4, (cuuint64_t)m.plane * 4};
    cuuint32_t box[3] = {box_cols, box_rows, 2};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, (void*)m.hi, dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

constexpr int kMaxUnitsForSplit = 4 * 148;


// The tail split's second pass: out = sum over the K ranges (in range order) of a tail tile's partial
// tiles, then the output path exactly as the GEMM's own epilogue runs it: bias, residual, the GELU
// forward modes (act 1 - 4) and the hi/lo planes.
__global__ void __launch_bounds__(256) tail_reduce_kernel(const float* __restrict__ partials, int splits, int tail_tiles,
                                                          int first_tile, int tiles_m, int tiles_n, int group_m, int bn, int M, int N,
                                                          float* D,
                                                          long long ldd, const float* __restrict__ bias,
                                                          const float* residual, float* d_hi, long long d_plane, int act) {
    pdl_wait();
    pdl_trigger();
    const int bn4 = bn / 4;
    const long long per_tile4 = 256LL * bn4, total = (long long)tail_tiles * per_tile4;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int j = (int)(i / per_tile4);
        const long long r = i - (long long)j * per_tile4;
        const int lr = (int)(r / bn4), c4 = (int)(r - (long long)lr * bn4);
        const int tile = first_tile + j;
        int tm, tn;
        raster_tile(tile, tiles_m, tiles_n, group_m, tm, tn);
        const int row = tm * 256 + lr, col = tn * bn + 4 * c4;
        if (row >= M || col >= N) continue;
        float4 t = ld4(partials, (long long)j * per_tile4 + r);
        for (int sp = 1; sp < splits; ++sp) t = add4(t, ld4(partials, ((long long)sp * tail_tiles + j) * per_tile4 + r));
        if (bias) t = add4(t, *reinterpret_cast<const float4*>(bias + col));
        const long long off = (long long)row * ldd + col;
        if (residual) t = add4(t, *reinterpret_cast<const float4*>(residual + off));
        float4 pv = t;
        if (act >= 1 && act <= 4) {
            const bool th = !(act & 1);
            float4 gp;
            gelu_both_f(t.x, th, pv.x, gp.x);
            gelu_both_f(t.y, th, pv.y, gp.y);
            gelu_both_f(t.z, th, pv.z, gp.z);
            gelu_both_f(t.w, th, pv.w, gp.w);
            if (act >= 3) t = gp;
        }
        if (D) *reinterpret_cast<float4*>(D + off) = t;
        if (d_hi) {
            float4 hh, ll;
            split_tf32(pv, hh, ll);
            *reinterpret_cast<float4*>(d_hi + off) = hh;
            *reinterpret_cast<float4*>(d_hi + d_plane + off) = ll;
        }
    }
}

struct Plan {
    int bn, splits, kb_per_split;
    double cost;
    bool two_cta;   // 256-row tiles on CTA pairs
    int tail_tiles, tail_splits, tail_kbps;   // pair tiles only: the last, partly filled round cut along K (0: not used)
};

// Picks tile width and K-split by a simple wave model.  Every work unit of one launch costs the
// same, so the launch takes ceil(units / SMs) unit times; a unit is (k-blocks + fixed overhead)
// x tile width, narrower tiles pay a small efficiency penalty, and a K-split pays for writing
// and re-reading its partial sums.
Plan make_plan(int64_t M, int64_t N, int kb_total, int bk, int sms, bool can_split, size_t max_partial_floats,
               int two_cta_mode,     // -1: the planner decides, 0: single-CTA tiles only, 1: pair tiles where M >= 256
               bool can_tail) {      // a tail split may be used (a partial buffer exists, no activation in the epilogue)
    const int tiles_m = (int)((M + BM - 1) / BM);
    const double kOverheadKb = 96.0 / bk;                     // pipeline fill + exposed epilogue, in k-blocks
    const double kb_seconds = 768.0 * (bk / 16.0) / 1.9e9;    // one 128x256 k-block of 3 MMAs at peak
    static const int kSplits[] = {1, 2, 3, 4, 5, 6, 8, 10, 12, 16, 20, 24, 32};
    // The tensor core adds into its FP32 accumulator with truncation: a chain of n MMAs can drift by
    // n 2^-25 of the running sum.  Where a K split is possible, no chain is longer than 8192 MMAs
    // (K = 21,845: only the input gradient of the LM head, K = 50,304, is affected).
    const int max_chain_kb = 8192 / (3 * (bk / 8));
    Plan best{256, 1, kb_total, 1e300, false, 0, 0, 0};
    for (int two = 0; two < 2; ++two) {
        if (two && (two_cta_mode == 0 || M < 256)) continue;
        if (!two && two_cta_mode == 1 && M >= 256) continue;
        for (int bn : {256, 192, 128}) {
            if (g_force_bn && bn != g_force_bn) continue;
            if (two && bn == 128) continue;
            if (bn > 128 && N <= bn - 64) continue;               // mostly padding
            const double pen = (bn == 256 ? 1.0 : bn == 192 ? 1.04 : 1.12) *
                               (two ? (bn == 256 ? kTwoCtaFactor256 : kTwoCtaFactor192) : 1.0);
            const long long tm = two ? (M + 2 * BM - 1) / (2 * BM) : tiles_m;
            const long long tiles = tm * ((N + bn - 1) / bn);
            const int slots = two ? sms / 2 : sms;
            for (int sp : kSplits) {
                if (sp > 1 && (!can_split || kb_total / sp < 8 || (size_t)sp * M * N > max_partial_floats)) continue;
                const int kbps = (kb_total + sp - 1) / sp;
                const int real_sp = (kb_total + kbps - 1) / kbps;
                if (real_sp != sp) continue;
                if (can_split && kbps > max_chain_kb && sp < 32) continue;
                const long long units = tiles * sp;
                const long long rounds = (units + slots - 1) / slots;
                double cost = (double)rounds * (kbps + kOverheadKb) * (bn / 256.0) * pen;
                if (sp > 1) cost += (double)(sp + 1) * M * N * 4.0 / 6.0e12 / kb_seconds;
                if (cost < best.cost) best = Plan{bn, sp, kbps, cost, two != 0, 0, 0, 0};
            }
            // Tail split: with few tiles per slot the last round is the expensive one (96 pair tiles on 74
            // pairs: two rounds for 1.3 rounds of work).  Its tiles are cut into as many K ranges as fill
            // the idle slots, so the round costs a fraction of a tile's time plus a small reduction pass.
            const long long full_rounds = tiles / slots, tail = tiles % slots;
            if (two && can_tail && g_tail_split && full_rounds >= 1 && tail > 0 && 2 * tail <= slots &&
                !(can_split && kb_total > max_chain_kb)) {
                int sp = (int)(slots / tail);
                if (sp > 8) sp = 8;
                while (sp > 1 && kb_total / sp < 8) --sp;
                const int kbps = (kb_total + sp - 1) / sp;
                const int real_sp = (kb_total + kbps - 1) / kbps;
                const size_t need = (size_t)real_sp * (size_t)tail * 256u * (size_t)bn;
                if (real_sp > 1 && need <= max_partial_floats) {
                    double cost = ((double)full_rounds * (kb_total + kOverheadKb) + (kbps + kOverheadKb)) * (bn / 256.0) * pen;
                    cost += ((double)(real_sp + 2) * tail * 256.0 * bn * 4.0 / 6.0e12 + 3.0e-6) / kb_seconds;   // the reduction pass and its launch
                    if (cost < best.cost) best = Plan{bn, 1, kb_total, cost, true, (int)tail, real_sp, kbps};
                }
            }
        }
    }
    return best;
}

}  // namespace

namespace tc {
EncodeTiledFn tensor_map_encoder() {
    gemm_tc_init(nullptr, 0);
    return g_encode;
}
int sm_count() {
    gemm_tc_init(nullptr, 0);
    return g_num_sms > 0 ? g_num_sms : 148;
}
}  // namespace tc

bool gemm_tc_init(char* err, size_t errlen) {
    std::call_once(g_once, init_once);
    if (!g_encode && err) snprintf(err, errlen, "%s", g_init_err);
    return g_encode != nullptr;
}

size_t gemm_tc_partial_floats_bound() { return (size_t)kMaxUnitsForSplit * BM * 256; }

// Partial-sum floats a product needs so that the planner can keep every accumulation chain within its
// cap (8192 MMAs) by cutting K: 0 where the whole K fits in one chain.
size_t gemm_tc_partial_floats_for_chain_cap(int64_t M, int64_t N, int64_t K) {
    const int bk = g_bk > 0 ? g_bk : 16;
    const int64_t kb_total = (K + bk - 1) / bk, max_chain_kb = 8192 / (3 * (bk / 8));
    const int64_t splits = (kb_total + max_chain_kb - 1) / max_chain_kb;
    return splits > 1 ? (size_t)splits * (size_t)M * (size_t)N : 0;
}

// What the planner would choose for a product (host arithmetic only; 148 SMs are assumed where no
// device has been initialised): out = {tile width, 1 if 256-row pair tiles, K splits, tail tiles,
// K ranges per tail tile, k-blocks per range}.
// Group height of the tile raster.  The `slots` units that run at the same time cover g row tiles by
// slots / g column tiles (several groups if a group has fewer units), walk K together, and share each A
// and B tile among them through L2; what the next set of units needs again has by then been pushed out by
// the operands and outputs streamed in between (an effective 40 MB of the L2 predicts the measured order
// of the group heights).  With the plain row-fastest order and at least `slots` row tiles, A is fetched
// from HBM once per tile column; with one row tile per group, B once per tile row.  Measured over the
// GPT-2 shapes at 8,192 and 32,768 rows: with few tile columns (N = 768 ... 3,072) groups of 4 are
// best or within 2 % of it (the units that share an A tile then sit on neighbouring CTAs); with many (the
// LM head: 197) 8 to 32, and 4 re-reads B too often.  Group heights of 1 and 2 were up to 17 % slower
// than 4 on the K-split LM-head input gradient and are not used.
int choose_group_m(int tiles_m, int tiles_n, int slots) {
    int g = g_group_m > 0 ? g_group_m : (4 * tiles_n <= slots ? 4 : 16);
    return g < tiles_m ? g : tiles_m;
}

void gemm_tc_plan_info(int64_t M, int64_t N, int64_t K, bool can_split, bool can_tail, int two_cta_mode, int out[7]) {
    const int sms = g_num_sms > 0 ? g_num_sms : 148;
    const int kb_total = (int)((K + g_bk - 1) / g_bk);
    const Plan p = make_plan(M, N, kb_total, g_bk, sms, can_split, gemm_tc_partial_floats_bound(),
                             two_cta_mode >= 0 ? two_cta_mode : g_two_cta, can_tail);
    out[0] = p.bn; out[1] = p.two_cta ? 1 : 0; out[2] = p.splits;
    out[3] = p.tail_tiles; out[4] = p.tail_splits; out[5] = p.tail_kbps;
    const int tiles_m = p.two_cta ? (int)((M + 2 * BM - 1) / (2 * BM)) : (int)((M + BM - 1) / BM);
    const int tiles_n = (int)((N + p.bn - 1) / p.bn);
    out[6] = choose_group_m(tiles_m, tiles_n, p.two_cta ? sms / 2 : sms);
}


template <int BK>
static cudaError_t launch_bk(int layout, int64_t M, int64_t N, int64_t K, const SplitMat& A, const SplitMat& B,
                             float* D, int64_t ldd, const float* bias, const float* residual, float* partials,
                             size_t max_partial_floats, int* err_word, float* d_hi, int64_t d_plane,
                             cudaStream_t s, int two_cta_mode, int act, float* col_partial) {
    const bool a_mn = (layout == kTN), b_mn = (layout != kNT);
    const int sms = g_num_sms > 0 ? g_num_sms : 148;
    const int kb_total = (int)((K + BK - 1) / BK);
    const bool can_split = !bias && !residual && partials && ldd == N && D && !d_hi;
    // (the GELU backward modes are left out: a reduction pass that also forms their column sums -- 32 rows
    // per thread -- was measured slower than the second round it replaces)
    const bool can_tail = partials && (D || d_hi) && act < 5;
    const Plan plan = make_plan(M, N, kb_total, BK, sms, can_split, max_partial_floats,
                                two_cta_mode >= 0 ? two_cta_mode : g_two_cta, can_tail);
    const int bn = plan.bn;

    const CUtensorMapSwizzle sw_k = (BK == 32) ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
    const CUtensorMapSwizzle sw_mn = CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B;
    CUtensorMap tmA, tmB;
    bool ok = a_mn ? encode_map(&tmA, A, 32, BK, sw_mn) : encode_map(&tmA, A, BK, BM, sw_k);
    ok = ok && (b_mn ? encode_map(&tmB, B, 32, BK, sw_mn)
                     : encode_map(&tmB, B, BK, (uint32_t)(plan.two_cta ? bn / 2 : bn), sw_k));
    if (!ok) return cudaErrorInvalidValue;

    GemmArgs g;
    g.M = (int)M; g.N = (int)N; g.K = (int)K;
    g.D = D; g.ldd = ldd; g.bias = bias; g.residual = residual;
    g.tiles_m = plan.two_cta ? (int)((M + 2 * BM - 1) / (2 * BM)) : (int)((M + BM - 1) / BM);
    g.tiles_n = (int)((N + bn - 1) / bn);
    g.splits = plan.splits;
    g.kb_per_split = plan.kb_per_split; g.kb_total = kb_total;
    g.group_m = choose_group_m(g.tiles_m, g.tiles_n, plan.two_cta ? sms / 2 : sms);
    g.partials = partials; g.err = err_word;
    g.tail_tiles = plan.tail_tiles; g.tail_splits = plan.tail_splits; g.tail_kbps = plan.tail_kbps;
    g.full_units = g.tiles_m * g.tiles_n - plan.tail_tiles;
    g.d_hi = d_hi; g.d_plane = d_plane; g.act = (d_hi || act >= 5) ? act : 0;
    g.col_partial = act >= 5 ? col_partial : nullptr;
    const long long units = plan.tail_splits > 1 ? (long long)g.full_units + (long long)plan.tail_tiles * plan.tail_splits
                                                 : (long long)g.tiles_m * g.tiles_n * g.splits;
    const int grid = (int)(units < sms ? units : sms);
    if (plan.two_cta) {
        const int pairs = (int)(units < sms / 2 ? units : sms / 2);
#define BT_LAUNCH2(AM, BMN, BNV)                                                                             \
    BT_KERNEL_LAUNCH((gemm_tc2_kernel<AM, BMN, BNV, BK>), 2 * pairs, kThreads2, (Cfg2<BNV, BK>::kSmemBytes), s, tmA, tmB, g)
#define BT_LAUNCH2_BN(BNV)                                                                                   \
    do {                                                                                                     \
        if (layout == kNT) BT_LAUNCH2(false, false, BNV);                                                    \
        else if (layout == kNN) BT_LAUNCH2(false, true, BNV);                                                \
        else BT_LAUNCH2(true, true, BNV);                                                                    \
    } while (0)
        if (bn == 256) BT_LAUNCH2_BN(256);
        else BT_LAUNCH2_BN(192);
#undef BT_LAUNCH2_BN
#undef BT_LAUNCH2
        BT_COUNT_LAUNCH();
        cudaError_t e2 = cudaGetLastError();
        if (e2 != cudaSuccess) return e2;
        if (g.splits > 1) return launch_splitk_reduce(partials, g.splits, M * N, D, s);
        if (g.tail_splits > 1) {
            const long long n4 = (long long)g.tail_tiles * 256 * (bn / 4);
            const long long want = (n4 + 255) / 256;
            const int rgrid = (int)(want < 148 * 16 ? want : 148 * 16);
            BT_KERNEL_LAUNCH((tail_reduce_kernel), rgrid, 256, 0, s, (const float*)partials, g.tail_splits, g.tail_tiles,
                             g.full_units, g.tiles_m, g.tiles_n, g.group_m, bn, g.M, g.N, D, (long long)ldd, bias, residual, d_hi,
                             (long long)d_plane, g.act);
            BT_COUNT_LAUNCH();
            return cudaGetLastError();
        }
        return cudaSuccess;
    }

#define BT_LAUNCH(AM, BMN, BNV)                                                                              \
    BT_KERNEL_LAUNCH((gemm_tc_kernel<AM, BMN, BNV, BK>), grid, kThreads, (Cfg<BNV, BK>::kSmemBytes), s, tmA, tmB, g)
#define BT_LAUNCH_BN(BNV)                                                                                    \
    do {                                                                                                     \
        if (layout == kNT) BT_LAUNCH(false, false, BNV);                                                     \
        else if (layout == kNN) BT_LAUNCH(false, true, BNV);                                                 \
        else BT_LAUNCH(true, true, BNV);                                                                     \
    } while (0)
    if (bn == 256) BT_LAUNCH_BN(256);
    else if (bn == 192) BT_LAUNCH_BN(192);
    else BT_LAUNCH_BN(128);
#undef BT_LAUNCH_BN
#undef BT_LAUNCH
    BT_COUNT_LAUNCH();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (g.splits > 1) return launch_splitk_reduce(partials, g.splits, M * N, D, s);
    return cudaSuccess;
}

cudaError_t launch_gemm_tc(int layout, int64_t M, int64_t N, int64_t K, SplitMat A, SplitMat B, float* D, int64_t ldd,
                           const float* bias, const float* residual, float* partials, size_t max_partial_floats,
                           int* err_word, cudaStream_t s, float* d_hi, int64_t d_plane, int two_cta_mode, int act,
                           float* col_partial) {
    if (!gemm_tc_init(nullptr, 0)) return cudaErrorNotSupported;
    if (!D && !d_hi) return cudaErrorInvalidValue;
    if (act >= 5 && (!residual || bias)) return cudaErrorInvalidValue;   // the gate operand travels as `residual`
    if (g_bk == 32)
        return launch_bk<32>(layout, M, N, K, A, B, D, ldd, bias, residual, partials, max_partial_floats, err_word,
                             d_hi, d_plane, s, two_cta_mode, act, col_partial);
    return launch_bk<16>(layout, M, N, K, A, B, D, ldd, bias, residual, partials, max_partial_floats, err_word, d_hi,
                         d_plane, s, two_cta_mode, act, col_partial);
}

}  // namespace bt
