// PTX wrappers shared by the tcgen05 kernels (GEMM and attention): mbarriers with bounded waits,
// TMA tiled loads, tcgen05 MMA / commit / TMEM load-store, shared-memory matrix descriptors and
// the tensor-map encoder handle.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"

namespace bt {
namespace tc {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
// The issuing roles (TMA producer, MMA issuer) run their control flow on the WHOLE warp so that
// addresses and descriptors stay warp-uniform (cheap to hand to the asynchronous units); only the
// instruction itself is predicated on `pred` (non-zero in exactly one lane).
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes, uint32_t pred = 1u) {
    asm volatile(
        "{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %2, 0;\n\t"
        "@q mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n\t}" ::"r"(bar), "r"(bytes), "r"(pred)
        : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: gives up after limit_ns nanoseconds of the global timer (one second unless the
// caller passes another limit).  Returns false after raising the error word.
constexpr unsigned long long kWaitLimitNs = 1000000000ull;
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int* err, int code,
                                          unsigned long long limit_ns = kWaitLimitNs) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = globaltimer_ns();
    for (;;) {
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (globaltimer_ns() - t0 > limit_ns) {
            atomicCAS(err, 0, code);  // the first wait that ran out is the one reported
            return false;
        }
    }
}

// The same wait with its polling loop out of line.  The attention kernels wait at dozens of sites and
// their code has to stay within the instruction cache (every CTA start fetches it again: 175 KB of
// inlined code cost the backward kernels 8 % of their time against 123 KB); a wait that did not
// succeed at once has the time for a call.  Roles whose live registers are at the limit keep the
// inline form (a call spills them).
static __device__ __noinline__ bool mbar_wait_poll(uint32_t bar, uint32_t parity, int* err, int code,
                                                   unsigned long long limit_ns) {
    const unsigned long long t0 = globaltimer_ns();
    for (;;) {
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (globaltimer_ns() - t0 > limit_ns) {
            atomicCAS(err, 0, code);  // the first wait that ran out is the one reported
            return false;
        }
    }
}
__device__ __forceinline__ bool mbar_wait_ool(uint32_t bar, uint32_t parity, int* err, int code,
                                              unsigned long long limit_ns = kWaitLimitNs) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_poll(bar, parity, err, code, limit_ns);
}
__device__ __forceinline__ bool mbar_wait_warp_ool(uint32_t bar, uint32_t parity, int* err, int code,
                                                   unsigned long long limit_ns = kWaitLimitNs) {
    const bool ok = mbar_wait_ool(bar, parity, err, code, limit_ns);
    return __all_sync(0xffffffffu, ok);
}

// The same wait made by a whole warp, with a warp-uniform result: the callers go on to issue
// .sync.aligned tensor-memory instructions, which every lane of the warp must reach together.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, int* err, int code,
                                               unsigned long long limit_ns = kWaitLimitNs) {
    const bool ok = mbar_wait(bar, parity, err, code, limit_ns);
    return __all_sync(0xffffffffu, ok);
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int c0, int c1,
                                            int c2, uint32_t pred = 1u) {
    asm volatile(
        "{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %6, 0;\n\t"
        "@q cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        "\n\t}" ::"r"(dst), "l"((unsigned long long)tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(pred)
        : "memory");
}

// Brings a tensor map (a __grid_constant__ kernel parameter) into the descriptor cache ahead of the
// first copy that uses it; issued by one thread while the CTA is still setting up.
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* tm) {
    asm volatile("prefetch.tensormap [%0];" ::"l"((unsigned long long)tm) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate, uint32_t pred = 1u) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "setp.ne.b32 q, %5, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(pred)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar, uint32_t pred = 1u) {
    asm volatile(
        "{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %1, 0;\n\t"
        "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(bar), "r"(pred)
        : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor (sm_100 format): start address, leading / stride byte offsets
// (all >> 4), descriptor version 1, swizzle mode in bits 61-63.
//   K-major, 128B swizzle          : mode 2, SBO = 1024 (8 rows x 128 B), LBO unused.
//   MN-major, 128B swizzle/32B atom: mode 1, SBO = 512 (4 k-rows x 128 B), LBO = distance between
//                                    32-element column groups.
__device__ __forceinline__ uint64_t make_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t mode) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFFu);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)mode << 61;
    return d;
}


// TF32 split on the integer pipe: adding half a TF32 ulp to the bit pattern and clearing the low
// 13 bits rounds the magnitude to the nearest TF32 value (ties away from zero) -- the result of
// cvt.rna.tf32.f32 for finite inputs -- without occupying the conversion unit the exponentials use.
__device__ __forceinline__ void split_tf32_int(float x, uint32_t& hi, uint32_t& lo) {
    hi = (__float_as_uint(x) + 0x1000u) & 0xFFFFE000u;
    lo = __float_as_uint(x - __uint_as_float(hi));
}

// A descriptor whose start address is advanced by compile-time byte offsets: the constant high
// word and the low word of the tile base are built once, each MMA then costs one integer add.
struct DescBase {
    uint32_t lo, hi;
    __device__ __forceinline__ uint64_t at(uint32_t byte_offset) const {
        return ((uint64_t)hi << 32) | (uint64_t)(lo + (byte_offset >> 4));
    }
};
__device__ __forceinline__ DescBase make_desc_base(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t mode) {
    DescBase d;
    d.lo = ((addr >> 4) & 0x3FFFu) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
    d.hi = ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (mode << 29);
    return d;
}

// A operand from tensor memory (row i of A in lane i, the 8 k-values of the step in 8 consecutive
// 32-bit columns), B from shared memory.
__device__ __forceinline__ void umma_tf32_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc,
                                             uint32_t accumulate, uint32_t pred = 1u) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "setp.ne.b32 q, %5, 0;\n\t"
        "@q tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(pred)
        : "memory");
}

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]),
          "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]),
          "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Instruction descriptor of tcgen05.mma.kind::tf32 with FP32 accumulation: D format F32 (bits
// 4-5 = 1), A and B format TF32 (bits 7-9, 10-12 = 2), operand major-ness (bit 15 / 16: 1 = the
// M / N extent is contiguous), N >> 3 in bits 17-22, M >> 4 in bits 24-28.
__host__ __device__ constexpr uint32_t make_idesc_tf32(int m, int n, bool a_mn_major, bool b_mn_major) {
    return (1u << 4) | (2u << 7) | (2u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
           ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// ---------------------------------------------------------------- row-owner results -> global memory
// In the attention kernels a thread owns a row (its tensor-memory lane).  Written straight out,
// one warp store would touch 32 rows x 16 bytes; instead the warp's 32 x 32 chunk goes through a
// shared-memory tile (144-byte pitch: conflict-free both ways) and leaves as full 128-byte row
// segments: lane -> rows (lane >> 3) + 4 i, columns 4 (lane & 7) .. + 3.
//   v        this lane's 32 columns of the chunk (lane = row inside the warp's 32 rows)
//   tile     the warp's own 32 x 144-byte shared-memory tile
//   nvalid   how many of the warp's 32 rows exist (rows >= nvalid are neither stored nor summed)
//   raw/hi/lo  destination of row 0, column 0 of the chunk (any may be null); row_stride in floats
//   sums     nullable: 32 floats receiving the column sums over the valid rows (fixed order)
constexpr uint32_t kRowTilePitch = 144u;
constexpr uint32_t kRowTileBytes = 32u * kRowTilePitch;
__device__ __forceinline__ void warp_rows_store(const float (&v)[32], float* tile, int lane, int nvalid, float* raw,
                                                float* hi, float* lo, long long row_stride, float* sums) {
    float4* wr = reinterpret_cast<float4*>(reinterpret_cast<uint8_t*>(tile) + lane * kRowTilePitch);
#pragma unroll
    for (int q = 0; q < 8; ++q) wr[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
    __syncwarp();
    const int sub = lane >> 3, cq = lane & 7;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = sub + 4 * i;
        if (r < nvalid) {
            const float4 x = *reinterpret_cast<const float4*>(reinterpret_cast<const uint8_t*>(tile) + r * kRowTilePitch + cq * 16);
            const long long off = (long long)r * row_stride + 4 * cq;
            if (raw) *reinterpret_cast<float4*>(raw + off) = x;
            if (hi) {
                float4 h, l;
                bt::split_tf32(x, h, l);
                *reinterpret_cast<float4*>(hi + off) = h;
                *reinterpret_cast<float4*>(lo + off) = l;
            }
            acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
        }
    }
    if (sums) {   // warp-uniform
        acc.x += __shfl_xor_sync(0xffffffffu, acc.x, 8);  acc.y += __shfl_xor_sync(0xffffffffu, acc.y, 8);
        acc.z += __shfl_xor_sync(0xffffffffu, acc.z, 8);  acc.w += __shfl_xor_sync(0xffffffffu, acc.w, 8);
        acc.x += __shfl_xor_sync(0xffffffffu, acc.x, 16); acc.y += __shfl_xor_sync(0xffffffffu, acc.y, 16);
        acc.z += __shfl_xor_sync(0xffffffffu, acc.z, 16); acc.w += __shfl_xor_sync(0xffffffffu, acc.w, 16);
        if (sub == 0) *reinterpret_cast<float4*>(sums + 4 * cq) = acc;
    }
    __syncwarp();   // the tile is rewritten by the next chunk
}

// ---------------------------------------------------------------- helpers of the attention kernels
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Byte offset of k-step ks (8 contraction values) in a K-major operand tile of `rows` rows held as
// k-blocks of [hi | lo][rows][128 B] (32 floats of the contraction index per block).
__device__ __forceinline__ constexpr uint32_t kmaj_off(int rows, int ks, bool lo) {
    return (uint32_t)(ks >> 2) * 2u * (uint32_t)rows * 128u + (lo ? (uint32_t)rows * 128u : 0u) + (uint32_t)(ks & 3) * 32u;
}
__device__ __forceinline__ DescBase kmaj_base(uint32_t tile) { return make_desc_base(tile, 16u, 1024u, 2u); }

// The warp's 32 rows x 64 floats (given as hi/lo planes; row r of the warp at src + r * row_stride)
// -> (hi + lo) * mul -> re-split -> hi/lo columns of tensor memory, lane = row.  The rows are read
// the way they lie in memory (8 lanes x 16 bytes = one 128-byte row segment, all loads of a chunk in
// flight together) and turned so that every lane ends up with its own row through the warp's
// shared-memory tile.  Rows >= nvalid are read as the last valid row (their results are never used).
__device__ __forceinline__ void rows_to_tmem(const float* src_hi, const float* src_lo, long long row_stride, int nvalid,
                                             float mul, uint32_t t_hi, uint32_t t_lo, float* tile, int lane) {
    const int sub = lane >> 3, cq = lane & 7;
#pragma unroll 1   // runs once per CTA: one copy of the body (the kernels' code has to fit the instruction cache)
    for (int half = 0; half < 2; ++half) {
        float4 a[8], b[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int r = max(0, min(sub + 4 * i, nvalid - 1));
            const long long off = (long long)r * row_stride + half * 32 + 4 * cq;
            a[i] = *reinterpret_cast<const float4*>(src_hi + off);
            b[i] = *reinterpret_cast<const float4*>(src_lo + off);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float4 x = make_float4((a[i].x + b[i].x) * mul, (a[i].y + b[i].y) * mul, (a[i].z + b[i].z) * mul,
                                         (a[i].w + b[i].w) * mul);
            *reinterpret_cast<float4*>(reinterpret_cast<uint8_t*>(tile) + (sub + 4 * i) * kRowTilePitch + cq * 16) = x;
        }
        __syncwarp();
        uint32_t h[32], l[32];
        const float4* rd = reinterpret_cast<const float4*>(reinterpret_cast<const uint8_t*>(tile) + lane * kRowTilePitch);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const float4 x = rd[q];
            const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float fh, fl;
                split_tf32(xs[e], fh, fl);
                h[4 * q + e] = __float_as_uint(fh);
                l[4 * q + e] = __float_as_uint(fl);
            }
        }
        tmem_st32(t_hi + half * 32, h);
        tmem_st32(t_lo + half * 32, l);
        __syncwarp();   // the tile is rewritten by the next half
    }
    tmem_st_wait();
}

// ---------------------------------------------------------------- CTA pairs (cta_group::2)
// A cluster of two CTAs on neighbouring SMs issues one MMA of M = 256: each CTA supplies its own
// 128 rows of A and HALF of the B tile from its own shared memory and holds its own 128 rows of
// the accumulator in its own tensor memory.  Only the even CTA (the leader) issues.
// Work item of a CTA in a (sequence x head, block) grid whose CTAs start in the order of their linear
// index (x fastest).  The heads are taken in groups of `head_group`: inside a group the heads run fastest,
// then the blocks, then the next group, so that the CTAs in flight at one time belong to few heads and
// share those heads' operand tiles through L2.  head_group <= 0 or >= gridDim.x: one group.
__device__ __forceinline__ void grouped_block(int head_group, int& bh, int& y) {
    const int nh = (int)gridDim.x, ny = (int)gridDim.y;
    const int G = (head_group > 0 && head_group < nh) ? head_group : nh;
    const int id = (int)blockIdx.y * nh + (int)blockIdx.x;
    const int per = G * ny, grp = id / per, rem = id - grp * per;
    const int first = grp * G, heads = min(G, nh - first);
    y = rem / heads;
    bh = first + (rem - y * heads);
}

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of `addr` (a shared::cta address of this CTA) in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Tiled load into THIS CTA's shared memory whose byte count is credited to a barrier of the pair's
// leader (a shared::cluster address).  No cluster-wide delivery of the data itself.
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* tm, uint32_t leader_bar, int c0,
                                                 int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"((unsigned long long)tm), "r"(leader_bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void umma2_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                           uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrives (once the MMAs issued so far have completed) on the barrier at the same shared-memory
// offset in every CTA of `cta_mask`.
__device__ __forceinline__ void umma2_commit(uint32_t bar, uint16_t cta_mask) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(cta_mask)
                 : "memory");
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
// Resolved once by gemm_tc_init(); nullptr when the driver does not provide it.
EncodeTiledFn tensor_map_encoder();
int sm_count();

}  // namespace tc
}  // namespace bt
