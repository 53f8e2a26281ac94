// The verification step taken straight from the LM head: the logits z[r, v] = sum_h hidden[r, h] * W[v, h] of
// Algorithm 1's single target pass are produced by a tcgen05 GEMM whose epilogue reduces them to the per-row
// statistics of S1 (maximum, lowest arg-max, sum of exponentials) and picks out the draft tokens' logits, so
// the [rows, V] logit tensor never reaches HBM.
//
//   lmhead_stats_kernel     persistent, one CTA per SM, 320 threads:
//       warp 0      one thread issues the TMA loads (cp.async.bulk.tensor, 128-byte swizzle) of the k-blocks:
//                   64 columns of the hidden rows (a box of up to 128 rows and one of the rows beyond) and of the
//                   vocabulary tile's W rows, into a ring of as many shared-memory stages as fit (3 to 8)
//       warp 1      one thread issues the MMAs (tcgen05.mma, kind::f16, M = 128, N = tile width, K = 16, fp32
//                   accumulators in tensor memory: columns [0, N) for rows 0..127, [256, 256 + N) for rows
//                   128..255) and commits each stage back to the loader, each finished tile to the epilogue
//       warps 2..9  epilogue: warps 2..5 take the first row tile, warps 6..9 the second; thread i of the warp covering
//                   TMEM lanes 32q..32q+31 owns logit row 32q + i of its tile; it reads the row's accumulators 64
//                   columns at a time (two tcgen05.ld in flight) and folds them into a running (max, arg-max,
//                   reference exponent, sum) -- no exchange between threads, a row lives in one thread -- and
//                   keeps z[row, draft[row]] when that column comes by
//     A CTA owns a contiguous run of vocabulary tiles and ends with one partial per logit row.
//   lmhead_stats_pair_kernel  the same by clusters of two CTAs (tcgen05 cta_group::2, M = 256): each CTA holds half of
//                           the rows against a tile twice as wide and loads half of every W tile; see its own text.
//   lmhead_finalize_kernel  one block per batch row: folds the CTAs' partials in a fixed order, then S2..S5
//                           exactly as the streaming step does; the memory update follows as its own launch.
// Both GEMM kernels may be launched programmatically behind the kernels of the step before: they read only the step's
// inputs until their first store, ahead of which they wait for those kernels (griddepcontrol.wait).
//
// Every wait on an mbarrier is bounded (about two seconds of clock cycles): when one runs out, the CTA raises
// CSD_FLAG_INTERNAL (debug_site 30; 31 in the pair kernel), all its roles leave their loops, it waits for copies that may still be in
// flight, frees its tensor memory and returns.
#pragma once

#include <cuda.h>

#include "../../include/csd.h"
#include "csd_common.cuh"
#include "csd_ocm.cuh"

namespace csd {
namespace lmhead {

constexpr int kBlockK = 64;                 // bf16 elements of a k-block: one 128-byte swizzle row
constexpr int kMaxStages = 8;
constexpr int kMTile = 128;
constexpr int kRowsMax = 2 * kMTile;        // logit rows of a row group
constexpr int kNMax = 256;                  // widest vocabulary tile
constexpr int kThreads = 320;                // warp 0 loads, warp 1 issues MMAs, warps 2..5 / 6..9 reduce the first / second row tile
constexpr int kRowBytes = kBlockK * 2;      // one row of a k-block
constexpr int kBarrierBytes = 1024;
// A row tile's operand is read as 128 rows although only the rows that exist are loaded: the read runs on into
// whatever follows (the stage's W tile, the next stage, or this slack), which only feeds accumulator rows that
// nobody reads.
constexpr int kSlackBytes = kMTile * kRowBytes;
constexpr int kSmemLimit = 226 * 1024;      // of the 227 KiB a block may have (some is static)
constexpr int kTmemCols = 512;
constexpr long long kWaitCycles = 4000000000ll;

struct Params {
    int R, H, V, B, K;
    int n_tile;             // columns of a vocabulary tile: multiple of 16, at most kNMax
    int tiles_total;        // ceil(V / n_tile)
    int tiles_per_cta;
    int rows1;              // rows loaded for the first row tile of the LAST row group: 128, or the rows it has rounded up to 8
    int rows2;              // rows loaded for the second row tile of the LAST row group (0 if it has <= 128 rows), a multiple of 8
    int a_bytes;            // bytes of a hidden k-block in a stage (both row tiles), a multiple of 1 KiB
    int sub_bytes;          // a_bytes + the W tile's k-block, a multiple of 1 KiB
    int kblocks_per_stage;  // k-blocks loaded, consumed and released together (H is a multiple of 64 times this)
    int n_stages;
    const int *draft;       // [B, K]
    Partial *partials;      // [R, gridDim.x]
    float *zd;              // [B, K]  z[b, i, draft[b, i]] (written for valid draft ids only)
    OcmStatsDev *stats;
};

__device__ __forceinline__ unsigned int smem_u32(const void *p) { return static_cast<unsigned int>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(unsigned int bar, unsigned int count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned int bar, unsigned int bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned int bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned int bar, unsigned int parity)
{
    unsigned int ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok)
                 : "r"(bar), "r"(parity)
                 : "memory");
    return ok != 0u;
}
// Bounded wait.  False if the wait ran out or another role of the CTA has given up.
__device__ __forceinline__ bool mbar_wait(unsigned int bar, unsigned int parity, volatile int *give_up)
{
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (*give_up) return false;
        if (clock64() - t0 > kWaitCycles) {
            *give_up = 1;
            return false;
        }
    }
    return true;
}

__device__ __forceinline__ void tma_load_2d(unsigned int dst, const CUtensorMap *map, unsigned int bar, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
                 "l"(map), "r"(bar), "r"(x), "r"(y)
                 : "memory");
}

__device__ __forceinline__ void tmem_alloc(unsigned int smem_dst, unsigned int cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() { asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_dealloc(unsigned int taddr, unsigned int cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(unsigned int bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 operands, fp32 accumulators.
__device__ __forceinline__ void tc_mma_bf16(unsigned int d_tmem, unsigned long long a_desc, unsigned long long b_desc, unsigned int idesc,
                                            unsigned int accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
                 "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
                 : "memory");
}
// 32 consecutive accumulator columns of this thread's TMEM lane.  The load is asynchronous; load and wait are one
// statement so that nothing can read the registers in between.
__device__ __forceinline__ void tmem_ld32(unsigned int taddr, float (&x)[32])
{
    unsigned int r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int j = 0; j < 32; ++j) x[j] = __uint_as_float(r[j]);
}
// 64 consecutive columns: two loads in flight, one wait.
__device__ __forceinline__ void tmem_ld64(unsigned int taddr, float (&x)[32], float (&y)[32])
{
    unsigned int r[64];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%64];\n\t"
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%65];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
        : "r"(taddr), "r"(taddr + 32u)
        : "memory");
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        x[j] = __uint_as_float(r[j]);
        y[j] = __uint_as_float(r[32 + j]);
    }
}

// Shared-memory operand descriptor of a K-major bf16 tile stored as rows of 128 bytes with the 128-byte swizzle
// (what the TMA loads above produce): groups of 8 rows lie 1024 bytes apart, the tile starts on a 1 KiB boundary.
__device__ __forceinline__ unsigned long long operand_desc(unsigned int smem_addr)
{
    unsigned long long d = 0;
    d |= static_cast<unsigned long long>((smem_addr & 0x3FFFFu) >> 4);     // start address
    d |= 1ull << 16;                                                       // leading-dimension offset: unused for this layout
    d |= static_cast<unsigned long long>(1024 >> 4) << 32;                 // stride between 8-row groups
    d |= 1ull << 46;                                                       // descriptor version of this architecture
    d |= 2ull << 61;                                                       // 128-byte swizzle
    return d;
}

__device__ __forceinline__ unsigned int instr_desc(int n)
{
    // fp32 accumulators, bf16 A and B, both K-major, N = n, M = 128
    return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<unsigned int>(n >> 3) << 17) | (static_cast<unsigned int>(kMTile >> 4) << 24);
}

// Running reduction of one logit row inside one thread.
struct RowRun {
    float m, c;
    int idx;
    unsigned long long acc0, acc1;
};

__device__ __forceinline__ void row_init(RowRun &r)
{
    r.m = -INFINITY;
    r.c = kNoRef;
    r.idx = 0x7fffffff;
    r.acc0 = pack2(0.f, 0.f);
    r.acc1 = r.acc0;
}

// 32 logits of columns v0 .. v0 + 31 (ascending over a thread's life, so a strict improvement keeps the lowest index).
__device__ __forceinline__ void row_take(RowRun &r, const float (&x)[32], int v0)
{
    float cm = x[0];
#pragma unroll
    for (int j = 1; j < 32; ++j) cm = fmaxf(cm, x[j]);
    if (cm > r.m) {
        int at = 31;
#pragma unroll
        for (int j = 30; j >= 0; --j) at = (x[j] == cm) ? j : at;
        r.m = cm;
        r.idx = v0 + at;
        const float cn = rintf(cm * kLog2e);
        if (cn > r.c) {
            const float f = pow2_nonpos(r.c - cn);
            const unsigned long long f2 = pack2(f, f);
            r.acc0 = mul2(r.acc0, f2);
            r.acc1 = mul2(r.acc1, f2);
            r.c = cn;
        }
    }
    const unsigned long long l2e2 = pack2(kLog2e, kLog2e), negc2 = pack2(-r.c, -r.c);
#pragma unroll
    for (int j = 0; j < 32; j += 4) {
        accum_pair(x[j], x[j + 1], l2e2, negc2, r.acc0);
        accum_pair(x[j + 2], x[j + 3], l2e2, negc2, r.acc1);
    }
}

__global__ void __launch_bounds__(kThreads, 1)
lmhead_stats_kernel(const __grid_constant__ CUtensorMap map_hidden, const __grid_constant__ CUtensorMap map_hidden2,
                    const __grid_constant__ CUtensorMap map_weight, const Params p)
{
    extern __shared__ unsigned char smem_raw[];
    __shared__ unsigned int tmem_base_slot;
    __shared__ int give_up_flag;
    volatile int *give_up = &give_up_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const unsigned int raw = smem_u32(smem_raw);
    const unsigned int bars = (raw + 1023u) & ~1023u;
    const unsigned int stages = bars + kBarrierBytes;
    const int n_stages = p.n_stages;
    const int kps = p.kblocks_per_stage;                   // k-blocks that travel and are released together
    const int sub_bytes = p.sub_bytes, a_bytes = p.a_bytes, stage_bytes = kps * sub_bytes;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (kMaxStages + s); };
    const unsigned int tmem_full = bars + 8u * (2 * kMaxStages);
    const unsigned int tmem_empty = bars + 8u * (2 * kMaxStages + 1);

    // Logit rows are taken in groups of 256 (two row tiles), one group after the other: a group sees the whole
    // vocabulary range of this CTA before the next begins, so a row's running statistics live in one thread.
    const int n_groups = (p.R + kRowsMax - 1) / kRowsMax;
    const int k_steps = p.H / (kBlockK * kps);             // stage fills per tile
    const int tile0 = blockIdx.x * p.tiles_per_cta;
    int tile1 = tile0 + p.tiles_per_cta;
    if (tile1 > p.tiles_total) tile1 = p.tiles_total;
    const int my_tiles = tile1 > tile0 ? tile1 - tile0 : 0;
    auto rows_of = [&](int g) { return min(kRowsMax, p.R - g * kRowsMax); };

    if (threadIdx.x == 0) {
        give_up_flag = 0;
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        mbar_init(tmem_full, 1);
        mbar_init(tmem_empty, 8 * 32);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // the decision kernel behind this one may be brought in now; it waits for this grid before it reads anything
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (warp == 2) {
        tmem_alloc(smem_u32(&tmem_base_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned int tmem_base = tmem_base_slot;

    if (warp == 0) {
        // ---- loader ----
        if (lane == 0) {
            int it = 0;
            for (int g = 0; g < n_groups && !*give_up; ++g) {
                const int rows = rows_of(g);
                const bool last_group = g == n_groups - 1;
                // the second row tile: 128 rows in a full group, the rows that exist (rounded up to 8) in the last one
                const int rows2 = rows > kMTile ? (last_group ? p.rows2 : kMTile) : 0;
                // the first: 128 rows, or in a last group of fewer only those (map_hidden2's box is then this one)
                const int rows1 = last_group ? p.rows1 : kMTile;
                const unsigned int tx = static_cast<unsigned int>(kps * (rows1 + rows2 + p.n_tile) * kRowBytes);
                for (int t = tile0; t < tile1 && !*give_up; ++t) {
                    const int v0 = t * p.n_tile;
                    for (int ks = 0; ks < k_steps; ++ks, ++it) {
                        const int s = it % n_stages;
                        if (!mbar_wait(empty_bar(s), ((it / n_stages) & 1) ^ 1, give_up)) break;
                        mbar_expect_tx(full_bar(s), tx);
                        for (int sub = 0; sub < kps; ++sub) {
                            const unsigned int a = stages + s * stage_bytes + sub * sub_bytes, b = a + a_bytes;
                            const int x = (ks * kps + sub) * kBlockK;
                            tma_load_2d(a, rows1 == kMTile ? &map_hidden : &map_hidden2, full_bar(s), x, g * kRowsMax);
                            if (rows2 == kMTile)
                                tma_load_2d(a + kMTile * kRowBytes, &map_hidden, full_bar(s), x, g * kRowsMax + kMTile);
                            else if (rows2 > 0)
                                tma_load_2d(a + kMTile * kRowBytes, &map_hidden2, full_bar(s), x, g * kRowsMax + kMTile);
                            tma_load_2d(b, &map_weight, full_bar(s), x, v0);
                        }
                    }
                }
            }
            // every commit aimed at the "empty" barriers has landed before the CTA goes on towards its end
            for (int k = 0; k < n_stages && !*give_up; ++k, ++it) mbar_wait(empty_bar(it % n_stages), ((it / n_stages) & 1) ^ 1, give_up);
        }
    } else if (warp == 1) {
        // ---- MMA issuer ----
        if (lane == 0) {
            const unsigned int idesc = instr_desc(p.n_tile);
            int it = 0, tt = 0;
            bool ok = true;
            for (int g = 0; g < n_groups && ok && !*give_up; ++g) {
                const int n_mt = rows_of(g) > kMTile ? 2 : 1;
                for (int t = 0; t < my_tiles && ok && !*give_up; ++t, ++tt) {
                    if (!mbar_wait(tmem_empty, (tt & 1) ^ 1, give_up)) {      // the epilogue has drained the previous tile
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    for (int ks = 0; ks < k_steps; ++ks, ++it) {
                        const int s = it % n_stages;
                        if (!mbar_wait(full_bar(s), (it / n_stages) & 1, give_up)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        for (int sub = 0; sub < kps; ++sub) {
                            const unsigned int a = stages + s * stage_bytes + sub * sub_bytes, b = a + a_bytes;
                            const unsigned long long a0_desc = operand_desc(a), a1_desc = operand_desc(a + kMTile * kRowBytes);
                            const unsigned long long b_desc = operand_desc(b);
#pragma unroll
                            for (int k4 = 0; k4 < kBlockK / 16; ++k4) {
                                const unsigned int acc = (ks | sub | k4) != 0 ? 1u : 0u;
                                // 16 columns further along K: 32 bytes, 2 in the descriptor's units of 16 bytes
                                tc_mma_bf16(tmem_base, a0_desc + 2ull * k4, b_desc + 2ull * k4, idesc, acc);
                                if (n_mt == 2) tc_mma_bf16(tmem_base + kNMax, a1_desc + 2ull * k4, b_desc + 2ull * k4, idesc, acc);
                            }
                        }
                        tc_commit(empty_bar(s));          // the stage may be refilled once these MMAs have read it
                    }
                    if (ok) tc_commit(tmem_full);         // the tile's accumulators are complete
                }
            }
        }
    } else {
        // ---- epilogue: warp w covers TMEM lanes 32 (w % 4) .. + 31; warps 2..5 take the first row tile of a
        // group, warps 6..9 the second; a thread owns one logit row ----
        const int q = warp & 3;
        const int mt = warp >= 6 ? 1 : 0;
        const unsigned int lane_base = tmem_base + (static_cast<unsigned int>(32 * q) << 16) + (mt ? kNMax : 0);
        int tt = 0;
        bool ok = true;
        for (int g = 0; g < n_groups && ok; ++g) {
            const int row = g * kRowsMax + mt * kMTile + 32 * q + lane;
            const bool has = row < p.R;
            const bool warp_has = g * kRowsMax + mt * kMTile + 32 * q < p.R;      // the warp has any row in this group
            RowRun rr;
            row_init(rr);
            int d = -1;
            if (has) {
                const int b = row / (p.K + 1), i = row - b * (p.K + 1);
                if (i < p.K) d = __ldg(p.draft + b * p.K + i);
            }
            float zd = 0.f;
            bool got = false;
            for (int t = 0; t < my_tiles; ++t, ++tt) {
                if (!mbar_wait(tmem_full, tt & 1, give_up)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const int v0 = (tile0 + t) * p.n_tile;
                const int v_end = min(p.V, v0 + p.n_tile);          // columns beyond the tile or the vocabulary are masked
                if (warp_has) {
                    for (int c0 = 0; c0 < p.n_tile; c0 += 64) {
                        const int vc = v0 + c0;
                        if (vc >= v_end) break;
                        const bool second = c0 + 32 < p.n_tile && vc + 32 < v_end;
                        float x[32], y[32];
                        if (second)
                            tmem_ld64(lane_base + c0, x, y);
                        else
                            tmem_ld32(lane_base + c0, x);
                        auto take = [&](float (&v)[32], int vb) {
                            if (vb + 32 > v_end) {
#pragma unroll
                                for (int j = 0; j < 32; ++j) v[j] = (vb + j < v_end) ? v[j] : -INFINITY;
                            }
                            if (has) {
                                row_take(rr, v, vb);
                                if (static_cast<unsigned int>(d - vb) < 32u && d < v_end) {
#pragma unroll
                                    for (int j = 0; j < 32; ++j) zd = (d - vb == j) ? v[j] : zd;
                                    got = true;
                                }
                            }
                        };
                        take(x, vc);
                        if (second) take(y, vc + 32);
                    }
                }
                tc_fence_before();
                mbar_arrive(tmem_empty);
            }
            // the partials of the step before may still be being read: this grid may have started ahead of the end of the
            // kernels before it on the stream, and waits for them here, ahead of its first store
            asm volatile("griddepcontrol.wait;" ::: "memory");
            if (has) {
                float s0, s1, s2, s3;
                unpack2(rr.acc0, s0, s1);
                unpack2(rr.acc1, s2, s3);
                Partial out;
                out.m = rr.m;
                out.idx = rr.idx;
                out.c = rr.c;
                out.s = (s0 + s1) + (s2 + s3);
                st_partial_cg(p.partials + static_cast<size_t>(row) * gridDim.x + blockIdx.x, out);
                if (got) {
                    const int b = row / (p.K + 1), i = row - b * (p.K + 1);
                    __stcg(p.zd + b * p.K + i, zd);
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (*give_up) {
        // a wait ran out: say so, and let copies that may still be in flight land before the block's memory is released
        if (threadIdx.x == 0) index_check_failed(p.stats, 30u);
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) {
        }
        __syncthreads();
    }
    if (warp == 2) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ---- the same reduction by PAIRS of CTAs (thread-block clusters of two, tcgen05 cta_group::2) -------------------
//
// Two SMs work on one vocabulary tile: the pair's MMA has M = 256, each CTA holding HALF of a row group's rows (128
// each in a full group; the last group's rows are split evenly, rounded up to 8) in its shared memory and their
// accumulators in its tensor memory, and each CTA brings in only half of every W tile -- the pair's MMA reads both
// halves.  A CTA's tensor memory then holds its rows against 2 N <= 512 columns (two MMAs per k-step, accumulators at
// columns 0 and 256), twice the width a lone CTA can hold for 256 rows, so the hidden states, which are read again for
// every vocabulary tile, are spread over twice as many columns: a k-block costs an SM (rows / 2 + N) x 128 bytes of
// shared-memory traffic instead of (rows + N) x 128.
//   both CTAs   warp 0: TMA loads of the CTA's own operands (cp.async.bulk.tensor with cta_group::2: the bytes are
//               counted on CTA 0's "full" barrier); warps 2..9: epilogue on the CTA's own tensor memory (warps 2..5
//               columns [0, N) of the tile, warps 6..9 columns [N, 2N)), one arrival per warp on CTA 0's "accumulators
//               drained" barrier
//   CTA 0 only  warp 1: issues the pair's MMAs; its commits arrive on the "stage empty" and "accumulators full"
//               barriers of BOTH CTAs (tcgen05.commit with a CTA mask: barrier arrivals, no data is moved)
// Partials: one per (pair, column half) and row, slot 2 * pair + half.  Bounded waits as above (debug_site 31); the two
// CTAs meet at a cluster barrier before the first signal crosses and before the tensor memory is freed.
constexpr unsigned int kPeerMask = 0xFEFFFFFFu;       // a shared-memory address with this mask applied is CTA 0's copy of it

__device__ __forceinline__ unsigned int cluster_rank()
{
    unsigned int r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.aligned;\n\tbarrier.cluster.wait.aligned;" ::: "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(unsigned int dst, const CUtensorMap *map, unsigned int bar, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
                 "l"(map), "r"(bar & kPeerMask), "r"(x), "r"(y)
                 : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(unsigned int d_tmem, unsigned long long a_desc, unsigned long long b_desc, unsigned int idesc,
                                                 unsigned int accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
                 "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
                 : "memory");
}
// Arrives on the barrier at this shared-memory offset in both CTAs of the pair once the MMAs issued so far are complete.
__device__ __forceinline__ void tc_commit_pair(unsigned int bar)
{
    const unsigned short both = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar), "h"(both)
                 : "memory");
}
// One arrival on CTA 0's copy of a barrier, from either CTA.
__device__ __forceinline__ void mbar_arrive_cta0(unsigned int bar)
{
    asm volatile("{\n\t.reg .b32 remote;\n\tmapa.shared::cluster.u32 remote, %0, 0;\n\tmbarrier.arrive.release.cluster.shared::cluster.b64 _, [remote];\n\t}" ::"r"(bar)
                 : "memory");
}
__device__ __forceinline__ unsigned int instr_desc_pair(int n)
{
    // as instr_desc, M = 256 over the two CTAs
    return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<unsigned int>(n >> 3) << 17) | (static_cast<unsigned int>(256 >> 4) << 24);
}

// Params as for the lone-CTA kernel, read this way: n_tile = N, the columns of one MMA (a tile of the pair has 2 N);
// tiles_per_cta = tiles per pair; rows2 = rows per CTA in the last row group (a multiple of 8, at most 128; map_hidden2's
// box); a_bytes = a CTA's hidden k-block; sub_bytes = a stage: a_bytes + two half W sub-tiles of N / 2 rows each.
__global__ void __launch_bounds__(kThreads, 1)
lmhead_stats_pair_kernel(const __grid_constant__ CUtensorMap map_hidden, const __grid_constant__ CUtensorMap map_hidden2,
                         const __grid_constant__ CUtensorMap map_weight, const Params p)
{
    extern __shared__ unsigned char smem_raw[];
    __shared__ unsigned int tmem_base_slot;
    __shared__ int give_up_flag;
    volatile int *give_up = &give_up_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int rank = static_cast<int>(cluster_rank());      // 0 issues the MMAs
    const int pair = blockIdx.x >> 1;
    const unsigned int raw = smem_u32(smem_raw);
    const unsigned int bars = (raw + 1023u) & ~1023u;
    const unsigned int stages = bars + kBarrierBytes;
    const int n_stages = p.n_stages;
    const int a_bytes = p.a_bytes, stage_bytes = p.sub_bytes;
    const int half_bytes = (stage_bytes - a_bytes) / 2;      // this CTA's half of one W sub-tile
    const int N = p.n_tile;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (kMaxStages + s); };
    const unsigned int tmem_full = bars + 8u * (2 * kMaxStages);
    const unsigned int tmem_empty = bars + 8u * (2 * kMaxStages + 1);

    const int n_groups = (p.R + kRowsMax - 1) / kRowsMax;
    const int kblocks = p.H / kBlockK;
    const int tile0 = pair * p.tiles_per_cta;
    int tile1 = tile0 + p.tiles_per_cta;
    if (tile1 > p.tiles_total) tile1 = p.tiles_total;
    const int my_tiles = tile1 > tile0 ? tile1 - tile0 : 0;
    // rows a CTA holds of group g: CTA 0 rows [256 g, + half), CTA 1 rows [256 g + half, + half)
    auto half_of = [&](int g) { return g == n_groups - 1 ? p.rows2 : kMTile; };

    if (threadIdx.x == 0) {
        give_up_flag = 0;
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        mbar_init(tmem_full, 1);
        mbar_init(tmem_empty, 2 * 8);                        // one arrival per epilogue warp of both CTAs
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                      // both CTAs' barriers exist before a signal crosses
    tc_fence_after();
    const unsigned int tmem_base = tmem_base_slot;

    if (warp == 0) {
        // ---- loader (both CTAs) ----
        if (lane == 0) {
            int it = 0;
            bool ok = true;
            for (int g = 0; g < n_groups && ok && !*give_up; ++g) {
                const int half = half_of(g);
                const bool full_group = half == kMTile && g != n_groups - 1;
                const unsigned int tx_pair = static_cast<unsigned int>((2 * half + 2 * N) * kRowBytes);      // the bytes of both CTAs
                const int row0 = g * kRowsMax + rank * half;
                for (int t = tile0; t < tile1 && ok && !*give_up; ++t) {
                    const int v0 = t * 2 * N + rank * (N / 2);
                    for (int kb = 0; kb < kblocks; ++kb, ++it) {
                        const int s = it % n_stages;
                        if (!mbar_wait(empty_bar(s), ((it / n_stages) & 1) ^ 1, give_up)) {
                            ok = false;
                            break;
                        }
                        if (rank == 0) mbar_expect_tx(full_bar(s), tx_pair);
                        const unsigned int a = stages + s * stage_bytes, b0 = a + a_bytes, b1 = b0 + half_bytes;
                        const int x = kb * kBlockK;
                        tma_load_2d_pair(a, full_group ? &map_hidden : &map_hidden2, full_bar(s), x, row0);
                        tma_load_2d_pair(b0, &map_weight, full_bar(s), x, v0);           // W rows [v0, + N / 2) of the first N columns
                        tma_load_2d_pair(b1, &map_weight, full_bar(s), x, v0 + N);       // and of the second N
                    }
                }
            }
            // every commit aimed at this CTA's "empty" barriers has landed before the CTA goes on towards its end
            for (int k = 0; k < n_stages && ok; ++k, ++it) ok = mbar_wait(empty_bar(it % n_stages), ((it / n_stages) & 1) ^ 1, give_up);
        }
    } else if (warp == 1) {
        // ---- MMA issuer (CTA 0 of the pair) ----
        if (lane == 0 && rank == 0) {
            const unsigned int idesc = instr_desc_pair(N);
            int it = 0, tt = 0;
            bool ok = true;
            for (int g = 0; g < n_groups && ok && !*give_up; ++g) {
                for (int t = 0; t < my_tiles && ok && !*give_up; ++t, ++tt) {
                    if (!mbar_wait(tmem_empty, (tt & 1) ^ 1, give_up)) {      // both CTAs have drained the previous tile
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    for (int kb = 0; kb < kblocks; ++kb, ++it) {
                        const int s = it % n_stages;
                        if (!mbar_wait(full_bar(s), (it / n_stages) & 1, give_up)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after();
                        const unsigned int a = stages + s * stage_bytes, b0 = a + a_bytes, b1 = b0 + half_bytes;
                        const unsigned long long a_desc = operand_desc(a), b0_desc = operand_desc(b0), b1_desc = operand_desc(b1);
#pragma unroll
                        for (int k4 = 0; k4 < kBlockK / 16; ++k4) {
                            const unsigned int acc = (kb | k4) != 0 ? 1u : 0u;
                            tc_mma_bf16_pair(tmem_base, a_desc + 2ull * k4, b0_desc + 2ull * k4, idesc, acc);
                            tc_mma_bf16_pair(tmem_base + kNMax, a_desc + 2ull * k4, b1_desc + 2ull * k4, idesc, acc);
                        }
                        tc_commit_pair(empty_bar(s));
                    }
                    if (ok) tc_commit_pair(tmem_full);
                }
            }
        }
    } else {
        // ---- epilogue (both CTAs): warps 2..5 the tile's first N columns, warps 6..9 its second N; a thread owns one
        // logit row of its CTA for one column half ----
        const int q = warp & 3;
        const int chalf = warp >= 6 ? 1 : 0;
        const unsigned int lane_base = tmem_base + (static_cast<unsigned int>(32 * q) << 16) + (chalf ? kNMax : 0);
        int tt = 0;
        bool ok = true;
        for (int g = 0; g < n_groups && ok; ++g) {
            const int half = half_of(g);
            const int row = g * kRowsMax + rank * half + 32 * q + lane;
            const bool has = 32 * q + lane < half && row < p.R;
            const bool warp_has = 32 * q < half && g * kRowsMax + rank * half + 32 * q < p.R;
            RowRun rr;
            row_init(rr);
            int d = -1;
            if (has) {
                const int b = row / (p.K + 1), i = row - b * (p.K + 1);
                if (i < p.K) d = __ldg(p.draft + b * p.K + i);
            }
            float zd = 0.f;
            bool got = false;
            for (int t = 0; t < my_tiles; ++t, ++tt) {
                if (!mbar_wait(tmem_full, tt & 1, give_up)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const int v0 = (tile0 + t) * 2 * N + chalf * N;
                const int v_end = min(p.V, v0 + N);
                if (warp_has) {
                    for (int c0 = 0; c0 < N; c0 += 64) {
                        const int vc = v0 + c0;
                        if (vc >= v_end) break;
                        const bool second = c0 + 32 < N && vc + 32 < v_end;
                        float x[32], y[32];
                        if (second)
                            tmem_ld64(lane_base + c0, x, y);
                        else
                            tmem_ld32(lane_base + c0, x);
                        auto take = [&](float (&v)[32], int vb) {
                            if (vb + 32 > v_end) {
#pragma unroll
                                for (int j = 0; j < 32; ++j) v[j] = (vb + j < v_end) ? v[j] : -INFINITY;
                            }
                            if (has) {
                                row_take(rr, v, vb);
                                if (static_cast<unsigned int>(d - vb) < 32u && d < v_end) {
#pragma unroll
                                    for (int j = 0; j < 32; ++j) zd = (d - vb == j) ? v[j] : zd;
                                    got = true;
                                }
                            }
                        };
                        take(x, vc);
                        if (second) take(y, vc + 32);
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cta0(tmem_empty);
            }
            // the partials of the step before may still be being read: this grid may have started ahead of the end of the
            // kernels before it on the stream, and waits for them here, ahead of its first store
            asm volatile("griddepcontrol.wait;" ::: "memory");
            if (has) {
                float s0, s1, s2, s3;
                unpack2(rr.acc0, s0, s1);
                unpack2(rr.acc1, s2, s3);
                Partial out;
                out.m = rr.m;
                out.idx = rr.idx;
                out.c = rr.c;
                out.s = (s0 + s1) + (s2 + s3);
                st_partial_cg(p.partials + static_cast<size_t>(row) * gridDim.x + 2 * pair + chalf, out);
                if (got) {
                    const int b = row / (p.K + 1), i = row - b * (p.K + 1);
                    __stcg(p.zd + b * p.K + i, zd);
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (*give_up) {
        if (threadIdx.x == 0) index_check_failed(p.stats, 31u);
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000ll) {
        }
        __syncthreads();
    }
    cluster_sync_all();                                      // no signal is on its way to a CTA that has left; the pair frees together
    if (warp == 2) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// ---- S1 (last level) and S2..S5 per batch row, from the partials of the LM-head kernel ----------------
struct FinalizeParams {
    int B, K, V, n_parts;
    const Partial *partials;     // [B*(K+1), n_parts]
    const float *zd;             // [B, K]
    const int *draft;
    OcmView ocm;
    float log_tau;
    int *accept_len;
    int *next_token;
    unsigned char *rescued;
    int *rej_d;
    int *rej_t;
    csd_diag_t diag;
};

constexpr int kFinalizeWarps = 8;

// One block per batch row.  Its warps fold the partials of the row's K + 1 logit rows (a warp per logit row, all
// loads of a round in flight together: the fold costs a few memory latencies, not one per partial); warp 0 then takes
// the decisions.
__global__ void __launch_bounds__(32 * kFinalizeWarps) lmhead_finalize_kernel(const FinalizeParams p)
{
    __shared__ float sm_m[1][CSD_MAX_K + 1], sm_s[1][CSD_MAX_K + 1];
    __shared__ int sm_t[1][CSD_MAX_K + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int w = 0;
    const int b = blockIdx.x;
    // launched programmatically behind the GEMM kernel: let the memory's update kernel in, then wait for the GEMM
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int K = p.K, K1 = K + 1;
    // the draft tokens and their logits do not depend on the fold: requested first
    int d = -1;
    bool valid = false;
    float zd = __int_as_float(0x7fc00000);
    if (warp == 0 && lane < K) {
        d = __ldg(p.draft + (size_t)b * K + lane);
        valid = static_cast<unsigned int>(d) < static_cast<unsigned int>(p.V);
        if (valid) zd = __ldcg(p.zd + (size_t)b * K + lane);
    }
    for (int i = warp; i < K1; i += kFinalizeWarps) {
        const Partial *src = p.partials + (static_cast<size_t>(b) * K1 + i) * p.n_parts;
        Partial v = partial_identity();
        for (int k0 = lane; k0 < p.n_parts; k0 += 128) {      // lane k folds parts k, k + 32, ... in order, four loads at a time
            Partial x[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (k0 + 32 * j < p.n_parts) x[j] = ld_partial_cg(src + k0 + 32 * j);
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (k0 + 32 * j < p.n_parts) v = (k0 + 32 * j == lane) ? x[j] : combine(v, x[j]);
        }
        // fixed-shape butterfly: maximum and its lowest index, then the sums rescaled (exactly) to its reference
        float m = v.m;
        int idx = v.idx;
        for (int o = 1; o < 32; o <<= 1) {
            const float om = __shfl_xor_sync(kFull, m, o);
            const int oi = __shfl_xor_sync(kFull, idx, o);
            const bool take = (om > m) || (om == m && oi < idx);
            m = take ? om : m;
            idx = take ? oi : idx;
        }
        const float c = (m == -INFINITY) ? kNoRef : rintf(m * kLog2e);
        float s = v.s * pow2_nonpos(v.c - c);
        for (int o = 1; o < 32; o <<= 1) s += __shfl_xor_sync(kFull, s, o);
        if (lane == 0) {
            sm_m[w][i] = m;
            sm_s[w][i] = s * exp2f(fmaf(-m, kLog2e, c));      // sum exp(x - m)
            sm_t[w][i] = idx;
        }
    }
    __syncthreads();
    if (warp != 0) return;
    __syncwarp();
    for (int row = lane; row <= K; row += 32) {
        const size_t at = (size_t)b * K1 + row;
        const float s_m = sm_s[w][row];
        if (!(s_m == s_m) || s_m == INFINITY) atomicOr(&p.ocm.stats->flags, CSD_FLAG_NAN_LOGIT);
        if (p.diag.m) p.diag.m[at] = sm_m[w][row];
        if (p.diag.s) p.diag.s[at] = s_m;
        if (p.diag.lse) p.diag.lse[at] = sm_m[w][row] + logf(s_m);
        if (p.diag.t) p.diag.t[at] = sm_t[w][row];
    }
    bool match = false, ok = false;
    int t = -1;
    unsigned int cnt = 0;
    if (lane < K) {
        t = sm_t[w][lane];
        match = (d == t);
        if (valid) cnt = ocm_lookup(p.ocm, make_key(d, t));                        // S3
        const float m = sm_m[w][lane], s_m = sm_s[w][lane];
        const bool is_freq = cnt >= p.ocm.lambda;
        const bool is_safe = (static_cast<double>(zd) - static_cast<double>(m)) >= static_cast<double>(p.log_tau);   // S4, Eq. 3
        ok = match || (valid && is_freq && is_safe);
        const size_t pos = (size_t)b * K + lane;
        if (p.diag.zd) p.diag.zd[pos] = zd;
        if (p.diag.cnt) p.diag.cnt[pos] = cnt;
        if (p.diag.score) p.diag.score[pos] = expf(zd - m);
        if (p.diag.p_d) p.diag.p_d[pos] = expf(zd - m) / s_m;
        if (p.diag.p_t) p.diag.p_t[pos] = 1.0f / s_m;
    }
    const unsigned int kmask = (K == 32) ? kFull : ((1u << K) - 1u);
    const unsigned int fail = ~(__ballot_sync(kFull, ok) & kmask) & kmask;
    const int n_acc = fail ? (__ffs(fail) - 1) : K;                                    // S5
    const bool reached = lane <= n_acc && lane < K;
    const bool record = reached && !match && valid;
    if (lane < K) {
        const size_t pos = (size_t)b * K + lane;
        p.rescued[pos] = (lane < n_acc && !match) ? 1 : 0;
        p.rej_d[pos] = record ? d : -1;
        p.rej_t[pos] = record ? t : -1;
    }
    const unsigned int m_match = __ballot_sync(kFull, reached && match);
    const unsigned int m_resc = __ballot_sync(kFull, lane < n_acc && !match && lane < K);
    const unsigned int m_rec = __ballot_sync(kFull, record);
    const unsigned int m_bad = __ballot_sync(kFull, lane < K && !valid);
    if (lane == 0) {
        p.accept_len[b] = n_acc;
        p.next_token[b] = sm_t[w][n_acc];
        OcmStatsDev *st = p.ocm.stats;
        atomicAdd(&st->positions, static_cast<unsigned long long>(K));
        if (m_match) atomicAdd(&st->matches, static_cast<unsigned long long>(__popc(m_match)));
        if (m_resc) atomicAdd(&st->rescues, static_cast<unsigned long long>(__popc(m_resc)));
        if (m_rec) atomicAdd(&st->rejections, static_cast<unsigned long long>(__popc(m_rec)));
        if (m_bad) atomicOr(&st->flags, CSD_FLAG_BAD_DRAFT);
        if (b == 0) atomicAdd(&st->steps, 1ull);
    }
}

}  // namespace lmhead
}  // namespace csd
