// The fused verification step: stream every logit row once (max / arg-max / sum-exp),
// then, per batch row, match test, OCM look-up, the gate of Eq. 3, the prefix scan of
// Algorithm 1's verification loop, and finally the memory update -- one launch.
//
// Work decomposition
//   * The R = B*(K+1) logit rows, each cut into 512-byte units, form one long unit
//     space that is split EVENLY and contiguously over the G blocks of a persistent
//     grid (block c owns units [c*T/G, (c+1)*T/G)); a block touches one or a few rows.
//   * Inside a block the span is cut into fixed chunks (4 to 32 KiB, never across
//     a row) that the block's warps pull from a shared-memory counter.  Shared-memory
//     atomics cost next to nothing, so the hand-out can be this fine, and it evens out
//     the large warp-to-warp differences in memory latency: a block is done when its
//     bytes are done, not when its unluckiest warp is.  The chunk geometry is fixed,
//     so which warp reduces a chunk has no effect on any result bit.
//   * A warp reduces a chunk on its own: a lane keeps 8 x 16 bytes in flight, carries a
//     running maximum, an integer reference exponent and four independent sum
//     accumulators; only the iteration in which the maximum last improved is
//     remembered, and the exact lowest arg-max index is recovered by re-reading that
//     one iteration (an L2 hit).  Chunk results go to a shared-memory table.
//   * The warp that delivers the last chunk of a row's part folds that part (fixed
//     order) while the others keep streaming; the warp that completes the block's last
//     fold publishes one partial per (block, row) to global memory: one fence and one
//     ticket per batch row touched, per BLOCK.  Everything up to here reads only the
//     logits and writes only this launch's scratch.
//   * Whichever block delivers a batch row's last part finalises it: the rows a block
//     completed are shared out over its warps, one warp per row.  The few partials per
//     row are folded by fixed-shape butterflies (maximum first, then the sums rescaled
//     to the row's reference: bit-reproducible), lanes 0..K-1 take the per-position
//     decisions, a ballot gives the accepted prefix.
//   * Memory update without a second probe: the look-up already found each recorded
//     pair's slot (absent pairs get an empty slot reserved with count 0, which no
//     look-up can tell from "absent"), and leaves it as a hint.  The warp finalising
//     the LAST batch row then only adds 1 to the hinted slots, so every look-up of the
//     step saw the step-start counts.  Near the key limit, where admission order
//     matters, that warp falls back to the canonical-order path.
//   * Within a launch nothing ever waits for another block: arrival counters only.
//
// Consecutive steps (programmatic dependent launch, opt-in)
//   * A launch may begin as soon as every block of the previous launch on the stream has
//     started.  The scratch exists kScratchRing times and launches take the copies in
//     turn, by a sequence number kept in the workspace itself (one word counts the blocks
//     of all launches; a block's count divided by the grid size is its launch's number,
//     and the next launch begins only after every block of this one has counted in).  Streaming, publication,
//     tickets and the per-row fold of step n therefore run while steps n-1, n-2, ... are
//     still finishing.
//   * What does depend on step n-1 is the memory (its update) and the output buffers.
//     The finalising warps wait for it just before their look-up: for the completion
//     count that the last warp of every launch publishes in the workspace (release store,
//     acquire polls) when the host vouches that step n-1 is the launch that will publish
//     it, else -- and whenever the bounded poll runs out -- for the previous grid to
//     retire (griddepcontrol.wait).  A copy of the scratch is reused only after the
//     launch that last used it has completed (same wait).
#pragma once

#include <cuda_bf16.h>

#include "../../include/csd.h"
#include "csd_common.cuh"
#include "csd_ocm.cuh"

namespace csd {

struct StepParams {
    const void *logits;
    int B, K, V;
    long long stride_b, stride_k;
    const int *draft;
    OcmView ocm;
    float log_tau;
    int do_update;
    int *accept_len;
    int *next_token;
    unsigned char *rescued;
    int *rej_d;
    int *rej_t;
    csd_diag_t diag;
    // kScratchRing copies of the scratch, used by consecutive launches in turn, so that a
    // launch can publish and fold while the launches before it are still finishing.  A copy:
    //   partials [R * slots_per_row]  one slot per (row, block touching it)       at 0
    //   slot hints [B * K]            slot of each recorded pair (see kHint*)     at hint_off
    //   batch-row tickets [B]                                                     at b_ticket_off
    //   global ticket [1]                                                         at g_ticket_off
    char *scratch;
    unsigned int copy_bytes, hint_off, b_ticket_off, g_ticket_off;
    unsigned long long *launch_seq;  // blocks counted in by all launches on this workspace since it was cleared
    unsigned int *completed;         // launches completed on this workspace
    int n_spans;             // G: blocks that own a span of the unit space
    int unit_elems;          // elements per 512-byte unit
    int units_per_row;       // U = ceil(V / unit_elems)
    int slots_per_row;       // S >= most blocks that can touch one row
    int chunk_units;         // units per chunk
    long long total_units;   // T = R * U
    int narrow;              // 1 if the span arithmetic fits 32 bits
    int stream_ordered;      // 1 for a plain launch: everything before it on the stream is complete when it starts
    int chain_by_flag;       // 1 if the host vouches that the previous step launch on the stream used this
                             // very workspace, memory and outputs: its completion word is then enough
    // ---- a launch that covers only some positions of some batch rows (the two phases of the early-exit step) ----
    // K_total = 0: an ordinary step (the fields below are unused).  Otherwise this launch verifies positions
    // pos0 .. pos0 + K - 1 of a step with K_total positions: logit rows pos0 .. pos0 + K, draft / output / diagnostic
    // arrays laid out for K_total; its batch rows are row_map[0 .. *n_rows) if row_map is set, else 0 .. B - 1.
    int K_total, pos0;
    const int *row_map;      // virtual batch row -> batch row of the step
    const int *n_rows;       // device word: how many virtual batch rows there are (at most B)
    int min_units;           // least 512-byte units per block when the grid is re-derived on the device
    int *alive_out;          // if set: the batch rows that accepted all K positions of this launch, ascending ...
    int *n_alive_out;        // ... and how many they are (written by the launch's last warp)
    int count_positions;     // what a finalised batch row adds to the statistics' position count
    int count_step;          // whether the launch counts as a step in the statistics
};

// What a launch works on: ordinary launches take it from the parameters, a launch over a row list from the device.
struct Extent {
    int B;                   // batch rows
    int G;                   // blocks that own a span
    long long T;             // units in all
};

// Where batch row b of the launch lives in the step's arrays.
struct RowPlace {
    long long br;            // batch row of the step
    size_t pos;              // index of its first position in [B, K_total] arrays
    size_t row;              // index of its first logit row in [B, K_total + 1] arrays
    int i0;                  // first logit row within the batch row
};

__device__ __forceinline__ RowPlace place_of(const StepParams &p, long long b)
{
    RowPlace r;
    if (p.K_total == 0) {
        r.br = b;
        r.pos = static_cast<size_t>(b) * p.K;
        r.row = static_cast<size_t>(b) * (p.K + 1);
        r.i0 = 0;
    } else {
        r.br = p.row_map ? __ldg(p.row_map + b) : b;
        r.pos = static_cast<size_t>(r.br) * p.K_total + p.pos0;
        r.row = static_cast<size_t>(r.br) * (p.K_total + 1) + p.pos0;
        r.i0 = p.pos0;
    }
    return r;
}

__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ unsigned int ld_acquire(const unsigned int *p)
{
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release(unsigned int *p, unsigned int v)
{
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void fence_acq_rel() { asm volatile("fence.acq_rel.gpu;" ::: "memory"); }
// Arrival counter: the add releases everything this thread has observed or written so far (and, through a
// preceding __syncwarp, what the other lanes of its warp wrote) and acquires what earlier arrivals released.
__device__ __forceinline__ unsigned int atom_add_acq_rel(unsigned int *p, unsigned int v)
{
    unsigned int old;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}

constexpr int kFlagPolls = 1 << 14;   // bounded: a few milliseconds, then the hardware wait takes over

// Named barriers (ids 1..15; id 0 is __syncthreads): `count` threads, whole warps, take part.
__device__ __forceinline__ void named_barrier_sync(int id, int count) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory"); }
__device__ __forceinline__ void named_barrier_arrive(int id, int count) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(count) : "memory"); }

constexpr unsigned int kScratchRing = 4;   // power of two

struct ScratchCopy {
    Partial *partials;
    int *slot_hint;
    unsigned int *b_ticket;
    unsigned int *g_ticket;
};

// The scratch copy that launch number `seq` on this workspace works in.
__device__ __forceinline__ ScratchCopy scratch_of(const StepParams &p, unsigned int seq)
{
    char *base = p.scratch + static_cast<size_t>(seq & (kScratchRing - 1u)) * p.copy_bytes;
    ScratchCopy c;
    c.partials = reinterpret_cast<Partial *>(base);
    c.slot_hint = reinterpret_cast<int *>(base + p.hint_off);
    c.b_ticket = reinterpret_cast<unsigned int *>(base + p.b_ticket_off);
    c.g_ticket = reinterpret_cast<unsigned int *>(base + p.g_ticket_off);
    return c;
}

constexpr int kHintNone = -1;          // nothing to record at this position
constexpr int kHintAbsent = -2;        // recorded pair not in the table and no slot reserved
constexpr int kHintCareful = 1 << 30;  // count close to saturation: add with the wrap check

// Wait until at least `need` launches have completed on this workspace (all of their
// writes to the memory, the outputs and the scratch are then visible).  The last warp of
// a launch publishes the count with a release store; waiting for the whole previous grid
// to retire (griddepcontrol.wait) costs several microseconds more per step, so when the
// host vouches that the previous step launch on the stream is the one that will publish
// the count (same workspace, memory and outputs), the count is polled instead.  That
// launch is resident by then (a dependent launch begins only after every block of its
// predecessor has started), so the poll ends; it is bounded all the same, and whenever
// it runs out, or the host could not vouch, the hardware wait decides.
__device__ __forceinline__ void wait_completed(const StepParams &p, unsigned int need)
{
    if (p.chain_by_flag) {
        for (int i = 0; i < kFlagPolls; ++i)
            if (static_cast<int>(ld_acquire(p.completed) - need) >= 0) return;
    }
    pdl_wait();
}

// ---- element access policies ---------------------------------------------------------

// fp32 logits, 16-byte vectors (4 elements).
struct LaneF32Vec {
    using elem = float;
    using unit = uint4;
    static constexpr int kPer = 4;
    static __device__ __forceinline__ unit load(const elem *base, int u) { return ld_stream16(base + (size_t)u * 4); }
    static __device__ __forceinline__ float load_elem(const elem *row, int idx) { return __ldg(row + idx); }
    static __device__ __forceinline__ unit neg_inf() { return make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u); }
    static __device__ __forceinline__ unit vmax(unit a, unit b)
    {
        return make_uint4(__float_as_uint(fmaxf(__uint_as_float(a.x), __uint_as_float(b.x))),
                          __float_as_uint(fmaxf(__uint_as_float(a.y), __uint_as_float(b.y))),
                          __float_as_uint(fmaxf(__uint_as_float(a.z), __uint_as_float(b.z))),
                          __float_as_uint(fmaxf(__uint_as_float(a.w), __uint_as_float(b.w))));
    }
    static __device__ __forceinline__ float hmax(unit a)
    {
        return fmaxf(fmaxf(__uint_as_float(a.x), __uint_as_float(a.y)), fmaxf(__uint_as_float(a.z), __uint_as_float(a.w)));
    }
    static __device__ __forceinline__ void accum(unit a, unsigned long long l2e2, unsigned long long negc2,
                                                 unsigned long long &acc)
    {
        accum_pair(__uint_as_float(a.x), __uint_as_float(a.y), l2e2, negc2, acc);
        accum_pair(__uint_as_float(a.z), __uint_as_float(a.w), l2e2, negc2, acc);
    }
    static __device__ __forceinline__ void unpack(unit a, float (&f)[4])
    {
        f[0] = __uint_as_float(a.x); f[1] = __uint_as_float(a.y); f[2] = __uint_as_float(a.z); f[3] = __uint_as_float(a.w);
    }
    static __device__ __forceinline__ int first_eq(unit a, float v)
    {
        if (__uint_as_float(a.x) == v) return 0;
        if (__uint_as_float(a.y) == v) return 1;
        if (__uint_as_float(a.z) == v) return 2;
        if (__uint_as_float(a.w) == v) return 3;
        return -1;
    }
};

// bf16 logits, 16-byte vectors (8 elements); the maximum is taken on packed pairs.
struct LaneBf16Vec {
    using elem = __nv_bfloat16;
    using unit = uint4;
    static constexpr int kPer = 8;
    static __device__ __forceinline__ unit load(const elem *base, int u) { return ld_stream16(base + (size_t)u * 8); }
    static __device__ __forceinline__ float load_elem(const elem *row, int idx)
    {
        const unsigned short h = __ldg(reinterpret_cast<const unsigned short *>(row) + idx);
        return __uint_as_float(static_cast<unsigned int>(h) << 16);
    }
    static __device__ __forceinline__ unit neg_inf() { return make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u); }
    static __device__ __forceinline__ unsigned int max2(unsigned int a, unsigned int b)
    {
        unsigned int r;
        asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
        return r;
    }
    static __device__ __forceinline__ unit vmax(unit a, unit b)
    {
        return make_uint4(max2(a.x, b.x), max2(a.y, b.y), max2(a.z, b.z), max2(a.w, b.w));
    }
    static __device__ __forceinline__ float lo(unsigned int w) { return __uint_as_float(w << 16); }
    static __device__ __forceinline__ float hi(unsigned int w) { return __uint_as_float(w & 0xffff0000u); }
    static __device__ __forceinline__ float hmax(unit a)
    {
        const unsigned int w = max2(max2(a.x, a.y), max2(a.z, a.w));
        return fmaxf(lo(w), hi(w));
    }
    static __device__ __forceinline__ void accum(unit a, unsigned long long l2e2, unsigned long long negc2,
                                                 unsigned long long &acc)
    {
        accum_pair(lo(a.x), hi(a.x), l2e2, negc2, acc);
        accum_pair(lo(a.y), hi(a.y), l2e2, negc2, acc);
        accum_pair(lo(a.z), hi(a.z), l2e2, negc2, acc);
        accum_pair(lo(a.w), hi(a.w), l2e2, negc2, acc);
    }
    static __device__ __forceinline__ void unpack(unit a, float (&f)[8])
    {
        f[0] = lo(a.x); f[1] = hi(a.x); f[2] = lo(a.y); f[3] = hi(a.y);
        f[4] = lo(a.z); f[5] = hi(a.z); f[6] = lo(a.w); f[7] = hi(a.w);
    }
    static __device__ __forceinline__ int first_eq(unit a, float v)
    {
        const unsigned int w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (lo(w[j]) == v) return 2 * j;
            if (hi(w[j]) == v) return 2 * j + 1;
        }
        return -1;
    }
};

// Element-wise fallbacks for layouts that are not 16-byte aligned.
struct LaneF32Scalar {
    using elem = float;
    using unit = float;
    static constexpr int kPer = 1;
    static __device__ __forceinline__ unit load(const elem *base, int u) { return __ldg(base + u); }
    static __device__ __forceinline__ float load_elem(const elem *row, int idx) { return __ldg(row + idx); }
    static __device__ __forceinline__ unit neg_inf() { return -INFINITY; }
    static __device__ __forceinline__ unit vmax(unit a, unit b) { return fmaxf(a, b); }
    static __device__ __forceinline__ float hmax(unit a) { return a; }
    static __device__ __forceinline__ void accum(unit a, unsigned long long l2e2, unsigned long long negc2,
                                                 unsigned long long &acc)
    {
        // one element: the second half of the pair adds 2^(-inf) = 0
        accum_pair(a, -INFINITY, l2e2, negc2, acc);
    }
    static __device__ __forceinline__ void unpack(unit a, float (&f)[1]) { f[0] = a; }
    static __device__ __forceinline__ int first_eq(unit a, float v) { return a == v ? 0 : -1; }
};

struct LaneBf16Scalar {
    using elem = __nv_bfloat16;
    using unit = float;
    static constexpr int kPer = 1;
    static __device__ __forceinline__ unit load(const elem *base, int u)
    {
        const unsigned short h = __ldg(reinterpret_cast<const unsigned short *>(base) + u);
        return __uint_as_float(static_cast<unsigned int>(h) << 16);
    }
    static __device__ __forceinline__ float load_elem(const elem *row, int idx) { return load(row, idx); }
    static __device__ __forceinline__ unit neg_inf() { return -INFINITY; }
    static __device__ __forceinline__ unit vmax(unit a, unit b) { return fmaxf(a, b); }
    static __device__ __forceinline__ float hmax(unit a) { return a; }
    static __device__ __forceinline__ void accum(unit a, unsigned long long l2e2, unsigned long long negc2,
                                                 unsigned long long &acc)
    {
        // one element: the second half of the pair adds 2^(-inf) = 0
        accum_pair(a, -INFINITY, l2e2, negc2, acc);
    }
    static __device__ __forceinline__ void unpack(unit a, float (&f)[1]) { f[0] = a; }
    static __device__ __forceinline__ int first_eq(unit a, float v) { return a == v ? 0 : -1; }
};

// ---- S1: one warp reduces one tile ---------------------------------------------------

// `l2e` = log2(e) / T: the sums are of 2^(x * l2e - c) = exp(x / T) up to the reference.
template <typename L>
__device__ __forceinline__ Partial warp_tile(const typename L::elem *row, int e0, int e1, int lane, const float l2e = kLog2e)
{
    using U = typename L::unit;
    const typename L::elem *base = row + e0;
    const int nunits = (e1 - e0) / L::kPer;
    constexpr int kPerIter = 32 * kUnroll;
    const int nfull = nunits / kPerIter;

    float m_thr = -INFINITY;   // running maximum of this lane
    float c_thr = kNoRef;      // integer reference exponent of the accumulators
    int it_thr = -1;           // iteration of the last strict improvement
    // four sums as two packed pairs: acc0 = (s0, s1), acc1 = (s2, s3)
    unsigned long long acc0 = pack2(0.f, 0.f), acc1 = acc0;
    const unsigned long long l2e2 = pack2(l2e, l2e);
    U v[kUnroll];

    auto consume = [&](const U (&v)[kUnroll], int it) {
        U mx = L::vmax(L::vmax(L::vmax(v[0], v[1]), L::vmax(v[2], v[3])),
                       L::vmax(L::vmax(v[4], v[5]), L::vmax(v[6], v[7])));
        const float bmax = L::hmax(mx);
        if (bmax > m_thr) {
            m_thr = bmax;
            it_thr = it;
            const float cn = rintf(bmax * l2e);
            if (cn > c_thr) {
                const float f = pow2_nonpos(c_thr - cn);
                const unsigned long long f2 = pack2(f, f);
                acc0 = mul2(acc0, f2);
                acc1 = mul2(acc1, f2);
                c_thr = cn;
            }
        }
        const unsigned long long negc2 = pack2(-c_thr, -c_thr);
#pragma unroll
        for (int k = 0; k < kUnroll; k += 2) {
            L::accum(v[k], l2e2, negc2, acc0);
            L::accum(v[k + 1], l2e2, negc2, acc1);
        }
    };

    // full iterations: one pointer, constant offsets, no bounds checks
    const typename L::elem *lp = base + (size_t)lane * L::kPer;
    for (int it = 0; it < nfull; ++it) {
#pragma unroll
        for (int k = 0; k < kUnroll; ++k) v[k] = L::load(lp, k * 32);
        lp += (size_t)kPerIter * L::kPer;
        consume(v, it);
    }
    if (nfull * kPerIter < nunits) {
#pragma unroll
        for (int k = 0; k < kUnroll; ++k) {
            const int u = (nfull * kUnroll + k) * 32 + lane;
            v[k] = u < nunits ? L::load(base, u) : L::neg_inf();
        }
        consume(v, nfull);
    }
    float s0, s1, s2, s3;
    unpack2(acc0, s0, s1);
    unpack2(acc1, s2, s3);

    // warp maximum, then everything is rescaled to the warp's reference exponent
    float wmax = m_thr;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) wmax = fmaxf(wmax, __shfl_xor_sync(kFull, wmax, o));
    const float cw = (wmax == -INFINITY) ? kNoRef : rintf(wmax * l2e);
    float s = ((s0 + s1) + (s2 + s3)) * pow2_nonpos(c_thr - cw);
    int cand = 0x7fffffff;
    if (it_thr >= 0 && m_thr == wmax) {
        // the lane's first element equal to the maximum lies in iteration it_thr
        for (int k = 0; k < kUnroll; ++k) {
            const int u = (it_thr * kUnroll + k) * 32 + lane;
            if (u >= nunits) break;
            const int j = L::first_eq(L::load(base, u), wmax);
            if (j >= 0) {
                cand = e0 + u * L::kPer + j;
                break;
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        s += __shfl_xor_sync(kFull, s, o);
        cand = min(cand, __shfl_xor_sync(kFull, cand, o));
    }
    Partial p;
    p.m = wmax;
    p.idx = (cand == 0x7fffffff) ? e0 : cand;   // a run without finite values reports its first element
    p.c = cw;
    p.s = s;
    return p;
}

// ---- the even split of the unit space over blocks -----------------------------------------

__device__ __forceinline__ long long span_begin(const StepParams &p, const Extent &e, int c)
{
    if (p.narrow)   // (T + 1) * (G + 1) < 2^32: 32-bit division is several times cheaper
        return static_cast<unsigned int>(c) * static_cast<unsigned int>(e.T) / static_cast<unsigned int>(e.G);
    return static_cast<long long>(c) * e.T / e.G;
}

// The block whose span holds global unit g: the largest c with span_begin(c) <= g.
__device__ __forceinline__ int owner_of(const StepParams &p, const Extent &e, long long g)
{
    if (p.narrow)
        return static_cast<int>(((static_cast<unsigned int>(g) + 1u) * static_cast<unsigned int>(e.G) - 1u) /
                                static_cast<unsigned int>(e.T));
    return static_cast<int>(((g + 1) * e.G - 1) / e.T);
}

constexpr int kFinalizeWarps = 8;  // warps of a block that share its batch rows to finalise
constexpr int kMaxSegs = 32;       // row parts a block handles between two block barriers
constexpr int kMaxChunks = 1024;   // chunk results held in shared memory at a time

struct BlockState {
    unsigned int seq;                   // this launch's sequence number on the workspace
    unsigned int next_chunk;            // hand-out counter
    unsigned int segs_folded;           // row parts folded so far
    unsigned int seg_done[kMaxSegs];    // chunks delivered per row part
    Partial seg_result[kMaxSegs];
    Partial chunk_part[kMaxChunks];
    int n_todo;                         // batch rows this block has to finalise in this window ...
    int todo_b[kMaxSegs];               // ... and which
    // Draft tokens of the first two batch rows the block touches, fetched when the block starts (their logits
    // are requested into L2 at the same time): a row this block then finalises finds them here.
    int pre_b[2];
    int pre_d[2][CSD_MAX_K];
};

// ---- S2..S5 for one batch row, by one warp ------------------------------------------

struct RowScratch {
    float m[CSD_MAX_K + 1];
    float s[CSD_MAX_K + 1];
    int t[CSD_MAX_K + 1];
    int parts[CSD_MAX_K + 1];   // number of blocks touching the row
};

enum UpdateRegime { kRegimeRoom = 0, kRegimeFull = 1, kRegimeTransition = 2, kRegimeShared = 3 };

// Which of the three update regimes this step is in.  n_keys_start is written when the
// previous update finished, so every warp of the launch computes the same answer.
__device__ __forceinline__ int update_regime(const StepParams &p)
{
    const unsigned long long nk = __ldcg(&p.ocm.stats->n_keys_start);
    const unsigned long long n = static_cast<unsigned long long>(p.B) * p.K;
    if (nk + n <= p.ocm.key_limit) return kRegimeRoom;
    if (nk >= p.ocm.key_limit) return kRegimeFull;
    return kRegimeTransition;
}

// Butterfly fold of one value per lane inside aligned groups of `width` lanes: maximum and
// its lowest index first, then the sums rescaled (exactly) to the group's reference.
// Every lane of a group ends with the group's total.
__device__ __forceinline__ Partial butterfly_fold(Partial v, int width, const float l2e = kLog2e)
{
    float m = v.m;
    int idx = v.idx;
    for (int o = 1; o < width; o <<= 1) {
        const float om = __shfl_xor_sync(kFull, m, o);
        const int oi = __shfl_xor_sync(kFull, idx, o);
        const bool take = (om > m) || (om == m && oi < idx);
        m = take ? om : m;
        idx = take ? oi : idx;
    }
    const float c = (m == -INFINITY) ? kNoRef : rintf(m * l2e);
    float s = v.s * pow2_nonpos(v.c - c);
    for (int o = 1; o < width; o <<= 1) s += __shfl_xor_sync(kFull, s, o);
    Partial r;
    r.m = m;
    r.idx = idx;
    r.c = c;
    r.s = s;
    return r;
}

// Fold the per-block partials of the K+1 logit rows of batch row b (S1, last level).  The
// lanes are arranged as (32 / width) rows x width slots, width = the power of two >= the
// slots per row (at most 32; more slots are pre-folded in lane order).
__device__ __forceinline__ void fold_rows(const StepParams &p, const Extent &e, const ScratchCopy &sc, int b, int lane, RowScratch &rs)
{
    const int K1 = p.K + 1, S = p.slots_per_row;
    int width = 1;
    while (width < S && width < 32) width <<= 1;
    const int rows_per_pass = 32 / width;
    const int sub = lane / width;          // which row of the pass
    const int k0 = lane - sub * width;     // first slot this lane folds
    const size_t row0 = (size_t)b * K1;
    const Partial *part = sc.partials + row0 * S;

    for (int r = lane; r < K1; r += 32) {
        const long long u0 = static_cast<long long>(row0 + r) * p.units_per_row;
        rs.parts[r] = owner_of(p, e, u0 + p.units_per_row - 1) - owner_of(p, e, u0) + 1;
    }
    __syncwarp();

    for (int r0 = 0; r0 < K1; r0 += rows_per_pass * 4) {
        Partial v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int row = r0 + q * rows_per_pass + sub;
            v[q] = partial_identity();
            if (row < K1) {
                int np = rs.parts[row];
                if (!CSD_INDEX_OK(np >= 1 && np <= S, p.ocm.stats, 3u)) np = 0;
                for (int k = k0; k < np; k += width) {       // one trip unless a row has > 32 parts
                    const Partial x = ld_partial_cg(part + (size_t)row * S + k);
                    v[q] = (k == k0) ? x : combine(v[q], x);
                }
            }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int row = r0 + q * rows_per_pass + sub;
            if (r0 + q * rows_per_pass >= K1) break;
            const Partial t = butterfly_fold(v[q], width);
            if (k0 == 0 && row < K1) {
                // sum exp(x - m) = s * 2^(c - m log2 e)
                const float s_m = t.s * exp2f(fmaf(-t.m, kLog2e, t.c));
                rs.m[row] = t.m;
                rs.s[row] = s_m;
                rs.t[row] = t.idx;
            }
        }
    }
    __syncwarp();
}

// Logit row i (within the launch) of batch row b (of the launch).
template <typename L>
__device__ __forceinline__ const typename L::elem *logit_row(const StepParams &p, long long b, int i)
{
    const RowPlace at = place_of(p, b);
    return reinterpret_cast<const typename L::elem *>(p.logits) + at.br * p.stride_b + static_cast<long long>(at.i0 + i) * p.stride_k;
}

__device__ __forceinline__ void prefetch_l2(const void *ptr) { asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr)); }

template <typename L>
__device__ int finalize_batch_row(const StepParams &p, const Extent &e, unsigned int seq, int b, int lane, RowScratch &rs,
                                  const BlockState &bs, int &hint_reg)
{
    hint_reg = kHintNone;
    const int K = p.K;
    const RowPlace at_b = place_of(p, b);

    // S2 (first half): the draft tokens and their logits do not depend on the reduction: the tokens were
    // fetched when the block started (else they are loaded now), the logits' loads are issued before the
    // partials are folded.
    int d = -1;
    float zd = __int_as_float(0x7fc00000);
    const int pre = bs.pre_b[0] == b ? 0 : (bs.pre_b[1] == b ? 1 : -1);
    if (lane < K) d = pre >= 0 ? bs.pre_d[pre][lane] : __ldg(p.draft + at_b.pos + lane);
    const bool valid = lane < K && static_cast<unsigned int>(d) < static_cast<unsigned int>(p.V);
    if (valid) zd = L::load_elem(logit_row<L>(p, b, lane), d);
    const ScratchCopy sc = scratch_of(p, seq);
    fold_rows(p, e, sc, b, lane, rs);

    // Everything above read only this launch's inputs and its own copy of the scratch.
    // From here on the previous launch must be complete: the memory, its statistics and
    // the output buffers come into play.
    wait_completed(p, seq);
    // S3.  The update regime (one load, used only after the look-up) is requested first so
    // that it travels together with the probe.
    const int regime = p.do_update ? (p.ocm.shared ? kRegimeShared : update_regime(p)) : kRegimeFull;
    bool match = false, ok = false;
    int t = -1;
    unsigned int cnt = 0;
    long long slot = -1, empty_slot = -1;
    if (lane < K) {
        t = rs.t[lane];
        match = (d == t);
        if (valid) cnt = ocm_lookup(p.ocm, make_key(d, t), &slot, &empty_slot);
    }
    for (int row = lane; row <= K; row += 32) {
        const size_t at = at_b.row + row;
        const float s_m = rs.s[row];
        if (!(s_m == s_m) || s_m == INFINITY) atomicOr(&p.ocm.stats->flags, CSD_FLAG_NAN_LOGIT);
        if (p.diag.m) p.diag.m[at] = rs.m[row];
        if (p.diag.s) p.diag.s[at] = s_m;
        if (p.diag.lse) p.diag.lse[at] = rs.m[row] + logf(s_m);
        if (p.diag.t) p.diag.t[at] = rs.t[row];
    }

    // S2 (second half), S4 per position; S5 across the warp.
    if (lane < K) {
        const float m = rs.m[lane];
        const float s_m = rs.s[lane];
        const bool is_freq = cnt >= p.ocm.lambda;
        const bool is_safe = (static_cast<double>(zd) - static_cast<double>(m)) >= static_cast<double>(p.log_tau);  // S4, Eq. 3
        ok = match || (valid && is_freq && is_safe);
        const size_t pos = at_b.pos + lane;
        if (p.diag.zd) p.diag.zd[pos] = zd;
        if (p.diag.cnt) p.diag.cnt[pos] = cnt;
        if (p.diag.score || p.diag.p_d) {
            const float score = expf(zd - m);
            if (p.diag.score) p.diag.score[pos] = score;
            if (p.diag.p_d) p.diag.p_d[pos] = score / s_m;
        }
        if (p.diag.p_t) p.diag.p_t[pos] = 1.0f / s_m;
    }
    const unsigned int kmask = (K == 32) ? kFull : ((1u << K) - 1u);
    const unsigned int okmask = __ballot_sync(kFull, ok) & kmask;
    const unsigned int fail = ~okmask & kmask;
    const int n_acc = fail ? (__ffs(fail) - 1) : K;                                   // S5
    const bool reached = lane <= n_acc && lane < K;
    const bool record = reached && !match && valid;
    if (lane < K) {
        const size_t pos = at_b.pos + lane;
        p.rescued[pos] = (lane < n_acc && !match) ? 1 : 0;
        p.rej_d[pos] = record ? d : -1;
        p.rej_t[pos] = record ? t : -1;
        if (p.do_update) {
            // S6, first half: leave the slot of every recorded pair for the final adder
            int hint = kHintNone;
            if (record) {
                if (slot < 0 && regime == kRegimeRoom) slot = ocm_reserve(p.ocm, make_key(d, t), empty_slot);
                if (slot < 0 && regime == kRegimeShared) slot = ocm_reserve_shared(p.ocm, make_key(d, t), empty_slot);
                hint = slot < 0 ? kHintAbsent : static_cast<int>(slot);
                const unsigned int room = 0xffffffffu - static_cast<unsigned int>(p.B * p.K);
                if (slot >= 0 && cnt > room) hint |= kHintCareful;
            }
            __stcg(sc.slot_hint + (size_t)b * K + lane, hint);
            hint_reg = hint;
        }
    } else if (p.K_total != 0 && p.pos0 == 0 && lane < p.K_total) {
        // first phase of a step in two phases: the positions it does not cover start out as "not reached"
        const size_t pos = at_b.pos + lane;
        p.rescued[pos] = 0;
        p.rej_d[pos] = -1;
        p.rej_t[pos] = -1;
    }
    const unsigned int m_match = __ballot_sync(kFull, reached && match);
    const unsigned int m_resc = __ballot_sync(kFull, lane < n_acc && !match && lane < K);
    const unsigned int m_rec = __ballot_sync(kFull, record);
    const unsigned int m_bad = __ballot_sync(kFull, lane < K && !valid);
    if (lane == 0) {
        p.accept_len[at_b.br] = at_b.i0 + n_acc;
        p.next_token[at_b.br] = rs.t[n_acc];
        OcmStatsDev *st = p.ocm.stats;
        const int counted = p.K_total != 0 ? p.count_positions : K;
        if (counted) atomicAdd(&st->positions, static_cast<unsigned long long>(counted));
        if (m_match) atomicAdd(&st->matches, static_cast<unsigned long long>(__popc(m_match)));
        if (m_resc) atomicAdd(&st->rescues, static_cast<unsigned long long>(__popc(m_resc)));
        if (m_rec) atomicAdd(&st->rejections, static_cast<unsigned long long>(__popc(m_rec)));
        if (m_bad) atomicOr(&st->flags, CSD_FLAG_BAD_DRAFT);
    }
    __syncwarp();
    return regime;
}

// One recorded pair's add, from the slot its look-up left (every lane of the warp calls this).
__device__ __forceinline__ void apply_hint(const StepParams &p, int hint)
{
    if (hint >= 0) {
        const unsigned long long s = static_cast<unsigned long long>(hint & ~kHintCareful);
        if (CSD_INDEX_OK(s <= p.ocm.mask, p.ocm.stats, 4u)) {
            if (hint & kHintCareful)
                ocm_add(p.ocm, s, 1u);
            else
                atomicAdd(&p.ocm.slots[s].count, 1u);
        }
    }
    const unsigned int dropped = __popc(__ballot_sync(kFull, hint == kHintAbsent));
    if ((threadIdx.x & 31) == 0 && dropped) atomicAdd(&p.ocm.stats->n_dropped, static_cast<unsigned long long>(dropped));
    __syncwarp();
}

// S6, second half, by the warp that finalised the last batch row: every look-up of the
// step is done, so the counts may change now.
__device__ void apply_step_update(const StepParams &p, const ScratchCopy &sc, int lane, CanonScratch &canon, int regime)
{
    const int n = p.B * p.K;
    if (regime == kRegimeTransition) {
        ocm_update_group<false>(p.ocm, p.rej_d, p.rej_t, nullptr, n, canon, lane, 32);
        return;
    }
    unsigned int dropped = 0;
    for (int j0 = 0; j0 < n; j0 += 32 * 16) {
        int h[16];
#pragma unroll
        for (int q = 0; q < 16; ++q) {
            const int j = j0 + q * 32 + lane;
            h[q] = j < n ? __ldcg(sc.slot_hint + j) : kHintNone;
        }
#pragma unroll
        for (int q = 0; q < 16; ++q) {
            if (h[q] >= 0) {
                const unsigned long long s = static_cast<unsigned long long>(h[q] & ~kHintCareful);
                if (!CSD_INDEX_OK(s <= p.ocm.mask, p.ocm.stats, 4u)) continue;
                if (h[q] & kHintCareful)
                    ocm_add(p.ocm, s, 1u);
                else
                    atomicAdd(&p.ocm.slots[s].count, 1u);
            } else if (h[q] == kHintAbsent) {
                ++dropped;
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) dropped += __shfl_xor_sync(kFull, dropped, o);
    if (lane == 0 && dropped) atomicAdd(&p.ocm.stats->n_dropped, static_cast<unsigned long long>(dropped));
    __syncwarp();
}

// Publication of a block's row parts: partials to global memory, one ticket per batch row
// touched.  Executed by ONE warp of the block.  The batch rows whose last part this block
// delivered are left in bs.todo_b for the block's warps to finalise.
//   nseg row parts, rows first_row .. first_row + nseg - 1, results in bs.seg_result;
//   next_b: batch row of the next row this block will still publish, or -1.
__device__ void publish_parts(const StepParams &p, const Extent &e, BlockState &bs, int first_row, int nseg, int next_b, int lane)
{
    const int K1 = p.K + 1;
    const int U = p.units_per_row;
    const unsigned int seq = bs.seq;
    const ScratchCopy sc = scratch_of(p, seq);
    // This copy was last used by launch seq - kScratchRing.  If that launch is known to be
    // complete the scratch can be written right away; otherwise wait for it (launches
    // complete in order).
    const unsigned int need = seq - (kScratchRing - 1u);
    if (!p.stream_ordered && static_cast<int>(ld_acquire(p.completed) - need) < 0) wait_completed(p, need);
    int my_b = -1;
    if (lane < nseg) {
        const int row = first_row + lane;
        const int slot = static_cast<int>(blockIdx.x) - owner_of(p, e, static_cast<long long>(row) * U);
        // the host sized slots_per_row from the same split: a slot beyond it would be a bug, and is reported
        if (CSD_CHECKED(slot >= 0 && slot < p.slots_per_row && row < e.B * K1, p.ocm.stats, 1u))
            st_partial_cg(sc.partials + (size_t)row * p.slots_per_row + slot, bs.seg_result[lane]);
        my_b = row / K1;
    }
    __syncwarp();         // every lane's partial before any lane's ticket (the ticket's add releases them)
    const int below_b = __shfl_down_sync(kFull, my_b, 1);
    bool completes = false;
    if (lane < nseg) {
        // the lane holding this block's last part of a batch row takes that row's ticket
        const bool closes = (lane == nseg - 1) ? (my_b != next_b) : (below_b != my_b);
        if (closes) {
            const long long u0 = static_cast<long long>(my_b) * K1 * U;
            const unsigned int expected = owner_of(p, e, u0 + static_cast<long long>(K1) * U - 1) - owner_of(p, e, u0) + 1;
            // the last arrival has acquired the other blocks' partials of the row; this block's warps read
            // them after the block barrier that follows
            completes = atom_add_acq_rel(sc.b_ticket + my_b, 1u) == expected - 1;
        }
    }
    const unsigned int todo = __ballot_sync(kFull, completes);
    if (completes && CSD_INDEX_OK(my_b >= 0 && my_b < e.B, p.ocm.stats, 2u)) bs.todo_b[__popc(todo & ((1u << lane) - 1u))] = my_b;
    if (lane == 0) bs.n_todo = __popc(todo);
}

// S2..S5 of batch row b by one warp, and, if that was the launch's last row, S6.
template <typename L>
__device__ void finalize_and_update(const StepParams &p, const Extent &e, unsigned int seq, int b, int lane, RowScratch &rs,
                                    CanonScratch &canon, const BlockState &bs)
{
    const ScratchCopy sc = scratch_of(p, seq);
    int own_hint;
    const int regime = finalize_batch_row<L>(p, e, seq, b, lane, rs, bs, own_hint);   // the same for every row of a launch
    bool last = false;
    if (lane == 0) sc.b_ticket[b] = 0u;               // ready for this copy's next launch
    __syncwarp();                                     // each lane's outputs and hints of this row before the row's ticket,
    // a launch of ONE batch row (the paper's own setting, batch 1) has no other row to wait for: no ticket, and the
    // slot hints go from this warp's look-ups to its adds in registers
    const bool lone_row = e.B == 1 && p.B == 1;
    if (!lone_row) {
        if (lane == 0) last = atom_add_acq_rel(sc.g_ticket, 1u) == static_cast<unsigned int>(e.B) - 1u;   // whose add releases them
        last = __shfl_sync(kFull, last, 0);
        if (!last) return;
    }

    // ---- every batch row is final (lane 0 has acquired what their warps released): S6 ----
    __syncwarp();
    OcmStatsDev *st = p.ocm.stats;
    // new keys are claimed by the look-ups (above) except near the key limit, where the
    // update itself inserts: only then does the key count have to be read afterwards
    const bool keys_settled = !p.do_update || regime != kRegimeTransition;
    unsigned long long nk = 0;
    if (lane == 0 && keys_settled) nk = atomicAdd(&st->n_keys, 0ull);   // in flight next to the hint loads
    if (p.do_update) {
        if (lone_row && regime != kRegimeTransition)
            apply_hint(p, own_hint);
        else
            apply_step_update(p, sc, lane, canon, regime);
    }
    if (p.K_total != 0 && p.alive_out) {
        // the batch rows that accepted every position of this launch go on to the next phase: their list, ascending
        int n_alive = 0;
        for (int b0 = 0; b0 < e.B; b0 += 32) {
            const int bb = b0 + lane;
            bool alive = false;
            long long br = 0;
            if (bb < e.B) {
                br = p.row_map ? __ldcg(p.row_map + bb) : bb;
                alive = __ldcg(p.accept_len + br) == p.pos0 + p.K;
            }
            const unsigned int mask = __ballot_sync(kFull, alive);
            if (alive) p.alive_out[n_alive + __popc(mask & ((1u << lane) - 1u))] = static_cast<int>(br);
            n_alive += __popc(mask);
        }
        if (lane == 0) *p.n_alive_out = n_alive;
    }
    if (lane == 0) {
        if (!keys_settled) {
            fence_acq_rel();
            nk = atomicAdd(&st->n_keys, 0ull);
        }
        st->n_keys_start = nk;
        if (p.K_total == 0 || p.count_step) atomicAdd(&st->steps, 1ull);
        *sc.g_ticket = 0u;
        st_release(p.completed, seq + 1u);            // everything above, and all it observed, first
    }
}

// ---- the kernel ------------------------------------------------------------------------

template <typename L>
__global__ void __launch_bounds__(1024) csd_step_kernel(const __grid_constant__ StepParams p)
{
    __shared__ BlockState bs;
    __shared__ RowScratch row_scratch[kFinalizeWarps];
    __shared__ CanonScratch canon;

    using E = typename L::elem;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int nwarps = blockDim.x >> 5;
    // Launch sequence number, one atomic: the word counts the blocks of every launch on this
    // workspace since it was cleared, and every launch between two clears has the same grid
    // (the host clears a workspace before a step of another layout uses it), so a block's
    // launch number is its count divided by the grid size.  The next launch can begin only
    // after every block of this one has released it, which a block does after its own count
    // has come back -- so the counts of two launches never interleave.
    // The block's LAST warp does this, so that the round trip of the (contended) atomic
    // delays neither the other warps' start nor the set-up of the shared tables; it joins
    // the streaming afterwards.
    const bool seq_warp = warp == nwarps - 1;
    unsigned long long seq_old = 0;
    if (seq_warp && lane == 0) seq_old = atomicAdd(p.launch_seq, 1ull);
    const int K1 = p.K + 1;
    const int U = p.units_per_row;
    const int CH = p.chunk_units;
    const int cpr = (U + CH - 1) / CH;                       // chunks of a whole row
    Extent e;
    e.B = p.B;
    e.G = p.n_spans;
    e.T = p.total_units;
    if (p.K_total != 0 && p.n_rows) {
        // a launch over a list of batch rows that an earlier launch wrote: the extent comes from the device, and the
        // blocks that share the work are re-derived from it by the host's rules (at most 64 per logit row, at least
        // min_units units each)
        e.B = __ldcg(p.n_rows);
        const long long rows = static_cast<long long>(e.B) * K1;
        e.T = rows * U;
        long long blocks = gridDim.x;
        if (blocks > rows * 64) blocks = rows * 64;
        const long long most = (e.T + p.min_units - 1) / p.min_units;
        if (blocks > most) blocks = most;
        e.G = static_cast<int>(blocks);
    }
    const bool idle = static_cast<int>(blockIdx.x) >= e.G;    // only possible for a launch over a row list
    long long g = idle ? 0 : span_begin(p, e, blockIdx.x);
    const long long g_end = idle ? 0 : span_begin(p, e, blockIdx.x + 1);
    // quotients of unit and row indices: 32-bit division where the host found that everything fits
    auto quot = [&](long long a, int b) -> long long {
        return p.narrow ? static_cast<long long>(static_cast<unsigned int>(a) / static_cast<unsigned int>(b)) : a / b;
    };

    bool first_window = true;
    while (g < g_end) {
        // ---- a window: up to kMaxSegs consecutive row parts of this block's span ----
        const long long row0 = quot(g, U);
        const int o0 = static_cast<int>(g - row0 * U);
        long long w_end = (row0 + kMaxSegs) * U;
        if (w_end > g_end) w_end = g_end;
        const int nseg = static_cast<int>(quot(w_end - row0 * U + U - 1, U));
        const long long first_len = w_end - row0 * U;        // units from row0's start to the window end
        const int b0 = first_len < U ? static_cast<int>(first_len) : U;
        const int n0 = (b0 - o0 + CH - 1) / CH;               // chunks of the first row part
        const int last_units = static_cast<int>(w_end - (row0 + nseg - 1) * U);
        const int n_last = (last_units + CH - 1) / CH;
        const int nchunks = nseg == 1 ? n0 : n0 + (nseg - 2) * cpr + n_last;
        const int next_b = w_end < g_end ? static_cast<int>(quot(quot(w_end, U), K1)) : -1;
        // the first window's fold count has one extra party: the sequence number's arrival
        const unsigned int fold_target = static_cast<unsigned int>(nseg) + (first_window ? 1u : 0u);

        // ---- S1 for chunk q of the window: which row part, which run of it, and its reduction ----
        struct ChunkAt {
            int seg, seg_first, seg_n;
            bool ok;
        };
        auto reduce_chunk = [&](unsigned int q, Partial &r) -> ChunkAt {
            ChunkAt at;
            int k, ua, ub;
            if (static_cast<int>(q) < n0) {
                at.seg = 0; k = q; at.seg_first = 0; at.seg_n = n0; ua = o0; ub = b0;
            } else {
                const int rr = static_cast<int>(q) - n0;
                at.seg = 1 + rr / cpr;
                k = rr - (at.seg - 1) * cpr;
                at.seg_first = n0 + (at.seg - 1) * cpr;
                ua = 0;
                if (at.seg == nseg - 1) { at.seg_n = n_last; ub = last_units; } else { at.seg_n = cpr; ub = U; }
            }
            const long long row = row0 + at.seg;
            const long long b = quot(row, K1);
            const int i = static_cast<int>(row - b * K1);
            const E *rp = logit_row<L>(p, b, i);
            const int u0 = ua + k * CH;
            const int u1 = min(ub, u0 + CH);
            const int e0 = u0 * p.unit_elems;
            const long long e1l = static_cast<long long>(u1) * p.unit_elems;
            const int e1 = e1l < p.V ? static_cast<int>(e1l) : p.V;
            at.ok = CSD_INDEX_OK(row < static_cast<long long>(e.B) * K1 && at.seg >= 0 && at.seg < nseg && nseg <= kMaxSegs &&
                                     q < static_cast<unsigned int>(kMaxChunks) && e0 >= 0 && e0 < e1 &&
                                     at.seg_first + at.seg_n <= kMaxChunks,
                                 p.ocm.stats, 5u);
            if (at.ok) r = warp_tile<L>(rp, e0, e1, lane);
            return at;
        };
        // ---- deliver a chunk's result; the warp bringing a row part's last chunk folds that part, the warp
        // completing the block's last fold publishes ----
        auto deliver = [&](unsigned int q, const ChunkAt &at, const Partial &r) {
            bool seg_complete = false;
            if (lane == 0) {
                bs.chunk_part[q] = r;
                __threadfence_block();
                seg_complete = atomicAdd(&bs.seg_done[at.seg], 1u) == static_cast<unsigned int>(at.seg_n) - 1u;
            }
            if (!__shfl_sync(kFull, seg_complete, 0)) return;
            __threadfence_block();
            Partial v = partial_identity();
            for (int j = lane; j < at.seg_n; j += 32) {
                const Partial x = bs.chunk_part[at.seg_first + j];
                v = (j == lane) ? x : combine(v, x);
            }
            v = butterfly_fold(v, 32);
            bool block_complete = false;
            if (lane == 0) {
                bs.seg_result[at.seg] = v;
                __threadfence_block();
                block_complete = atomicAdd(&bs.segs_folded, 1u) == fold_target - 1u;
            }
            if (!__shfl_sync(kFull, block_complete, 0)) return;
            __threadfence_block();
            publish_parts(p, e, bs, static_cast<int>(row0), nseg, next_b, lane);
        };

        // The shared tables of the window.  In the block's first window nothing waits for them yet: every warp
        // first takes chunk number `warp` without asking and reduces it, so that its loads are in flight a few
        // hundred cycles after the block started; the tables are needed only to deliver the result.
        if (threadIdx.x == 0) {
            bs.next_chunk = first_window ? static_cast<unsigned int>(nwarps) : 0u;
            bs.segs_folded = 0u;
            bs.n_todo = 0;
            if (!first_window) {
                bs.pre_b[0] = -1;
                bs.pre_b[1] = -1;
            }
        }
        if (threadIdx.x < kMaxSegs) bs.seg_done[threadIdx.x] = 0u;   // kMaxSegs <= 32: warp 0 only
        if (!first_window) __syncthreads();
        if (first_window && seq_warp) {
            // The launch's sequence number has arrived: from here on the next launch on the stream may begin.
            // This comes before the warp's own first chunk, because every block of a launch must get here
            // before the next launch can start at all.
            // While the sequence number travels, the same warp fetches the draft tokens of the first two batch
            // rows the block touches (a block that later finalises one of them finds them in shared memory).
            const int fb = static_cast<int>(quot(row0, K1));
            const bool two = quot(row0 + nseg - 1, K1) > fb;
            int d0 = -1, d1 = -1;
            if (lane < p.K) {
                d0 = __ldg(p.draft + place_of(p, fb).pos + lane);
                if (two) d1 = __ldg(p.draft + place_of(p, fb + 1).pos + lane);
            }
            if (lane == 0)
                bs.seq = (seq_old >> 32) == 0ull ? static_cast<unsigned int>(seq_old) / gridDim.x
                                                 : static_cast<unsigned int>(seq_old / gridDim.x);
            __syncwarp();
            pdl_launch_dependents();
            if (lane < p.K) {
                bs.pre_d[0][lane] = d0;
                bs.pre_d[1][lane] = d1;
                if (static_cast<unsigned int>(d0) < static_cast<unsigned int>(p.V)) prefetch_l2(logit_row<L>(p, fb, lane) + d0);
                if (static_cast<unsigned int>(d1) < static_cast<unsigned int>(p.V)) prefetch_l2(logit_row<L>(p, fb + 1, lane) + d1);
            }
            __syncwarp();
            if (lane == 0) {
                bs.pre_b[0] = fb;
                bs.pre_b[1] = two ? fb + 1 : -1;
            }
        }

        for (bool static_pick = first_window;; static_pick = false) {
            unsigned int q = static_cast<unsigned int>(warp);
            if (!static_pick) {
                if (lane == 0) q = atomicAdd(&bs.next_chunk, 1u);
                q = __shfl_sync(kFull, q, 0);
                if (q >= static_cast<unsigned int>(nchunks)) break;
            }
            Partial r;
            ChunkAt at;
            at.ok = false;
            if (q < static_cast<unsigned int>(nchunks)) at = reduce_chunk(q, r);
            if (static_pick) {
                // ---- once per block: the tables are set up; the sequence number counts as one more fold ----
                if (nwarps == 1) {
                    __syncthreads();
                } else if (seq_warp) {
                    named_barrier_sync(2, 64);                  // tables are set up (warp 0 arrived)
                } else {
                    if (warp == 0) named_barrier_arrive(2, 64);
                    named_barrier_sync(1, 32 * (nwarps - 1));   // the other warps go on without the last warp
                }
                if (seq_warp) {
                    bool block_complete = false;
                    if (lane == 0) {
                        __threadfence_block();
                        block_complete = atomicAdd(&bs.segs_folded, 1u) == fold_target - 1u;
                    }
                    if (__shfl_sync(kFull, block_complete, 0)) {   // everything else was already folded
                        __threadfence_block();
                        publish_parts(p, e, bs, static_cast<int>(row0), nseg, next_b, lane);
                    }
                }
            }
            if (at.ok) deliver(q, at, r);
        }
        first_window = false;
        // ---- the batch rows this block completed are shared out over its warps: S2..S6 ----
        __syncthreads();
        const int fin_warps = nwarps < kFinalizeWarps ? nwarps : kFinalizeWarps;
        if (warp < fin_warps && CSD_INDEX_OK(bs.n_todo >= 0 && bs.n_todo <= kMaxSegs, p.ocm.stats, 6u))
            for (int j = warp; j < bs.n_todo; j += fin_warps)
                finalize_and_update<L>(p, e, bs.seq, bs.todo_b[j], lane, row_scratch[warp], canon, bs);
        g = w_end;
        if (g < g_end) __syncthreads();       // the next window reuses the shared-memory tables
    }
}

}  // namespace csd
