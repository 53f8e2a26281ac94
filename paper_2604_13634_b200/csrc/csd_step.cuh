// The fused verification step: stream every logit row once (max / arg-max / sum-exp),
// then, per batch row, match test, OCM look-up, the gate of Eq. 3, the prefix scan of
// Algorithm 1's verification loop, and finally the memory update -- one launch.
//
// Work decomposition
//   * The R = B*(K+1) logit rows are cut into tiles of `tile_elems` contiguous
//     elements (at most ~32 tiles per row); a tile is reduced by ONE WARP on its own:
//     there is no block barrier anywhere.  Warps are persistent workers: tile t goes to
//     block t mod G, warp (t / G) mod 8, so every SM gets the same number of tiles +-1
//     and batch rows complete in index order while later ones are still streaming.
//   * A lane keeps 8 x 16 bytes in flight; a tile is reduced with a running maximum,
//     an integer reference exponent and four independent sum accumulators; only the
//     iteration in which the maximum last improved is remembered, and the exact
//     lowest arg-max index is recovered by re-reading that one iteration (an L2 hit).
//   * After each tile lane 0 stores the partial, fences, and takes a ticket on the
//     batch row's arrival counter.  Whichever warp delivers the last tile of a batch
//     row finalises it: the row's partials are prefetched together and folded by a
//     segmented warp scan in a fixed order (bit-reproducible sums), lanes 0..K-1 take
//     the per-position decisions, a ballot gives the accepted prefix.
//   * Memory update without a second probe: the look-up already found each recorded
//     pair's slot (absent pairs get an empty slot reserved with count 0, which no
//     look-up can tell from "absent"), and leaves it as a hint.  The warp finalising
//     the LAST batch row then only adds 1 to the hinted slots, so every look-up of the
//     step saw the step-start counts.  Near the key limit, where admission order
//     matters, that warp falls back to the canonical-order path.
//   * Nothing ever waits for another block: arrival counters only, so no launch can hang.
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
    Partial *partials;       // [R * n_split]
    long long *slot_hint;    // [B * K] slot of each recorded pair (see kHint*)
    unsigned int *b_ticket;  // [B]
    unsigned int *g_ticket;  // [1]
    int tile_elems;
    int n_split;             // tiles per logit row
    int total_tiles;
};

constexpr long long kHintNone = -1;          // nothing to record at this position
constexpr long long kHintAbsent = -2;        // recorded pair not in the table and no slot reserved
constexpr long long kHintCareful = 1ll << 62; // count close to saturation: add with the wrap check

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
    static __device__ __forceinline__ void accum(unit a, float negc, float &s0, float &s1)
    {
        s0 += ex2_approx(fmaf(__uint_as_float(a.x), kLog2e, negc));
        s1 += ex2_approx(fmaf(__uint_as_float(a.y), kLog2e, negc));
        s0 += ex2_approx(fmaf(__uint_as_float(a.z), kLog2e, negc));
        s1 += ex2_approx(fmaf(__uint_as_float(a.w), kLog2e, negc));
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
    static __device__ __forceinline__ void accum2(unsigned int w, float negc, float &s0, float &s1)
    {
        s0 += ex2_approx(fmaf(lo(w), kLog2e, negc));
        s1 += ex2_approx(fmaf(hi(w), kLog2e, negc));
    }
    static __device__ __forceinline__ void accum(unit a, float negc, float &s0, float &s1)
    {
        accum2(a.x, negc, s0, s1);
        accum2(a.y, negc, s0, s1);
        accum2(a.z, negc, s0, s1);
        accum2(a.w, negc, s0, s1);
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
    static __device__ __forceinline__ void accum(unit a, float negc, float &s0, float &s1)
    {
        s0 += ex2_approx(fmaf(a, kLog2e, negc));
        (void)s1;
    }
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
    static __device__ __forceinline__ void accum(unit a, float negc, float &s0, float &s1)
    {
        s0 += ex2_approx(fmaf(a, kLog2e, negc));
        (void)s1;
    }
    static __device__ __forceinline__ int first_eq(unit a, float v) { return a == v ? 0 : -1; }
};

// ---- S1: one warp reduces one tile ---------------------------------------------------

template <typename L>
__device__ __forceinline__ Partial warp_tile(const typename L::elem *row, int e0, int e1, int lane)
{
    using U = typename L::unit;
    const typename L::elem *base = row + e0;
    const int nunits = (e1 - e0) / L::kPer;
    constexpr int kPerIter = 32 * kUnroll;
    const int nfull = nunits / kPerIter;

    float m_thr = -INFINITY;   // running maximum of this lane
    float c_thr = kNoRef;      // integer reference exponent of the accumulators
    int it_thr = -1;           // iteration of the last strict improvement
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
    U v[kUnroll];

    auto consume = [&](const U (&v)[kUnroll], int it) {
        U mx = L::vmax(L::vmax(L::vmax(v[0], v[1]), L::vmax(v[2], v[3])),
                       L::vmax(L::vmax(v[4], v[5]), L::vmax(v[6], v[7])));
        const float bmax = L::hmax(mx);
        if (bmax > m_thr) {
            m_thr = bmax;
            it_thr = it;
            const float cn = rintf(bmax * kLog2e);
            if (cn > c_thr) {
                const float f = pow2_nonpos(c_thr - cn);
                s0 *= f; s1 *= f; s2 *= f; s3 *= f;
                c_thr = cn;
            }
        }
        const float negc = -c_thr;
#pragma unroll
        for (int k = 0; k < kUnroll; k += 2) {
            L::accum(v[k], negc, s0, s1);
            L::accum(v[k + 1], negc, s2, s3);
        }
    };

    for (int it = 0; it < nfull; ++it) {
#pragma unroll
        for (int k = 0; k < kUnroll; ++k) v[k] = L::load(base, (it * kUnroll + k) * 32 + lane);
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

    // warp maximum, then everything is rescaled to the warp's reference exponent
    float wmax = m_thr;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) wmax = fmaxf(wmax, __shfl_xor_sync(kFull, wmax, o));
    const float cw = (wmax == -INFINITY) ? kNoRef : rintf(wmax * kLog2e);
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

// ---- S2..S5 for one batch row, by one warp ------------------------------------------

struct RowScratch {
    float m[CSD_MAX_K + 1];
    float s[CSD_MAX_K + 1];
    int t[CSD_MAX_K + 1];
};

enum UpdateRegime { kRegimeRoom = 0, kRegimeFull = 1, kRegimeTransition = 2 };

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

template <typename L>
__device__ void finalize_batch_row(const StepParams &p, int b, int lane, RowScratch &rs)
{
    using E = typename L::elem;
    const int K = p.K, K1 = p.K + 1;
    const int n = K1 * p.n_split;
    const Partial *part = p.partials + (size_t)b * n;
    const size_t row0 = (size_t)b * K1;

    // S2 (first half): the draft tokens and their logits do not depend on the
    // reduction, so their loads are issued before the partials are folded.
    int d = -1;
    bool valid = false;
    float zd = __int_as_float(0x7fc00000);
    if (lane < K) {
        d = __ldg(p.draft + (size_t)b * K + lane);
        valid = static_cast<unsigned int>(d) < static_cast<unsigned int>(p.V);
        if (valid) {
            const E *rowp = reinterpret_cast<const E *>(p.logits) + (size_t)b * p.stride_b + (size_t)lane * p.stride_k;
            zd = L::load_elem(rowp, d);
        }
    }

    // S1 (second half): fold the K+1 rows' partials with a segmented inclusive scan,
    // 32 partials at a time, always in the same order; up to 256 are fetched at once.
    Partial carry = partial_identity();
    int carry_row = -1;
    for (int g0 = 0; g0 < n; g0 += 256) {
        Partial pre[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int e = g0 + q * 32 + lane;
            pre[q] = e < n ? ld_partial_cg(part + e) : partial_identity();
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int base = g0 + q * 32;
            if (base >= n) break;
            const int e = base + lane;
            const bool in = e < n;
            const int row = in ? e / p.n_split : 0x7ffffff0 + lane;
            Partial v = pre[q];
            if (lane == 0 && carry_row == row) v = combine(carry, v);
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const Partial up = shfl_up_partial(v, o);
                const int up_row = __shfl_up_sync(kFull, row, o);
                if (lane >= o && up_row == row) v = combine(up, v);
            }
            if (in && (e + 1) % p.n_split == 0) {
                // last partial of a row: v is the row's total.  sum exp(x - m) = s * 2^(c - m log2 e)
                const float r = fmaf(-v.m, kLog2e, v.c);
                const float s_m = v.s * exp2f(r);
                rs.m[row] = v.m;
                rs.s[row] = s_m;
                rs.t[row] = v.idx;
                if (!(s_m == s_m) || s_m == INFINITY) atomicOr(&p.ocm.stats->flags, CSD_FLAG_NAN_LOGIT);
                if (p.diag.m) p.diag.m[row0 + row] = v.m;
                if (p.diag.s) p.diag.s[row0 + row] = s_m;
                if (p.diag.lse) p.diag.lse[row0 + row] = v.m + logf(s_m);
                if (p.diag.t) p.diag.t[row0 + row] = v.idx;
            }
            carry = shfl_partial(v, 31);
            carry_row = __shfl_sync(kFull, row, 31);
        }
    }
    __syncwarp();

    // S2 (second half), S3, S4 per position; S5 across the warp.
    bool match = false, ok = false;
    int t = -1;
    unsigned int cnt = 0;
    long long slot = -1;
    if (lane < K) {
        t = rs.t[lane];
        const float m = rs.m[lane];
        const float s_m = rs.s[lane];
        match = (d == t);
        if (valid) cnt = ocm_lookup(p.ocm, make_key(d, t), &slot);                     // S3
        const bool is_freq = cnt >= p.ocm.lambda;
        const bool is_safe = (static_cast<double>(zd) - static_cast<double>(m)) >= static_cast<double>(p.log_tau);  // S4, Eq. 3
        ok = match || (valid && is_freq && is_safe);
        const size_t pos = (size_t)b * K + lane;
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
        const size_t pos = (size_t)b * K + lane;
        p.rescued[pos] = (lane < n_acc && !match) ? 1 : 0;
        p.rej_d[pos] = record ? d : -1;
        p.rej_t[pos] = record ? t : -1;
        if (p.do_update) {
            // S6, first half: leave the slot of every recorded pair for the final adder
            long long hint = kHintNone;
            if (record) {
                if (slot < 0 && update_regime(p) == kRegimeRoom) slot = ocm_reserve(p.ocm, make_key(d, t));
                hint = slot < 0 ? kHintAbsent : slot;
                const unsigned int room = 0xffffffffu - static_cast<unsigned int>(p.B * p.K);
                if (slot >= 0 && cnt > room) hint |= kHintCareful;
            }
            __stcg(p.slot_hint + pos, hint);
        }
    }
    const unsigned int m_match = __ballot_sync(kFull, reached && match);
    const unsigned int m_resc = __ballot_sync(kFull, lane < n_acc && !match && lane < K);
    const unsigned int m_rec = __ballot_sync(kFull, record);
    const unsigned int m_bad = __ballot_sync(kFull, lane < K && !valid);
    if (lane == 0) {
        p.accept_len[b] = n_acc;
        p.next_token[b] = rs.t[n_acc];
        OcmStatsDev *st = p.ocm.stats;
        atomicAdd(&st->positions, static_cast<unsigned long long>(K));
        if (m_match) atomicAdd(&st->matches, static_cast<unsigned long long>(__popc(m_match)));
        if (m_resc) atomicAdd(&st->rescues, static_cast<unsigned long long>(__popc(m_resc)));
        if (m_rec) atomicAdd(&st->rejections, static_cast<unsigned long long>(__popc(m_rec)));
        if (m_bad) atomicOr(&st->flags, CSD_FLAG_BAD_DRAFT);
    }
    __syncwarp();
}

// S6, second half, by the warp that finalised the last batch row: every look-up of the
// step is done, so the counts may change now.
__device__ void apply_step_update(const StepParams &p, int lane, CanonScratch &canon)
{
    const int n = p.B * p.K;
    const int regime = update_regime(p);
    if (regime == kRegimeTransition) {
        ocm_update_group<false>(p.ocm, p.rej_d, p.rej_t, nullptr, n, canon, lane, 32);
        return;
    }
    unsigned int dropped = 0;
    for (int j = lane; j < n; j += 32) {
        const long long h = __ldcg(p.slot_hint + j);
        if (h >= 0) {
            const unsigned long long s = static_cast<unsigned long long>(h & ~kHintCareful);
            if (h & kHintCareful)
                ocm_add(p.ocm, s, 1u);
            else
                atomicAdd(&p.ocm.slots[s].count, 1u);
        } else if (h == kHintAbsent) {
            ++dropped;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) dropped += __shfl_xor_sync(kFull, dropped, o);
    if (lane == 0 && dropped) atomicAdd(&p.ocm.stats->n_dropped, static_cast<unsigned long long>(dropped));
    __syncwarp();
}

// ---- the kernel ------------------------------------------------------------------------

template <typename L>
__global__ void __launch_bounds__(kThreads, 4) csd_step_kernel(const __grid_constant__ StepParams p)
{
    __shared__ RowScratch row_scratch[kWarps];
    __shared__ CanonScratch canon;

    using E = typename L::elem;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int K1 = p.K + 1;
    const int G = gridDim.x;
    const int W = G * kWarps;
    const unsigned int tiles_per_b = static_cast<unsigned int>(K1 * p.n_split);

    for (int tile = warp * G + blockIdx.x; tile < p.total_tiles; tile += W) {
        // ---- S1: this warp reduces one tile ----
        const int row = tile / p.n_split;
        const int chunk = tile - row * p.n_split;
        const int b = row / K1;
        const int i = row - b * K1;
        const E *rp = reinterpret_cast<const E *>(p.logits) + (size_t)b * p.stride_b + (size_t)i * p.stride_k;
        const int e0 = chunk * p.tile_elems;
        const int e1 = min(p.V, e0 + p.tile_elems);
        const Partial r = warp_tile<L>(rp, e0, e1, lane);

        // ---- publish it and take a ticket on the batch row's arrival counter ----
        bool completes = false;
        if (lane == 0) {
            st_partial_cg(p.partials + tile, r);
            __threadfence();
            completes = atomicAdd(p.b_ticket + b, 1u) == tiles_per_b - 1;
        }
        completes = __shfl_sync(kFull, completes, 0);
        if (!completes) continue;

        // ---- this warp delivered the batch row's last tile: S2..S5 ----
        __threadfence();
        finalize_batch_row<L>(p, b, lane, row_scratch[warp]);
        bool last = false;
        if (lane == 0) p.b_ticket[b] = 0u;               // ready for the next launch
        __threadfence();
        __syncwarp();
        if (lane == 0) last = atomicAdd(p.g_ticket, 1u) == static_cast<unsigned int>(p.B) - 1u;
        last = __shfl_sync(kFull, last, 0);
        if (!last) continue;

        // ---- every batch row is final: S6 ----
        __threadfence();
        if (p.do_update) apply_step_update(p, lane, canon);
        if (lane == 0) {
            OcmStatsDev *st = p.ocm.stats;
            __threadfence();
            st->n_keys_start = atomicAdd(&st->n_keys, 0ull);
            atomicAdd(&st->steps, 1ull);
            *p.g_ticket = 0u;
        }
    }
}

}  // namespace csd
