// Stochastic verification (Algorithm 1 as printed, temperature T > 0):
//     alpha = min(1, p(d)/q(d)), accepted iff r <= alpha                       (Eq. 2)
//     else  t* ~ norm(max(0, p - q)),  is_freq, is_safe against t*, UpdateMemory, rescue
//     all accepted: bonus token ~ p_{gamma+1}
// with p = softmax(z/T), q = softmax(y/T).
//
// A categorical draw is an exponential race: the winner among items with weights W and clocks
// E ~ Exp(1) is argmax W / E; clocks are E = -ln(1 - u), u from one word of Philox4x32-10 keyed by
// the call's seed (clock n of stream s of a draw: word n & 3 of counter (n >> 2, row, s, 0)).  It runs
// in two levels: among the groups of eight consecutive tokens (stream 0), then among the winning
// group's tokens (stream 1).  A race is one more streaming arg-max: no normaliser, no prefix sums, and
// every tile of a row can run independently.
//
// Algorithm 1 stops a row at its first un-rescued rejection, so most residual draws of a step are never
// needed: a row's FIRST failed position always is, the later ones only if that one was rescued.  The
// draws therefore run in two rounds: round 1 races each row's first failed position (or its bonus row if
// every position passed) and finalises every row that stops there; round 2 races the remaining failed
// positions and the bonus row of the rows whose first failure was rescued, and finalises those.
// A step of a few megabytes makes all of them in ONE round instead (round 0: every failed position and every bonus
// row; B and C once): there two launches cost more than the draws that are saved.
//
// Six launches (A, A2, B1, C1, B2, C2; or four: A, A2, B0, C0) plus the memory's update kernel.  Each is launched programmatically
// behind the one before and waits for it (griddepcontrol.wait) before it reads or writes anything that
// others share.  B, C and the update kernel let their successor in before they wait, the decision kernel
// only when it exits.  Kernel A reads only the step's inputs and writes only the chunk statistics, which
// nobody else writes and only this step's decision kernel reads: with step overlap switched on, the
// statistics kernel of step n+1 may therefore stream as soon as step n's decision kernel has finished
// and step n's later kernels are all resident (in practice: beside its second round and its update),
// and waits for them at its end -- so that its own completion, which the next decision kernel waits
// for, implies theirs.
//   A  sampled_stats_kernel    every row of z and y once: max and sum exp(x/T) per chunk
//   A2 sampled_decide_kernel   per position: normalisers, alpha, the stochastic test
//   B  sampled_race_kernel     the round's draws (z and y rows again; bonus rows: z only): best group
//                              key per tile, atomicMax into one word per draw
//   C  sampled_finalize_kernel per batch row: t*, look-up, gate, prefix scan, outputs
// followed by the memory's own update kernel on the recorded pairs.
#pragma once

#include "csd_common.cuh"
#include "csd_ocm.cuh"
#include "csd_step.cuh"

namespace csd {

struct RowNorm {
    float m;        // max of the raw logits
    float lse2;     // log2 of sum_v 2^(x_v * log2(e)/T): the normaliser in base-2 units
    int argmax;     // lowest index attaining m
    float zcut;     // target rows: a token whose logit is below this can never win the row's draw
                    // (see race_skip_bound); -inf if no bound is known
};

// The best group of a draw so far, as one word that atomicMax can maintain: the key's bits above (keys
// are positive floats, whose bit patterns order like their values), ~group below (so that of two equal
// keys the lower group wins).  0 = no group with a positive weight yet.  The maximum does not depend on
// the order in which the tiles arrive.
__device__ __forceinline__ unsigned long long race_pack(float key, int group)
{
    return (static_cast<unsigned long long>(__float_as_uint(key)) << 32) | (0xffffffffu - static_cast<unsigned int>(group));
}

struct SampledParams {
    const void *z, *y;
    int B, K, V;
    long long z_sb, z_sk, y_sb, y_sk;
    const int *draft;
    const float *r;
    unsigned int seed_lo, seed_hi;
    float l2e_T;              // log2(e) / T
    OcmView ocm;
    float log_tau;
    int *accept_len;
    int *next_token;
    unsigned char *rescued;
    int *rej_d;
    int *rej_t;
    csd_sampled_diag_t diag;
    // workspace
    Partial *stat_part;       // [(B*(K+1) + B*K) * nchunks]
    RowNorm *rownorm;         // [B*(K+1) + B*K]: target rows first, then draft rows
    float *alpha;             // [B*K]
    unsigned char *accepted;  // [B*K]
    unsigned long long *race_best;   // [B*(K+1)] see race_pack; cleared by the decision kernel
    unsigned char *row_state; // [B] 1 while a batch row still needs the second round of draws
    int chunk_elems, nchunks;             // tiles of the statistics kernel
    int race_chunk_elems, race_nchunks;   // tiles of the race kernel: smaller, a round has few rows to spread
};

__device__ __forceinline__ long long sampled_rows_z(const SampledParams &p) { return static_cast<long long>(p.B) * (p.K + 1); }

template <typename E>
__device__ __forceinline__ const E *sampled_row_ptr(const SampledParams &p, long long row)
{
    const long long rz = sampled_rows_z(p);
    if (row < rz) {
        const long long b = row / (p.K + 1);
        const int i = static_cast<int>(row - b * (p.K + 1));
        return reinterpret_cast<const E *>(p.z) + b * p.z_sb + i * p.z_sk;
    }
    row -= rz;
    const long long b = row / p.K;
    const int i = static_cast<int>(row - b * p.K);
    return reinterpret_cast<const E *>(p.y) + b * p.y_sb + i * p.y_sk;
}

// ---- A: per-chunk max / sum exp(x/T) of every row of both tensors -------------------------

template <typename L>
__global__ void __launch_bounds__(256) sampled_stats_kernel(const __grid_constant__ SampledParams p)
{
    using E = typename L::elem;
    const int lane = threadIdx.x & 31;
    const long long warps = static_cast<long long>(gridDim.x) * (blockDim.x >> 5);
    const long long rows = sampled_rows_z(p) + static_cast<long long>(p.B) * p.K;
    const long long tiles = rows * p.nchunks;
    pdl_launch_dependents();
    for (long long tile = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); tile < tiles; tile += warps) {
        const long long row = tile / p.nchunks;
        const int c = static_cast<int>(tile - row * p.nchunks);
        const int e0 = c * p.chunk_elems;
        const int e1 = min(p.V, e0 + p.chunk_elems);
        const Partial r = warp_tile<L>(sampled_row_ptr<E>(p, row), e0, e1, lane, p.l2e_T);
        if (lane == 0) st_partial_cg(p.stat_part + tile, r);
    }
    pdl_wait();       // this kernel's completion then implies that of everything before it on the stream
}

// A weight that can never win a draw.  Clocks lie in [E_min, E_max] = [-ln(1 - 2^-24), -ln(2^-24)]
// = [5.96e-8, 16.64].  If some token is known to have weight w0 > 0, the winning key is at least
// w0 / E_max (its group weighs at least w0), and a group of eight tokens that each weigh
// w <= 3.7e-10 * w0 has key <= 8 w / E_min <= 0.0497 * w0 < w0 / E_max = 0.0601 * w0: it loses
// whatever the clocks are (the 20 % margin dwarfs rounding).  The bound depends only on the row's
// statistics, so skipping by it changes no result bit.
__device__ __forceinline__ float race_skip_bound(float w0) { return w0 > 0.0f ? 3.7e-10f * w0 : 0.0f; }

// ---- A2: normalisers, alpha and the stochastic test, one warp per (b, i <= K) --------------

// All lanes return the row's statistics.  Lane k pre-folds chunks k, k+32, ... in order, then a
// fixed-shape butterfly: the result does not depend on timing.
__device__ __forceinline__ RowNorm fold_row_norm(const SampledParams &p, long long row, int lane)
{
    Partial acc = partial_identity();
    for (int c = lane; c < p.nchunks; c += 32) {
        const Partial x = ld_partial_cg(p.stat_part + row * p.nchunks + c);
        acc = (c == lane) ? x : combine(acc, x);
    }
    acc = butterfly_fold(acc, 32, p.l2e_T);
    RowNorm n;
    n.m = acc.m;
    n.lse2 = acc.c + log2f(acc.s);
    n.argmax = acc.idx;
    n.zcut = -INFINITY;
    return n;
}

// The same for two rows at once (a position's target and draft row): both rows' loads are in flight together.
__device__ __forceinline__ void fold_row_norm2(const SampledParams &p, long long row_a, long long row_b, int lane, RowNorm &na, RowNorm &nb)
{
    Partial a = partial_identity(), b = partial_identity();
    for (int c = lane; c < p.nchunks; c += 32) {
        const Partial xa = ld_partial_cg(p.stat_part + row_a * p.nchunks + c);
        const Partial xb = ld_partial_cg(p.stat_part + row_b * p.nchunks + c);
        a = (c == lane) ? xa : combine(a, xa);
        b = (c == lane) ? xb : combine(b, xb);
    }
    a = butterfly_fold(a, 32, p.l2e_T);
    b = butterfly_fold(b, 32, p.l2e_T);
    na.m = a.m; na.lse2 = a.c + log2f(a.s); na.argmax = a.idx; na.zcut = -INFINITY;
    nb.m = b.m; nb.lse2 = b.c + log2f(b.s); nb.argmax = b.idx; nb.zcut = -INFINITY;
}

// The logit below which p(v) <= race_skip_bound(w0): (z - m) * l2e_T - (lse2 - m * l2e_T) <= log2(bound),
// lowered by 1e-3 so that rounding can only make the cut more cautious.
__device__ __forceinline__ float race_logit_cut(const RowNorm &n, float w0, float l2e_T)
{
    const float bound = race_skip_bound(w0);
    if (!(bound > 0.0f)) return -INFINITY;
    return static_cast<float>((static_cast<double>(n.lse2) + log2(static_cast<double>(bound))) / static_cast<double>(l2e_T) - 1e-3);
}

template <typename L>
__global__ void __launch_bounds__(128) sampled_decide_kernel(const __grid_constant__ SampledParams p)
{
    using E = typename L::elem;
    const int lane = threadIdx.x & 31;
    const long long n = sampled_rows_z(p);
    const long long j = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    pdl_wait();
    // no early trigger here: the kernels behind this one let their own successors in at once, down to the
    // next step's statistics kernel, which overwrites the chunk statistics this kernel is reading
    if (j >= n) return;
    const int K = p.K;
    const long long b = j / (K + 1);
    const int i = static_cast<int>(j - b * (K + 1));
    const long long pos = b * K + i;
    const long long yrow = n + pos;
    // the draft token and its two logits do not depend on the folds: requested first
    int d = -1;
    float zd = 0.0f, yd = 0.0f;
    if (i < K) {
        d = __ldg(p.draft + pos);
        if (static_cast<unsigned int>(d) < static_cast<unsigned int>(p.V)) {
            zd = L::load_elem(sampled_row_ptr<E>(p, j), d);
            yd = L::load_elem(sampled_row_ptr<E>(p, yrow), d);
        }
    }
    RowNorm np_, nq;
    if (i < K) {
        fold_row_norm2(p, j, yrow, lane, np_, nq);
    } else {
        np_ = fold_row_norm(p, j, lane);
        nq = np_;
    }
    if (lane != 0) return;
    p.race_best[j] = 0ull;
    if (!(np_.lse2 == np_.lse2) || np_.lse2 == INFINITY || np_.m == -INFINITY) atomicOr(&p.ocm.stats->flags, CSD_FLAG_NAN_LOGIT);
    if (p.diag.lse_p) p.diag.lse_p[j] = np_.lse2 * 0.6931471805599453f;
    // the probability of the row's arg-max: a weight known to take part in a draw from p
    const float p_top = exp2f(static_cast<float>(static_cast<double>(np_.m) * static_cast<double>(p.l2e_T) - static_cast<double>(np_.lse2)));
    if (i == K) {
        np_.zcut = race_logit_cut(np_, p_top, p.l2e_T);
        p.rownorm[j] = np_;
        return;
    }
    p.rownorm[yrow] = nq;
    {
        // the residual weight p - q at the target's arg-max (if positive) takes part in the residual draw
        const float y_top = L::load_elem(sampled_row_ptr<E>(p, yrow), np_.argmax);
        const float q_top = exp2f(static_cast<float>(static_cast<double>(y_top) * static_cast<double>(p.l2e_T) - static_cast<double>(nq.lse2)));
        np_.zcut = race_logit_cut(np_, 0.99f * (p_top - q_top), p.l2e_T);     // 1 % off for the rounding of p_top - q_top
        p.rownorm[j] = np_;
    }
    if (!(nq.lse2 == nq.lse2) || nq.lse2 == INFINITY || nq.m == -INFINITY) atomicOr(&p.ocm.stats->flags, CSD_FLAG_NAN_LOGIT);
    if (p.diag.lse_q) p.diag.lse_q[pos] = nq.lse2 * 0.6931471805599453f;
    float alpha = 0.0f;
    bool ok = false;
    if (static_cast<unsigned int>(d) < static_cast<unsigned int>(p.V)) {
        // log2 p(d) - log2 q(d) in double (one per position); alpha = min(1, p(d)/q(d))      (Eq. 2)
        const double lr = (static_cast<double>(zd) - static_cast<double>(yd)) * static_cast<double>(p.l2e_T) -
                          (static_cast<double>(np_.lse2) - static_cast<double>(nq.lse2));
        alpha = lr >= 0.0 ? 1.0f : static_cast<float>(exp2(lr));
        ok = __ldg(p.r + pos) <= alpha;
    } else {
        atomicOr(&p.ocm.stats->flags, CSD_FLAG_BAD_DRAFT);
    }
    p.alpha[pos] = alpha;
    p.accepted[pos] = ok ? 1 : 0;
    if (p.diag.alpha) p.diag.alpha[pos] = alpha;
    if (p.diag.accepted) p.diag.accepted[pos] = ok ? 1 : 0;
}

// ---- B: exponential races --------------------------------------------------------------------
//
// Two levels.  First among the groups of 8 consecutive tokens, weight W_g = sum of the group's
// weights, clock number g of stream 0: this is what kernel B streams for.  Then among the 8
// tokens of the winning group, clock number v of stream 1: eight gathers in kernel C.
// P(v) = W_g / sum W * w(v) / W_g = w(v) / sum w, with one random number per eight tokens.

constexpr int kRaceGroup = 8;

__device__ __forceinline__ uint4 philox4x32_10(uint4 c, unsigned int k0, unsigned int k1)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const unsigned int hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
        const unsigned int hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
        c = make_uint4(hi1 ^ c.y ^ k0, lo1, hi0 ^ c.w ^ k1, lo0);
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return c;
}

__device__ __forceinline__ unsigned int philox_word(const uint4 &r, unsigned int n)
{
    return (n & 3u) == 0u ? r.x : (n & 3u) == 1u ? r.y : (n & 3u) == 2u ? r.z : r.w;
}

// u = (j + 1/2) / 2^23 from the top 23 bits of a word: exact in binary32, and so is 1 - u.
__device__ __forceinline__ float clock_u(unsigned int word) { return (static_cast<float>(word >> 9) + 0.5f) * 1.1920928955078125e-07f; }
__device__ __forceinline__ float clock_of(float u) { return -log1pf(-u); }      // E = -ln(1 - u) ~ Exp(1)

// What a draw needs of its two rows.  Weights are w(v) = max(0, 2^((z-mz)*s - lp) - 2^((y-my)*s - lq))
// with lp = Lp - mz*s: the row maxima are taken out first so that the exponents of the tokens
// that matter are small and exact; a bonus draw has no draft row and w = p.
struct DrawCoef {
    float s, mz, lp, my, lq, zcut;
    bool has_q;
};

__device__ __forceinline__ DrawCoef draw_coef(const SampledParams &p, long long row, bool bonus, long long yrow)
{
    DrawCoef c;
    const RowNorm np_ = p.rownorm[row];
    c.s = p.l2e_T;
    c.mz = np_.m;
    c.lp = static_cast<float>(static_cast<double>(np_.lse2) - static_cast<double>(np_.m) * static_cast<double>(p.l2e_T));
    c.zcut = np_.zcut;
    c.has_q = !bonus;
    c.my = 0.0f;
    c.lq = 0.0f;
    if (!bonus) {
        const RowNorm nq = p.rownorm[yrow];
        c.my = nq.m;
        c.lq = static_cast<float>(static_cast<double>(nq.lse2) - static_cast<double>(nq.m) * static_cast<double>(p.l2e_T));
    }
    return c;
}

__device__ __forceinline__ float draw_weight(const DrawCoef &c, float z, float y)
{
    float w = ex2_approx(fmaf(z - c.mz, c.s, -c.lp));
    if (c.has_q) w -= ex2_approx(fmaf(y - c.my, c.s, -c.lq));
    return fmaxf(w, 0.0f);
}

// Sum of a group's weights, in a fixed order.  The affine part runs on packed pairs (one instruction
// for two tokens; each half rounds exactly like the scalar operation in draw_weight).
__device__ __forceinline__ float group_weight(const DrawCoef &c, const float (&z)[8], const float (&y)[8])
{
    const unsigned long long s2 = pack2(c.s, c.s);
    const unsigned long long nmz = pack2(-c.mz, -c.mz), nlp = pack2(-c.lp, -c.lp);
    const unsigned long long nmy = pack2(-c.my, -c.my), nlq = pack2(-c.lq, -c.lq);
    float w[8];
#pragma unroll
    for (int e = 0; e < 8; e += 2) {
        float a0, a1;
        unpack2(fma2(add2(pack2(z[e], z[e + 1]), nmz), s2, nlp), a0, a1);
        w[e] = ex2_approx(a0);
        w[e + 1] = ex2_approx(a1);
        if (c.has_q) {
            float b0, b1;
            unpack2(fma2(add2(pack2(y[e], y[e + 1]), nmy), s2, nlq), b0, b1);
            w[e] -= ex2_approx(b0);
            w[e + 1] -= ex2_approx(b1);
        }
        w[e] = fmaxf(w[e], 0.0f);
        w[e + 1] = fmaxf(w[e + 1], 0.0f);
    }
    return ((w[0] + w[1]) + (w[2] + w[3])) + ((w[4] + w[5]) + (w[6] + w[7]));
}

struct RaceBest {
    float key;
    int idx;
};

// Eight consecutive tokens of a row starting at v0 (a multiple of 8); tokens at or beyond V read
// as -inf (weight 0).  The vector forms need the row 16-byte aligned.
template <typename L>
struct Group8;

template <>
struct Group8<LaneBf16Vec> {
    static constexpr int kVec = 1;
    static __device__ __forceinline__ void load(const __nv_bfloat16 *row, int v0, int V, uint4 (&raw)[1]) { raw[0] = ld_stream16(row + v0); }
    static __device__ __forceinline__ float hmax(const uint4 (&raw)[1]) { return LaneBf16Vec::hmax(raw[0]); }
    static __device__ __forceinline__ void unpack(const uint4 (&raw)[1], float (&f)[8]) { LaneBf16Vec::unpack(raw[0], f); }
};

template <>
struct Group8<LaneF32Vec> {
    static constexpr int kVec = 2;
    static __device__ __forceinline__ void load(const float *row, int v0, int V, uint4 (&raw)[2])
    {
        // a lane's two vectors share a 32-byte sector: cached loads, so that the second one hits
        raw[0] = __ldg(reinterpret_cast<const uint4 *>(row + v0));
        raw[1] = v0 + 4 < V ? __ldg(reinterpret_cast<const uint4 *>(row + v0 + 4)) : LaneF32Vec::neg_inf();   // V is a multiple of 4 here
    }
    static __device__ __forceinline__ float hmax(const uint4 (&raw)[2]) { return fmaxf(LaneF32Vec::hmax(raw[0]), LaneF32Vec::hmax(raw[1])); }
    static __device__ __forceinline__ void unpack(const uint4 (&raw)[2], float (&f)[8])
    {
        float a[4], b[4];
        LaneF32Vec::unpack(raw[0], a);
        LaneF32Vec::unpack(raw[1], b);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            f[e] = a[e];
            f[4 + e] = b[e];
        }
    }
};

template <typename L>
struct Group8Scalar {
    static constexpr int kVec = 8;
    using E = typename L::elem;
    static __device__ __forceinline__ void load(const E *row, int v0, int V, float (&raw)[8])
    {
#pragma unroll
        for (int e = 0; e < 8; ++e) raw[e] = v0 + e < V ? L::load_elem(row, v0 + e) : -INFINITY;
    }
    static __device__ __forceinline__ float hmax(const float (&raw)[8])
    {
        float m = raw[0];
#pragma unroll
        for (int e = 1; e < 8; ++e) m = fmaxf(m, raw[e]);
        return m;
    }
    static __device__ __forceinline__ void unpack(const float (&raw)[8], float (&f)[8])
    {
#pragma unroll
        for (int e = 0; e < 8; ++e) f[e] = raw[e];
    }
};

template <>
struct Group8<LaneF32Scalar> : Group8Scalar<LaneF32Scalar> {};
template <>
struct Group8<LaneBf16Scalar> : Group8Scalar<LaneBf16Scalar> {};

template <typename L>
struct Group8Raw {
    using type = uint4;
};
template <>
struct Group8Raw<LaneF32Scalar> {
    using type = float;
};
template <>
struct Group8Raw<LaneBf16Scalar> {
    using type = float;
};

template <typename L>
__global__ void __launch_bounds__(256, 4) sampled_race_kernel(const __grid_constant__ SampledParams p, const int round)
{
    using E = typename L::elem;
    using G = Group8<L>;
    using Raw = typename Group8Raw<L>::type;
    constexpr int kGroups = G::kVec == 1 ? 4 : G::kVec == 2 ? 2 : 1;      // groups a lane has in flight (8 vectors)
    const int lane = threadIdx.x & 31;
    const int K = p.K;
    const long long warps = static_cast<long long>(gridDim.x) * (blockDim.x >> 5);
    const long long draws = sampled_rows_z(p);
    // round 1 has one draw per batch row (tiles run over batch rows), round 2 up to K per pending row; round 0 is the
    // single round of a step that makes every draw a row could need at once (all failed positions, every bonus row)
    const long long tiles = (round == 1 ? static_cast<long long>(p.B) : draws) * p.race_nchunks;
    pdl_launch_dependents();
    pdl_wait();
    for (long long tile = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); tile < tiles; tile += warps) {
        const long long unit = tile / p.race_nchunks;
        const int c = static_cast<int>(tile - unit * p.race_nchunks);
        const long long b = round == 1 ? unit : unit / (K + 1);
        if (round == 2 && p.row_state[b] == 0) continue;            // finalised in round 1
        // f0 = the batch row's first failed position, K if none
        const unsigned int failed = __ballot_sync(kFull, lane < K && p.accepted[b * K + lane] == 0);
        const int f0 = failed ? __ffs(failed) - 1 : K;
        const int i = round == 1 ? f0 : static_cast<int>(unit - b * (K + 1));
        const bool bonus = i == K;
        if (round == 2 && !(i > f0 && (bonus || ((failed >> i) & 1u)))) continue;
        if (round == 0 && !(bonus || ((failed >> i) & 1u))) continue;
        const long long row = b * (K + 1) + i;
        const long long yrow = draws + b * K + i;
        const DrawCoef cf = draw_coef(p, row, bonus, yrow);
        const E *zr = sampled_row_ptr<E>(p, row);
        const E *yr = bonus ? zr : sampled_row_ptr<E>(p, yrow);
        const int g0 = c * (p.race_chunk_elems / kRaceGroup);
        const int g1 = min((p.V + kRaceGroup - 1) / kRaceGroup, g0 + p.race_chunk_elems / kRaceGroup);
        RaceBest best;
        best.key = 0.0f;
        best.idx = 0x7fffffff;
        for (int gb = g0; gb < g1; gb += 32 * kGroups) {
            Raw zraw[kGroups][G::kVec], yraw[kGroups][G::kVec];
#pragma unroll
            for (int k = 0; k < kGroups; ++k) {
                const int g = gb + k * 32 + lane;
                if (g < g1) {
                    G::load(zr, g * kRaceGroup, p.V, zraw[k]);
                    if (!bonus) G::load(yr, g * kRaceGroup, p.V, yraw[k]);
                }
            }
#pragma unroll
            for (int k = 0; k < kGroups; ++k) {
                const int g = gb + k * 32 + lane;
                // A group all of whose logits are below the row's cut cannot win: no exponentials.
                float W = 0.0f;
                if (g < g1 && G::hmax(zraw[k]) > cf.zcut) {
                    float zf[8], yf[8];
                    G::unpack(zraw[k], zf);
                    if (!bonus) G::unpack(yraw[k], yf);
                    W = group_weight(cf, zf, bonus ? zf : yf);
                }
                // One Philox block serves four consecutive groups, i.e. four consecutive lanes: the
                // first of them computes it when any of the four has a weight, the others take its words.
                const unsigned int need = __ballot_sync(kFull, W > 0.0f);
                if (need == 0u) continue;                    // (the whole warp) nothing here can win: no clocks
                const int leader = lane & ~3;
                uint4 rnd = make_uint4(0u, 0u, 0u, 0u);
                if (lane == leader && ((need >> leader) & 0xfu))
                    rnd = philox4x32_10(make_uint4(static_cast<unsigned int>(g) >> 2, static_cast<unsigned int>(row), 0u, 0u), p.seed_lo, p.seed_hi);
                rnd.x = __shfl_sync(kFull, rnd.x, leader);
                rnd.y = __shfl_sync(kFull, rnd.y, leader);
                rnd.z = __shfl_sync(kFull, rnd.z, leader);
                rnd.w = __shfl_sync(kFull, rnd.w, leader);
                if (W > 0.0f) {
                    const float u = clock_u(philox_word(rnd, static_cast<unsigned int>(g)));
                    if (W > best.key * u) {                  // E >= u: otherwise the key cannot exceed the best
                        const float key = W / clock_of(u);
                        if (key > best.key) {                // groups ascend within a lane: strict keeps the lowest
                            best.key = key;
                            best.idx = g;
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float ok = __shfl_xor_sync(kFull, best.key, o);
            const int oi = __shfl_xor_sync(kFull, best.idx, o);
            if (ok > best.key || (ok == best.key && oi < best.idx)) {
                best.key = ok;
                best.idx = oi;
            }
        }
        if (lane == 0 && best.key > 0.0f) atomicMax(p.race_best + row, race_pack(best.key, best.idx));
    }
}

// ---- C: per batch row: the draws' winners, look-up, gate, prefix scan -----------------------

// The drawn token of draw `row`: the winning group over the row's chunks, then the race among its
// (up to) eight tokens.  `fallback` if no group has a positive weight.
template <typename L>
__device__ __forceinline__ int race_winner(const SampledParams &p, long long row, bool bonus, long long yrow, int fallback)
{
    using E = typename L::elem;
    const unsigned long long top = __ldcg(p.race_best + row);
    if (top == 0ull) return fallback;
    const int g = static_cast<int>(0xffffffffu - static_cast<unsigned int>(top & 0xffffffffull));
    const DrawCoef cf = draw_coef(p, row, bonus, yrow);
    const E *zr = sampled_row_ptr<E>(p, row);
    const E *yr = bonus ? zr : sampled_row_ptr<E>(p, yrow);
    float zf[kRaceGroup], yf[kRaceGroup];
#pragma unroll
    for (int e = 0; e < kRaceGroup; ++e) {       // all gathers in flight together
        const int v = g * kRaceGroup + e;
        zf[e] = v < p.V ? L::load_elem(zr, v) : -INFINITY;
        yf[e] = (v < p.V && !bonus) ? L::load_elem(yr, v) : -INFINITY;
    }
    float best = 0.0f;
    int t = g * kRaceGroup;
    uint4 rnd = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
    for (int e = 0; e < kRaceGroup; ++e) {
        const int v = g * kRaceGroup + e;
        if ((e & 3) == 0) rnd = philox4x32_10(make_uint4(static_cast<unsigned int>(v) >> 2, static_cast<unsigned int>(row), 1u, 0u), p.seed_lo, p.seed_hi);
        const float w = draw_weight(cf, zf[e], yf[e]);
        if (w > 0.0f) {
            const float k2 = w / clock_of(clock_u(philox_word(rnd, static_cast<unsigned int>(v))));
            if (k2 > best) {        // tokens ascend: strict keeps the lowest
                best = k2;
                t = v;
            }
        }
    }
    return t;
}

template <typename L>
__global__ void __launch_bounds__(128) sampled_finalize_kernel(const __grid_constant__ SampledParams p, const int round)
{
    using E = typename L::elem;
    const int lane = threadIdx.x & 31;
    const int K = p.K;
    const long long b = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    pdl_launch_dependents();
    pdl_wait();
    if (b >= p.B) return;
    if (round == 2 && p.row_state[b] == 0) return;       // finalised in round 1
    const long long row0 = b * (K + 1);

    bool passed = false, valid = false, ok = false;
    int d = -1, t = -1;
    unsigned int cnt = 0;
    if (lane < K) {
        const long long pos = b * K + lane;
        d = __ldg(p.draft + pos);
        valid = static_cast<unsigned int>(d) < static_cast<unsigned int>(p.V);
        passed = p.accepted[pos] != 0;
    }
    const unsigned int failed = __ballot_sync(kFull, lane < K && !passed);
    const int f0 = failed ? __ffs(failed) - 1 : K;        // the row's first failed position
    // The draws that exist so far: round 1 has made the one of position f0 (the bonus draw if f0 = K),
    // round 2 all the others of this row.  Lane i < K takes its residual draw t* ~ norm(max(0, p - q)),
    // lane K the bonus draw t ~ p_{gamma+1} -- one code path, so that they run side by side.
    const bool is_bonus = lane == K;
    const bool have = round == 1 ? lane == f0 : ((lane < K && !passed) || is_bonus);       // round 0: all of them exist
    int drawn = -1;
    if (have && lane <= K)
        drawn = race_winner<L>(p, row0 + lane, is_bonus, sampled_rows_z(p) + b * K + lane, p.rownorm[row0 + lane].argmax);
    float score = __int_as_float(0x7fc00000);
    if (lane < K) {
        ok = passed;
        if (!passed && have) {
            t = drawn;
            if (valid) {
                const E *zr = sampled_row_ptr<E>(p, row0 + lane);
                const float zd = L::load_elem(zr, d);
                const float zt = L::load_elem(zr, t);
                cnt = ocm_lookup(p.ocm, make_key(d, t));
                const bool is_freq = cnt >= p.ocm.lambda;
                const bool is_safe = (static_cast<double>(zd) - static_cast<double>(zt)) >= static_cast<double>(p.log_tau);   // Eq. 3
                ok = is_freq && is_safe;
                score = expf(zd - zt);
            }
        }
    }
    if (round == 1) {
        // first failure rescued: the row goes on, and needs the draws of round 2
        const bool pending = f0 < K && __shfl_sync(kFull, ok, f0);
        if (lane == 0) p.row_state[b] = pending ? 1 : 0;
        if (pending) return;
    }
    if (lane < K) {
        const long long pos = b * K + lane;
        if (p.diag.t_star) p.diag.t_star[pos] = t;
        if (p.diag.score) p.diag.score[pos] = score;
        if (p.diag.cnt) p.diag.cnt[pos] = cnt;
    }
    int bonus_t = K < 32 ? drawn : -1;          // lane K's, if there is a lane K and the draw was made
    if (K == 32 && lane == 0 && (round != 1 || f0 == K)) bonus_t = race_winner<L>(p, row0 + K, true, 0, p.rownorm[row0 + K].argmax);
    bonus_t = __shfl_sync(kFull, bonus_t, K < 32 ? K : 0);
    const unsigned int kmask = (K == 32) ? kFull : ((1u << K) - 1u);
    const unsigned int okmask = __ballot_sync(kFull, ok) & kmask;
    const unsigned int fail = ~okmask & kmask;
    const int n_acc = fail ? (__ffs(fail) - 1) : K;
    const bool reached = lane <= n_acc && lane < K;
    const bool record = reached && !passed && valid;
    if (lane < K) {
        const long long pos = b * K + lane;
        p.rescued[pos] = (lane < n_acc && !passed) ? 1 : 0;
        p.rej_d[pos] = record ? d : -1;
        p.rej_t[pos] = record ? t : -1;
    }
    const int t_stop = __shfl_sync(kFull, t, n_acc < K ? n_acc : 0);
    const unsigned int m_pass = __ballot_sync(kFull, reached && passed);
    const unsigned int m_resc = __ballot_sync(kFull, lane < n_acc && !passed && lane < K);
    const unsigned int m_rec = __ballot_sync(kFull, record);
    if (lane == 0) {
        int next = t_stop;
        if (n_acc == K) next = bonus_t;
        p.accept_len[b] = n_acc;
        p.next_token[b] = next;
        if (p.diag.bonus) p.diag.bonus[b] = bonus_t;
        OcmStatsDev *st = p.ocm.stats;
        atomicAdd(&st->positions, static_cast<unsigned long long>(K));
        if (m_pass) atomicAdd(&st->matches, static_cast<unsigned long long>(__popc(m_pass)));
        if (m_resc) atomicAdd(&st->rescues, static_cast<unsigned long long>(__popc(m_resc)));
        if (m_rec) atomicAdd(&st->rejections, static_cast<unsigned long long>(__popc(m_rec)));
        if (b == 0) atomicAdd(&st->steps, 1ull);
    }
}

}  // namespace csd
