// Stochastic verification (Algorithm 1 as printed, temperature T > 0):
//     alpha = min(1, p(d)/q(d)), accepted iff r <= alpha                       (Eq. 2)
//     else  t* ~ norm(max(0, p - q)),  is_freq, is_safe against t*, UpdateMemory, rescue
//     all accepted: bonus token ~ p_{gamma+1}
// with p = softmax(z/T), q = softmax(y/T).
//
// A categorical draw is an exponential race: argmax_v w(v) / E_v, E_v = -ln(1 - u_v),
// u_v from one word of Philox4x32-10 keyed by the call's seed, counter (v >> 2, row, 0, 0).
// A race is one more streaming arg-max: no normaliser, no prefix sums, no second pass over
// the winner's neighbourhood, and every tile of a row can run independently.
//
// Four launches, stream-ordered:
//   A  sampled_stats_kernel    every row of z and y once: max and sum exp(x/T) per chunk
//   A2 sampled_decide_kernel   per position: normalisers, alpha, the stochastic test
//   B  sampled_race_kernel     rows that failed the test (z and y again) and the bonus rows:
//                              best key per chunk
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
    float skip;     // target rows: weights up to this can never win the row's draw (see race_skip_bound)
};

struct __align__(8) RacePart {
    float key;      // best w/E of the chunk (0 if none)
    int idx;        // its index (lowest on ties), 0x7fffffff if none
};

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
    RacePart *race_part;      // [B*(K+1) * nchunks]
    int chunk_elems, nchunks;
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
    for (long long tile = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); tile < tiles; tile += warps) {
        const long long row = tile / p.nchunks;
        const int c = static_cast<int>(tile - row * p.nchunks);
        const int e0 = c * p.chunk_elems;
        const int e1 = min(p.V, e0 + p.chunk_elems);
        const Partial r = warp_tile<L>(sampled_row_ptr<E>(p, row), e0, e1, lane, p.l2e_T);
        if (lane == 0) st_partial_cg(p.stat_part + tile, r);
    }
}

// A weight that can never win a draw.  Clocks lie in [E_min, E_max] = [-ln(1 - 2^-24), -ln(2^-24)]
// = [5.96e-8, 16.64].  If some token is known to have weight w0 > 0, the winning key is at least
// w0 / E_max, and a token with weight w <= 3.0e-9 * w0 has key <= w / E_min <= 0.0503 * w0
// < w0 / E_max = 0.0601 * w0: it loses whatever the clocks are (the 19 % margin dwarfs rounding).
// The bound depends only on the row's statistics, so skipping by it changes no result bit.
__device__ __forceinline__ float race_skip_bound(float w0) { return w0 > 0.0f ? 3.0e-9f * w0 : 0.0f; }

// ---- A2: normalisers, alpha and the stochastic test, one thread per (b, i <= K) -----------

__device__ __forceinline__ RowNorm fold_row_norm(const SampledParams &p, long long row)
{
    Partial acc = partial_identity();
    for (int c = 0; c < p.nchunks; ++c) {
        Partial x = ld_partial_cg(p.stat_part + row * p.nchunks + c);
        // partials carry c = rint(m * log2(e)/T) of their own chunk; combine() rescales exactly
        acc = (c == 0) ? x : combine(acc, x);
    }
    RowNorm n;
    n.m = acc.m;
    n.lse2 = acc.c + log2f(acc.s);
    n.argmax = acc.idx;
    n.skip = 0.0f;
    return n;
}

template <typename L>
__global__ void sampled_decide_kernel(const __grid_constant__ SampledParams p)
{
    using E = typename L::elem;
    const long long n = sampled_rows_z(p);
    const long long j = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (j >= n) return;
    const int K = p.K;
    const long long b = j / (K + 1);
    const int i = static_cast<int>(j - b * (K + 1));
    RowNorm np_ = fold_row_norm(p, j);
    if (!(np_.lse2 == np_.lse2) || np_.lse2 == INFINITY || np_.m == -INFINITY) atomicOr(&p.ocm.stats->flags, CSD_FLAG_NAN_LOGIT);
    if (p.diag.lse_p) p.diag.lse_p[j] = np_.lse2 * 0.6931471805599453f;
    // the probability of the row's arg-max: a weight known to take part in a draw from p
    const float p_top = exp2f(static_cast<float>(static_cast<double>(np_.m) * static_cast<double>(p.l2e_T) - static_cast<double>(np_.lse2)));
    if (i == K) {
        np_.skip = race_skip_bound(p_top);
        p.rownorm[j] = np_;
        return;
    }
    const long long pos = b * K + i;
    const long long yrow = n + pos;
    const RowNorm nq = fold_row_norm(p, yrow);
    p.rownorm[yrow] = nq;
    {
        // the residual weight p - q at the target's arg-max (if positive) takes part in the residual draw
        const float y_top = L::load_elem(sampled_row_ptr<E>(p, yrow), np_.argmax);
        const float q_top = exp2f(static_cast<float>(static_cast<double>(y_top) * static_cast<double>(p.l2e_T) - static_cast<double>(nq.lse2)));
        np_.skip = race_skip_bound(0.99f * (p_top - q_top));     // 1 % off for the rounding of p_top - q_top
        p.rownorm[j] = np_;
    }
    if (!(nq.lse2 == nq.lse2) || nq.lse2 == INFINITY || nq.m == -INFINITY) atomicOr(&p.ocm.stats->flags, CSD_FLAG_NAN_LOGIT);
    if (p.diag.lse_q) p.diag.lse_q[pos] = nq.lse2 * 0.6931471805599453f;
    const int d = __ldg(p.draft + pos);
    float alpha = 0.0f;
    bool ok = false;
    if (static_cast<unsigned int>(d) < static_cast<unsigned int>(p.V)) {
        const float zd = L::load_elem(sampled_row_ptr<E>(p, j), d);
        const float yd = L::load_elem(sampled_row_ptr<E>(p, yrow), d);
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

struct RaceBest {
    float key;
    int idx;
};

// One candidate: weight w > 0 at index v with random word `word`.  u = (j + 1/2) / 2^23 is
// exact in binary32; E = -ln(1 - u) >= u, so a candidate with w <= best * u cannot win and
// the logarithm is skipped for it.
__device__ __forceinline__ void race_candidate(RaceBest &best, float w, unsigned int word, int v)
{
    const float u = (static_cast<float>(word >> 9) + 0.5f) * 1.1920928955078125e-07f;
    if (!(w > best.key * u)) return;
    const float key = w / (-log1pf(-u));
    if (key > best.key) {       // indices ascend within a lane: strict keeps the lowest
        best.key = key;
        best.idx = v;
    }
}

// w(v) = max(0, 2^((z-mz)*s - lp) - 2^((y-my)*s - lq)), lp = Lp - mz*s: the row maxima are
// taken out first so that the exponents of the tokens that matter are small and exact;
// without a draft row (bonus draw) w = p.
template <typename L, bool kHasQ>
__device__ __forceinline__ void race_vector(RaceBest &best, typename L::unit zv, typename L::unit yv, int v0, float s, float mz, float lp,
                                            float my, float lq, float skip, unsigned int row, unsigned int k0, unsigned int k1)
{
    float zf[L::kPer], yf[L::kPer], w[L::kPer];
    L::unpack(zv, zf);
    if (kHasQ) L::unpack(yv, yf);
#pragma unroll
    for (int e = 0; e < L::kPer; ++e) {
        w[e] = exp2f(fmaf(zf[e] - mz, s, -lp));
        if (kHasQ) w[e] -= exp2f(fmaf(yf[e] - my, s, -lq));
    }
    // one Philox block serves four consecutive indices; it is computed only if one of them can win
    constexpr int kGroup = L::kPer < 4 ? L::kPer : 4;
#pragma unroll
    for (int g0 = 0; g0 < L::kPer; g0 += kGroup) {
        bool any = false;
#pragma unroll
        for (int e = g0; e < g0 + kGroup; ++e) any = any || (w[e] > skip);
        if (!any) continue;
        const uint4 rnd = philox4x32_10(make_uint4(static_cast<unsigned int>(v0 + g0) >> 2, row, 0u, 0u), k0, k1);
#pragma unroll
        for (int e = g0; e < g0 + kGroup; ++e) {
            const int v = v0 + e;
            const unsigned int word = (v & 3) == 0 ? rnd.x : (v & 3) == 1 ? rnd.y : (v & 3) == 2 ? rnd.z : rnd.w;
            if (w[e] > skip) race_candidate(best, w[e], word, v);
        }
    }
}

template <typename L>
__global__ void __launch_bounds__(256) sampled_race_kernel(const __grid_constant__ SampledParams p)
{
    using E = typename L::elem;
    using U = typename L::unit;
    const int lane = threadIdx.x & 31;
    const int K = p.K;
    const long long warps = static_cast<long long>(gridDim.x) * (blockDim.x >> 5);
    const long long draws = sampled_rows_z(p);
    const long long tiles = draws * p.nchunks;
    for (long long tile = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5); tile < tiles; tile += warps) {
        const long long row = tile / p.nchunks;
        const int c = static_cast<int>(tile - row * p.nchunks);
        const long long b = row / (K + 1);
        const int i = static_cast<int>(row - b * (K + 1));
        const bool bonus = i == K;
        if (!bonus && p.accepted[b * K + i]) continue;       // passed the stochastic test: no draw
        const RowNorm np_ = p.rownorm[row];
        const float lp = static_cast<float>(static_cast<double>(np_.lse2) - static_cast<double>(np_.m) * static_cast<double>(p.l2e_T));
        float lq = 0.0f, my = 0.0f;
        const E *zr = sampled_row_ptr<E>(p, row);
        const E *yr = zr;
        if (!bonus) {
            const long long yrow = draws + b * K + i;
            const RowNorm nq = p.rownorm[yrow];
            my = nq.m;
            lq = static_cast<float>(static_cast<double>(nq.lse2) - static_cast<double>(nq.m) * static_cast<double>(p.l2e_T));
            yr = sampled_row_ptr<E>(p, yrow);
        }
        const int e0 = c * p.chunk_elems;
        const int e1 = min(p.V, e0 + p.chunk_elems);
        const int nunits = (e1 - e0) / L::kPer;
        RaceBest best;
        best.key = 0.0f;
        best.idx = 0x7fffffff;
        for (int u = lane; u < nunits; u += 32) {
            const int v0 = e0 + u * L::kPer;
            const U zv = L::load(zr + e0, u);
            if (bonus) {
                race_vector<L, false>(best, zv, zv, v0, p.l2e_T, np_.m, lp, 0.0f, 0.0f, np_.skip, static_cast<unsigned int>(row), p.seed_lo, p.seed_hi);
            } else {
                const U yv = L::load(yr + e0, u);
                race_vector<L, true>(best, zv, yv, v0, p.l2e_T, np_.m, lp, my, lq, np_.skip, static_cast<unsigned int>(row), p.seed_lo, p.seed_hi);
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
        if (lane == 0) {
            RacePart out;
            out.key = best.key;
            out.idx = best.idx;
            p.race_part[tile] = out;
        }
    }
}

// ---- C: per batch row: the draws' winners, look-up, gate, prefix scan -----------------------

__device__ __forceinline__ int race_winner(const SampledParams &p, long long row, int fallback)
{
    float key = 0.0f;
    int idx = fallback;
    for (int c = 0; c < p.nchunks; ++c) {
        const RacePart x = p.race_part[row * p.nchunks + c];
        if (x.key > key) {          // chunks ascend: strict keeps the lowest index
            key = x.key;
            idx = x.idx;
        }
    }
    return idx;
}

template <typename L>
__global__ void __launch_bounds__(128) sampled_finalize_kernel(const __grid_constant__ SampledParams p)
{
    using E = typename L::elem;
    const int lane = threadIdx.x & 31;
    const int K = p.K;
    const long long b = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (b >= p.B) return;
    const long long row0 = b * (K + 1);

    bool passed = false, valid = false, ok = false;
    int d = -1, t = -1;
    unsigned int cnt = 0;
    if (lane < K) {
        const long long pos = b * K + lane;
        d = __ldg(p.draft + pos);
        valid = static_cast<unsigned int>(d) < static_cast<unsigned int>(p.V);
        passed = p.accepted[pos] != 0;
        ok = passed;
        float score = __int_as_float(0x7fc00000);
        if (!passed) {
            const RowNorm np_ = p.rownorm[row0 + lane];
            t = race_winner(p, row0 + lane, np_.argmax);                                    // t* ~ norm(max(0, p - q))
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
        if (p.diag.t_star) p.diag.t_star[pos] = t;
        if (p.diag.score) p.diag.score[pos] = score;
        if (p.diag.cnt) p.diag.cnt[pos] = cnt;
    }
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
        if (n_acc == K) next = race_winner(p, row0 + K, p.rownorm[row0 + K].argmax);       // bonus ~ p_{gamma+1}
        p.accept_len[b] = n_acc;
        p.next_token[b] = next;
        if (p.diag.bonus) p.diag.bonus[b] = race_winner(p, row0 + K, p.rownorm[row0 + K].argmax);
        OcmStatsDev *st = p.ocm.stats;
        atomicAdd(&st->positions, static_cast<unsigned long long>(K));
        if (m_pass) atomicAdd(&st->matches, static_cast<unsigned long long>(__popc(m_pass)));
        if (m_resc) atomicAdd(&st->rescues, static_cast<unsigned long long>(__popc(m_resc)));
        if (m_rec) atomicAdd(&st->rejections, static_cast<unsigned long long>(__popc(m_rec)));
        if (b == 0) atomicAdd(&st->steps, 1ull);
    }
}

}  // namespace csd
