"""CPU oracle for the STOCHASTIC verification step of Calibrated Speculative Decoding.

TEST INFRASTRUCTURE ONLY (see csd_oracle.py: same rules; the only code shared with
that module is the memory class and the input decoders, which are oracle code too).

Algorithm 1 of the paper as it is printed, at temperature T > 0, one step, all float64:

    p_i = softmax(z_i / T)            target distribution at position i      (M_p^(T))
    q_i = softmax(y_i / T)            draft distribution at position i       (M_q^(T))
    r ~ U[0,1];  alpha = min(1, p_i(d) / q_i(d));   r <= alpha: accepted     (Eq. 2)
    else  t* ~ norm(max(0, p_i - q_i))                                       (residual)
          is_freq = T[(d, t*)] >= lambda                                     (Sec. 4.2)
          is_safe = p_i^(T=1)(d) / p_i^(T=1)(t*) >= tau
                  = z_i(d) - z_i(t*) >= ln tau   (raw logits, any T)         (Eq. 3)
          UpdateMemory(T, d, t*)
          is_freq and is_safe: rescued, go on;  else stop, emit t*
    all gamma accepted: emit t ~ p_{gamma+1}

Readings (the paper leaves these open; each is a convention of this build):
  S1  the uniforms r are INPUTS (one per position).
  S2  a categorical draw from non-negative weights w(v) is an exponential race: among
      items with weights W and independent clocks E ~ Exp(1) the winner is
      argmax W / E, lowest index on ties; P(item wins) = W / sum W exactly.  It needs
      no normaliser, no prefix sum and no second pass, and the integer it returns is
      well conditioned: it can only change when two keys nearly coincide.  (An
      inverse-CDF draw would make the index depend on rounding in a 150 000-term
      prefix sum.)  `draw_plain` is that race as the textbooks state it: one level,
      one clock per token, arg-max over the whole vocabulary.  `draw`, the one the
      step uses, runs it in two levels: first among the groups of GROUP = 8
      consecutive tokens (weight = the sum of the group), then among the tokens of
      the winning group: P(v) = W_g / sum W * w(v) / W_g = w(v) / sum w.  The two are
      different maps from a seed to a token and the same sampler; the tests pin them
      to each other and to w / sum w as distributions.  GROUP and the clock grid of
      S3 are frozen: they are part of the seed-to-token contract of the C header.
  S3  a clock is E = -ln(1 - u), u = (j + 1/2) / 2^23, j = the top 23 bits of one
      32-bit word (so that u and 1 - u are exact in binary32 as well) of
      Philox4x32-10 (Salmon et al., "Parallel random numbers: as easy as 1, 2, 3",
      SC'11) with key = (seed low, seed high).  Clock number n of stream s of draw
      `row` is word n & 3 of counter (n >> 2, row, s, 0); group g uses clock g of
      stream 0, token v uses clock v of stream 1; row = b * (K+1) + i (i = K: the
      bonus draw).
  S4  look-ups see the memory as it was when the step began; rejections are added
      afterwards in (b, i) order (as in the greedy oracle).
  S5  near-ties are reported, not decided on: |r - alpha| < 1e-5 for the acceptance
      test; for a draw, the winner (group, then token) is "clear" if it still wins
      after every p is scaled by (1 -+ 1e-5) and every q by (1 +- 1e-5) against it.  A result that depends on a
      near-tie is excluded from exactness by the tests.
  S6  a draft id outside [0, V) is a rejection that cannot be rescued and is not
      recorded; its alpha is 0.  PARITY UNPINNED (paper silent).
  S7  if every weight of a draw is zero (p == q everywhere: cannot follow a rejection
      in exact arithmetic) the draw falls back to the lowest arg-max of z.
"""

from __future__ import annotations

import numpy as np

from .csd_oracle import OCM, as_f64, scg_threshold  # noqa: F401  (OCM re-exported for the tests)

BAND = 1e-5

# ----------------------------------------------------------------------------
# Philox4x32-10, from its published definition (S3)
# ----------------------------------------------------------------------------
_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = 0x9E3779B9
_W1 = 0xBB67AE85
_MASK = np.uint64(0xFFFFFFFF)


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Ten rounds of Philox-4x32 on arrays of counters (uint32 values in uint64 arrays)."""
    c0 = np.asarray(c0, dtype=np.uint64); c1 = np.asarray(c1, dtype=np.uint64)
    c2 = np.asarray(c2, dtype=np.uint64); c3 = np.asarray(c3, dtype=np.uint64)
    k0 = int(k0) & 0xFFFFFFFF
    k1 = int(k1) & 0xFFFFFFFF
    for _ in range(10):
        p0 = _M0 * c0                      # 32 x 32 -> 64 bit products
        p1 = _M1 * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & _MASK
        hi1, lo1 = p1 >> np.uint64(32), p1 & _MASK
        c0, c1, c2, c3 = (hi1 ^ c1 ^ np.uint64(k0)), lo1, (hi0 ^ c3 ^ np.uint64(k1)), lo0
        k0 = (k0 + _W0) & 0xFFFFFFFF
        k1 = (k1 + _W1) & 0xFFFFFFFF
    return c0, c1, c2, c3


GROUP = 8


def race_clocks(seed: int, row: int, stream: int, first: int, n: int) -> np.ndarray:
    """Clocks first .. first+n-1 of stream `stream` of draw `row` (S3), float64, ~ Exp(1)."""
    idx = np.arange(first, first + n, dtype=np.uint64)
    blk = idx >> np.uint64(2)
    z = np.zeros(n, dtype=np.uint64)
    w = philox4x32_10(blk, z + np.uint64(row), z + np.uint64(stream), z, seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    words = np.choose((idx & np.uint64(3)).astype(np.int64), w)
    j = (words >> np.uint64(9)).astype(np.float64)
    u = (j + 0.5) / 8388608.0
    return -np.log1p(-u)


# ----------------------------------------------------------------------------
# distributions of one position
# ----------------------------------------------------------------------------
def log_softmax_T(x: np.ndarray, T: float):
    """(log-probabilities of softmax(x / T), max of x, lse of x / T)."""
    x = as_f64(x) / float(T)
    m = np.max(x)
    lse = m + np.log(np.sum(np.exp(x - m)))
    return x - lse, float(m * float(T)), float(lse)


def race(weights: np.ndarray, clocks: np.ndarray, fallback: int):
    """argmax_v weights[v] / clocks[v], lowest index on ties (S2); S7 if all weights are 0."""
    key = weights / clocks
    best = np.max(key)
    if not best > 0:
        return int(fallback), best
    return int(np.flatnonzero(key == best)[0]), float(best)


def _weights(p, q, sp=1.0, sq=1.0):
    return np.maximum(0.0, p * sp - (q * sq if q is not None else 0.0))


def _by_group(w):
    pad = (-len(w)) % GROUP
    return np.concatenate([w, np.zeros(pad)]).reshape(-1, GROUP)


def draw(p, q, seed: int, row: int, fallback: int):
    """One draw from norm(max(0, p - q)) (q None: from p) by the two-level race (S2, S3).

    Returns (token, clear): `clear` is False when the winning group or the winning token would
    change under relative perturbations of BAND on p and q (S5)."""
    w = _by_group(_weights(p, q))
    n_groups = w.shape[0]
    e_g = race_clocks(seed, row, 0, 0, n_groups)
    g, best = race(w.sum(axis=1), e_g, -1)
    if g < 0:                                                     # S7
        return int(fallback), True
    e_t = race_clocks(seed, row, 1, g * GROUP, GROUP)
    t, _ = race(w[g], e_t, 0)
    lo = _by_group(_weights(p, q, 1 - BAND, 1 + BAND))
    hi = _by_group(_weights(p, q, 1 + BAND, 1 - BAND))
    hi_g = hi.sum(axis=1) / e_g
    hi_g[g] = 0.0
    hi_t = hi[g] / e_t
    hi_t[t] = 0.0
    clear = lo[g].sum() / e_g[g] > np.max(hi_g) and lo[g, t] / e_t[t] > np.max(hi_t)
    return g * GROUP + t, bool(clear)


PLAIN_STREAM = 2      # the clocks of draw_plain: a stream of their own, one clock per token


def draw_plain(p, q, seed: int, row: int, fallback: int) -> int:
    """One draw from norm(max(0, p - q)) (q None: from p) by the ONE-level exponential race (S2):
    argmax_v w(v) / E_v over the whole vocabulary, lowest index on ties, clock v of stream
    PLAIN_STREAM of the draw's row; `fallback` if every weight is zero (S7).

    The reference statement of the categorical draws of Algorithm 1 (t* ~ norm(max(0, p - q)) and
    t ~ p_{gamma+1}).  `verify` does not call it: it exists so that the two-level `draw` can be
    pinned to the plain definition as a sampler of the same distribution."""
    w = _weights(p, q)
    t, _ = race(w, race_clocks(seed, row, PLAIN_STREAM, 0, len(w)), -1)
    return int(fallback) if t < 0 else t


# ----------------------------------------------------------------------------
# one step
# ----------------------------------------------------------------------------
def verify(z, y, draft, r, seed: int, T: float, ocm: OCM, tau: float):
    """Stochastic verification-and-rescue over z[B,K+1,V], y[B,K,V], draft[B,K], r[B,K].

    Returns a dict: accept_len, next_token, rescued_mask, rej_draft, rej_target (as the
    greedy oracle), and per position: alpha, accepted (the stochastic test alone),
    t_star (the residual draw of EVERY position that fails the stochastic test, reached
    or not; -1 where it passes), lse_p [B,K+1], lse_q [B,K], score = exp(z_d - z_t*),
    cnt, and the near-tie flags near_accept, unclear_draw [B,K+1] (column K: bonus draw).
    The memory is not modified; see `step`.
    """
    z = np.asarray(z); y = np.asarray(y)
    B, K1, V = z.shape
    K = K1 - 1
    draft = np.asarray(draft).reshape(B, K)
    r = np.asarray(r, dtype=np.float64).reshape(B, K)
    lf = scg_threshold(tau)

    alpha = np.zeros((B, K)); accepted = np.zeros((B, K), dtype=bool)
    t_star = np.full((B, K), -1, dtype=np.int64)
    lse_p = np.zeros((B, K1)); lse_q = np.zeros((B, K))
    score = np.full((B, K), np.nan); cnt = np.zeros((B, K), dtype=np.int64)
    near_accept = np.zeros((B, K), dtype=bool); unclear = np.zeros((B, K1), dtype=bool)
    accept_len = np.zeros(B, dtype=np.int32); next_token = np.zeros(B, dtype=np.int32)
    rescued = np.zeros((B, K), dtype=np.uint8)
    rej_d = np.full((B, K), -1, dtype=np.int32); rej_t = np.full((B, K), -1, dtype=np.int32)
    bonus = np.zeros(B, dtype=np.int64)

    for b in range(B):
        for i in range(K1):
            lp, _, lse_p[b, i] = log_softmax_T(z[b, i], T)
            row = b * K1 + i
            if i == K:                                              # bonus draw t ~ p_{gamma+1}
                bonus[b], clear = draw(np.exp(lp), None, seed, row, int(np.argmax(as_f64(z[b, i]))))
                unclear[b, i] = not clear
                continue
            lq, _, lse_q[b, i] = log_softmax_T(y[b, i], T)
            d = int(draft[b, i])
            if 0 <= d < V:
                alpha[b, i] = min(1.0, float(np.exp(lp[d] - lq[d])))             # Eq. 2
            accepted[b, i] = bool(r[b, i] <= alpha[b, i]) and 0 <= d < V
            near_accept[b, i] = abs(r[b, i] - alpha[b, i]) < BAND
            if accepted[b, i]:
                continue
            t_star[b, i], clear = draw(np.exp(lp), np.exp(lq), seed, row, int(np.argmax(as_f64(z[b, i]))))   # residual
            unclear[b, i] = not clear
            if 0 <= d < V:
                score[b, i] = np.exp(float(z[b, i, d]) - float(z[b, i, t_star[b, i]]))
                cnt[b, i] = ocm.count(d, t_star[b, i])

    for b in range(B):
        n = K
        for i in range(K):
            if accepted[b, i]:
                continue
            d = int(draft[b, i]); tt = int(t_star[b, i])
            if not (0 <= d < V):                                    # S6
                n = i
                break
            is_freq = cnt[b, i] >= ocm.lam
            is_safe = bool((float(z[b, i, d]) - float(z[b, i, tt])) >= lf)       # Eq. 3
            rej_d[b, i] = d
            rej_t[b, i] = tt
            if is_freq and is_safe:
                rescued[b, i] = 1
                continue
            n = i
            break
        accept_len[b] = n
        next_token[b] = bonus[b] if n == K else t_star[b, n]

    return dict(accept_len=accept_len, next_token=next_token, rescued_mask=rescued, rej_draft=rej_d,
                rej_target=rej_t, alpha=alpha, accepted=accepted, t_star=t_star, bonus=bonus, lse_p=lse_p,
                lse_q=lse_q, score=score, cnt=cnt, near_accept=near_accept, unclear_draw=unclear)


def step(z, y, draft, r, seed, T, ocm: OCM, tau):
    """verify, then feed the step's rejections to the memory in (b, i) order (S4)."""
    out = verify(z, y, draft, r, seed, T, ocm, tau)
    ocm.update(zip(out["rej_draft"].reshape(-1), out["rej_target"].reshape(-1)))
    return out
