"""CPU oracle for the verification-and-rescue step of Calibrated Speculative Decoding.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what one
verification step computes; it exists so that the CUDA path can be checked
against something written independently of it.  Only the test-suite, the smoke
check and the benchmark's CPU-baseline leg may import it.  It shares no code,
table or constant with the CUDA library, and never takes a value produced by it.

Everything is float64 numpy on the exact input bits (fp32 and bf16 widen to
float64 without rounding).  The decision procedure is Algorithm 1 of the paper
in its greedy (T = 0) instantiation, the evaluation mode of Sec. 5.1:

  * with one-hot p_i and q_i the acceptance probability of Eq. 2 is 1 when the
    draft token equals argmax p_i and 0 otherwise;
  * the residual norm(max(0, p_i - q_i)) is one-hot at argmax z_i, so the
    correction token t* is the arg-max of the target logits;
  * the bonus token drawn from p_{gamma+1} is the arg-max of the last row.

Conventions the paper leaves open (each one is a reading of this build):
  R1  arg-max ties: the lowest index wins.
  R2  all look-ups of one step see the memory as it was when the step began;
      the step's rejections are added afterwards, row-major by (b, i).  For a
      single row this gives the same decisions as Algorithm 1's sequential
      order (pinned in the tests).  Across rows the paper is silent.
  R3  capacity: the memory holds at most `limit` distinct pairs.  A pair that
      is already present always counts; a new pair is admitted only while
      fewer than `limit` pairs are stored, in (b, i) order; otherwise that
      occurrence is dropped and counted.  Nothing is evicted.   PARITY UNPINNED:
      the paper fixes no capacity rule.
  R4  counts are 32-bit and saturate.
  R5  a draft id outside [0, V) is a mismatch that can never be rescued and is
      not recorded.  PARITY UNPINNED (paper is silent).
  R6  the gate of Eq. 3 is decided in logit space: (z_d - z_t*) in float64
      against float32(ln(float32 tau)); equality passes.
  R7  ageing (opt-in; an alternative to "frozen when full" under R3): `age()`
      halves every count, rounding down, and removes the pairs that reach zero,
      which frees their room for new pairs.  It depends on nothing but the
      stored set, so it is independent of order, layout and timing.  PARITY
      UNPINNED: Sec. 4.2 says the memory keeps evolving online and names no
      forgetting rule.
"""

from __future__ import annotations

import numpy as np

COUNT_MAX = 2**32 - 1
NEAR_TIE_BAND = 1e-5


# ----------------------------------------------------------------------------
# input decoding (format definitions, no arithmetic of the method)
# ----------------------------------------------------------------------------
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """bfloat16 is the upper half of an IEEE binary32: widen the bit pattern."""
    b = np.ascontiguousarray(bits).view(np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def as_f64(z: np.ndarray) -> np.ndarray:
    """float32 / float64 logits widened (exactly) to float64."""
    return np.asarray(z, dtype=np.float64)


# ----------------------------------------------------------------------------
# S1: vocabulary-wide statistics of one logit row
# ----------------------------------------------------------------------------
def row_stats(x: np.ndarray):
    """max, arg-max (lowest index, R1), s = sum exp(x - max), lse = max + ln s.

    t* of Algorithm 1 (residual arg-max at T = 0) and the soft-max normaliser
    that defines p^(T=1) in Eq. 3.
    """
    x = as_f64(x)
    m = np.max(x)
    t = int(np.flatnonzero(x == m)[0]) if not np.isnan(m) else int(np.argmax(x))
    with np.errstate(invalid="ignore", over="ignore"):
        s = float(np.sum(np.exp(x - m)))
        lse = float(m + np.log(s)) if s > 0 else float("nan")
    return float(m), t, s, lse


def scg_threshold(tau: float) -> float:
    """ln(tau) as the gate uses it (R6): float32 tau, float64 log, rounded to float32."""
    tau32 = np.float32(tau)
    if tau32 == 0:
        return float("-inf")
    return float(np.float32(np.log(np.float64(tau32))))


# ----------------------------------------------------------------------------
# the Online Correction Memory (Sec. 4.2): ordered pair -> count
# ----------------------------------------------------------------------------
class OCM:
    """Frequency table T of divergence pairs (draft token, target token)."""

    def __init__(self, n_slots: int, lam: int = 6):
        self.n_slots = int(n_slots)
        self.limit = self.n_slots // 2          # R3
        self.lam = int(lam)                     # frequency threshold lambda
        self.table: dict[tuple[int, int], int] = {}
        self.n_dropped = 0

    def reset(self):
        self.table.clear()
        self.n_dropped = 0

    def count(self, d: int, t: int) -> int:
        return self.table.get((int(d), int(t)), 0)

    def update(self, pairs, weights=None):
        """UpdateMemory of Algorithm 1 applied to a batch, in the given order (R2, R3, R4).

        Entries with a negative token are placeholders and are skipped.
        """
        for j, (d, t) in enumerate(pairs):
            d = int(d)
            t = int(t)
            if d < 0 or t < 0:
                continue
            w = 1 if weights is None else int(weights[j])
            key = (d, t)
            if key in self.table:
                self.table[key] = min(self.table[key] + w, COUNT_MAX)
            elif len(self.table) < self.limit:
                self.table[key] = min(w, COUNT_MAX)
            else:
                self.n_dropped += 1

    def age(self):
        """Halve every count (floor) and forget the pairs that reach zero (R7)."""
        self.table = {k: c // 2 for k, c in self.table.items() if c // 2 > 0}

    def merge(self, other: "OCM"):
        """Add another memory's counts to this one: its pairs in sorted order, each with its count as
        the weight, under the same admission rule as any update (R3, R4)."""
        d, t, c = other.export()
        self.update(zip(d.tolist(), t.tolist()), weights=c.tolist())

    def export(self):
        """Sorted (draft, target, count) triples."""
        items = sorted((d, t, c) for (d, t), c in self.table.items())
        if not items:
            z = np.zeros(0, dtype=np.int64)
            return z, z.copy(), z.copy()
        a = np.asarray(items, dtype=np.int64)
        return a[:, 0], a[:, 1], a[:, 2]

    @property
    def n_keys(self) -> int:
        return len(self.table)


# ----------------------------------------------------------------------------
# one verification step (Algorithm 1, verification loop, greedy)
# ----------------------------------------------------------------------------
def verify(z: np.ndarray, draft: np.ndarray, ocm: OCM, tau: float, stats=None):
    """Verification-and-rescue pass over logits z[B, K+1, V] and draft[B, K].

    `stats` may carry precomputed (m, t, s) arrays of shape [B, K+1] (from
    `row_stats` or its C restatement); otherwise they are computed here.

    Returns a dict:
      accept_len[B]        n of Algorithm 1: leading positions accepted or rescued
      next_token[B]        t* of the failing position, or the bonus arg-max
      rescued_mask[B, K]   1 where a mismatch inside the accepted prefix was rescued
      rej_draft/rej_target[B, K]  pairs handed to UpdateMemory (-1 = none)
      m, s, lse, t [B, K+1]; zd, score, p_d, p_t [B, K] (float64); cnt [B, K]
      near_tie[B, K]       |score - tau| < 1e-5 at a mismatch
      bad_draft            number of draft ids outside [0, V)
    The memory is NOT modified; see `step`.
    """
    if not hasattr(z, "shape"):
        z = np.asarray(z)          # anything with .shape and [b, i, v] indexing will do (e.g. a lazy decoder)
    B, K1, V = z.shape
    K = K1 - 1
    draft = np.asarray(draft).reshape(B, K)
    lf = scg_threshold(tau)
    tau32 = float(np.float32(tau))

    m = np.empty((B, K1)); s = np.empty((B, K1)); lse = np.empty((B, K1))
    t = np.empty((B, K1), dtype=np.int64)
    if stats is not None:
        m[:], t[:], s[:] = stats
        with np.errstate(invalid="ignore", divide="ignore"):
            lse[:] = m + np.log(s)
    else:
        for b in range(B):
            for i in range(K1):
                m[b, i], t[b, i], s[b, i], lse[b, i] = row_stats(z[b, i])

    zd = np.full((B, K), np.nan); score = np.full((B, K), np.nan)
    p_d = np.full((B, K), np.nan); p_t = np.full((B, K), np.nan)
    cnt = np.zeros((B, K), dtype=np.int64)
    near = np.zeros((B, K), dtype=bool)
    accept_len = np.zeros(B, dtype=np.int32)
    next_token = np.zeros(B, dtype=np.int32)
    rescued = np.zeros((B, K), dtype=np.uint8)
    rej_d = np.full((B, K), -1, dtype=np.int32)
    rej_t = np.full((B, K), -1, dtype=np.int32)
    bad = 0

    # diagnostics for every position, whether or not the loop below reaches it
    with np.errstate(invalid="ignore", over="ignore", divide="ignore"):
        for b in range(B):
            for i in range(K):
                d = int(draft[b, i])
                p_t[b, i] = 1.0 / s[b, i]
                if 0 <= d < V:
                    zd[b, i] = float(z[b, i, d])
                    score[b, i] = np.exp(zd[b, i] - m[b, i])       # ratio of Eq. 3
                    p_d[b, i] = score[b, i] / s[b, i]
                    cnt[b, i] = ocm.count(d, t[b, i])

    for b in range(B):
        n = K
        for i in range(K):
            d = int(draft[b, i])
            tt = int(t[b, i])
            if d == tt:                          # exact match: accepted
                continue
            if not (0 <= d < V):                 # R5
                bad += 1
                n = i
                break
            is_freq = cnt[b, i] >= ocm.lam       # candidate proposal
            with np.errstate(invalid="ignore"):
                is_safe = bool((zd[b, i] - m[b, i]) >= lf)      # gate, Eq. 3 (R6)
            near[b, i] = abs(score[b, i] - tau32) < NEAR_TIE_BAND
            rej_d[b, i] = d                      # UpdateMemory is unconditional
            rej_t[b, i] = tt
            if is_freq and is_safe:              # rescued
                rescued[b, i] = 1
                continue
            n = i                                # un-rescued rejection ends the row
            break
        accept_len[b] = n
        next_token[b] = t[b, n]

    return dict(accept_len=accept_len, next_token=next_token, rescued_mask=rescued,
                rej_draft=rej_d, rej_target=rej_t, m=m, s=s, lse=lse, t=t,
                zd=zd, score=score, p_d=p_d, p_t=p_t, cnt=cnt, near_tie=near,
                bad_draft=bad)


def step(z, draft, ocm: OCM, tau: float, stats=None):
    """verify, then feed the step's rejections to the memory in (b, i) order (R2)."""
    out = verify(z, draft, ocm, tau, stats=stats)
    ocm.update(zip(out["rej_draft"].reshape(-1), out["rej_target"].reshape(-1)))
    return out
