"""CPU oracle for the verification step taken straight from the LM head (logits never stored).

TEST INFRASTRUCTURE ONLY (same rules as csd_oracle.py, whose step it calls).

Algorithm 1 obtains the target distributions p_1 .. p_{gamma+1} from ONE parallel target pass; the last
operation of that pass is the LM head: z[r, v] = sum_h hidden[r, h] * W[v, h] for every position r and
token v.  This module states the verification step for a caller that hands over the inputs of that last
operation instead of its result: the logits are the exact products summed in float64, and everything after
them is the greedy oracle unchanged.

What is new is only a statement about rounding.  A float32 tensor-core accumulation does not reproduce the
float64 sums bit for bit, so a decision that hangs on a difference smaller than the accumulation error is
not determined by the paper's arithmetic.  The oracle therefore reports, per logit row, a tolerance
    tol[r] = REL_TOL * ||hidden[r]||_2 * max_v ||W[v]||_2
(REL_TOL = 2^-16: a sum of n = 4096 exact products accumulated in float32 is off by at most n 2^-24 times
the product of the norms in the worst case, 2^-12, and by about sqrt(n) 2^-24 = 2^-18 of it statistically;
2^-16 lies four times above the estimate and sixteen times below the worst case) and flags
    argmax_unstable[b, i]   the two largest logits of the row are closer than 2 tol
    gate_unstable[b, i]     |(z_d - z_t*) - ln tau| <= 2 tol at a mismatch
Results that depend on a flagged quantity are excluded from exactness by the tests (counted and reported);
everything else must equal this oracle exactly, and the reported logits (m, z_d) must lie within tol of it.
PARITY UNPINNED by the paper: it never states the precision of the target pass.
"""

from __future__ import annotations

import numpy as np

from . import csd_oracle as greedy
from .csd_oracle import OCM, bf16_bits_to_f64  # noqa: F401  (re-exported for the tests)

REL_TOL = 2.0 ** -16


def logits(hidden: np.ndarray, weight: np.ndarray) -> np.ndarray:
    """z[..., v] = sum_h hidden[..., h] * weight[v, h] in float64 (hidden [..., H], weight [V, H])."""
    h = np.asarray(hidden, dtype=np.float64)
    w = np.asarray(weight, dtype=np.float64)
    return h @ w.T


def tolerance(hidden: np.ndarray, weight: np.ndarray) -> np.ndarray:
    """tol[...] per logit row, see the module text."""
    h = np.asarray(hidden, dtype=np.float64)
    w = np.asarray(weight, dtype=np.float64)
    return REL_TOL * np.sqrt((h * h).sum(axis=-1)) * np.sqrt((w * w).sum(axis=-1)).max()


def verify(hidden, weight, draft, ocm: OCM, tau: float):
    """The greedy verification step on z = logits(hidden, weight), hidden [B, K+1, H], weight [V, H].

    Returns the greedy oracle's dict plus z (float64 [B, K+1, V]), tol [B, K+1], argmax_unstable [B, K+1]
    and gate_unstable [B, K].  The memory is not modified."""
    z = logits(hidden, weight)
    out = greedy.verify(z, draft, ocm, tau)
    tol = tolerance(hidden, weight)
    top2 = np.partition(z, -2, axis=-1)[..., -2:]
    out["z"] = z
    out["tol"] = tol
    out["argmax_unstable"] = (top2[..., 1] - top2[..., 0]) <= 2 * tol
    lf = greedy.scg_threshold(tau)
    K = z.shape[1] - 1
    with np.errstate(invalid="ignore"):
        margin = np.abs((out["zd"] - out["m"][:, :K]) - lf)
    mismatch = np.asarray(draft).reshape(z.shape[0], K) != out["t"][:, :K]
    out["gate_unstable"] = mismatch & ~np.isnan(out["zd"]) & (margin <= 2 * tol[:, :K])
    return out


def step(hidden, weight, draft, ocm: OCM, tau: float):
    """verify, then the memory update with the step's rejections in (b, i) order."""
    out = verify(hidden, weight, draft, ocm, tau)
    ocm.update(zip(out["rej_draft"].reshape(-1), out["rej_target"].reshape(-1)))
    return out


def rows_excused(out) -> np.ndarray:
    """Batch rows whose result may legitimately differ: an unstable quantity at or before the stop."""
    B, K = out["rescued_mask"].shape
    exc = np.zeros(B, dtype=bool)
    for b in range(B):
        n = int(out["accept_len"][b])
        exc[b] = out["argmax_unstable"][b, :n + 1].any() or out["gate_unstable"][b, :min(n + 1, K)].any()
    return exc
