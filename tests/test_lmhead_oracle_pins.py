"""Pins of the LM-head form of the oracle (oracle/csd_lmhead_oracle.py), CPU only.

What fixes it from outside: the definition of a matrix product written as loops, selection matrices (the
logits are then a gather of the hidden values, so the step must equal the greedy oracle on the gathered
tensor), closed forms of the tolerance, float32 accumulations of the same products (which must stay inside
the tolerance the oracle grants them), constructed near-ties, and planted mistakes."""
import importlib.util

import numpy as np
import pytest

from oracle import csd_lmhead_oracle as ORACLE
from oracle import csd_oracle as GREEDY


def pin_product_is_the_definition(o):
    rng = np.random.default_rng(0)
    h = rng.normal(size=(2, 3, 5)); w = rng.normal(size=(7, 5))          # V = 7 != H = 5
    z = o.logits(h, w)
    assert z.shape == (2, 3, 7)
    for b in range(2):
        for i in range(3):
            for v in range(7):
                assert z[b, i, v] == pytest.approx(sum(h[b, i, k] * w[v, k] for k in range(5)), rel=1e-14, abs=1e-14)


def pin_selection_matrix_reduces_to_the_greedy_oracle(o):
    rng = np.random.default_rng(1)
    B, K, H, V = 3, 4, 12, 9
    h = rng.normal(size=(B, K + 1, H)) * 3
    perm = rng.permutation(H)[:V]
    w = np.zeros((V, H)); w[np.arange(V), perm] = 1.0                     # z[.., v] = h[.., perm[v]]
    zsel = h[..., perm]
    draft = np.where(rng.random((B, K)) < 0.5, zsel[:, :K].argmax(axis=2), rng.integers(0, V, size=(B, K)))
    mem_a, mem_b = o.OCM(64, 1), GREEDY.OCM(64, 1)
    for _ in range(4):
        a = o.step(h, w, draft, mem_a, 0.05)
        g = GREEDY.step(zsel, draft, mem_b, 0.05)
        for k in ("accept_len", "next_token", "rescued_mask", "rej_draft", "rej_target", "t", "cnt"):
            assert np.array_equal(a[k], g[k]), k
        for k in ("m", "s", "lse", "score", "p_d", "p_t", "zd"):
            np.testing.assert_allclose(a[k], g[k], rtol=1e-13, equal_nan=True)
    assert a["rescued_mask"].sum() > 0 and mem_a.table == mem_b.table


def pin_tolerance_closed_form_and_float32_accumulation(o):
    H = 4096
    assert o.tolerance(np.ones((1, 1, H)), np.ones((3, H)))[0, 0] == pytest.approx(2.0 ** -16 * H)
    assert o.tolerance(np.ones((1, 1, H)) * 2, np.vstack([np.ones(H), 3 * np.ones(H)]))[0, 0] == pytest.approx(2.0 ** -16 * 6 * H)
    # float32 accumulation of the exact products, in order and pairwise, stays well inside the tolerance
    import torch
    g = torch.Generator().manual_seed(5)
    h = torch.randn(6, H, generator=g).to(torch.bfloat16).to(torch.float64).numpy()
    w = (torch.randn(40, H, generator=g) / 64).to(torch.bfloat16).to(torch.float64).numpy()
    z = o.logits(h, w)
    tol = o.tolerance(h, w)
    prod = (h[:, None, :] * w[None, :, :]).astype(np.float32)              # bf16 x bf16 products are exact in float32
    assert np.array_equal(prod.astype(np.float64), h[:, None, :] * w[None, :, :])
    seq = np.zeros(prod.shape[:2], dtype=np.float32)
    for k in range(H):
        seq = seq + prod[:, :, k]
    pair = prod.sum(axis=2, dtype=np.float32)
    assert np.abs(seq - z).max() < 0.5 * tol.min() and np.abs(pair - z).max() < 0.25 * tol.min()
    assert np.abs(seq - z).max() > 0                                        # and float32 really is not float64


def pin_unstable_flags(o):
    H, V = 8, 6
    h = np.zeros((1, 3, H)); h[0, :, 0] = 1.0                              # z[.., v] = w[v, 0]
    w = np.zeros((V, H)); w[:, 0] = [5.0, 1.0, 4.0, 0.0, -1.0, 2.0]
    tol = o.tolerance(h, w)[0, 0]
    assert tol == pytest.approx(2.0 ** -16 * 5.0)
    draft = np.array([[0, 2]])
    out = o.verify(h, w, draft, o.OCM(64, 0), 0.3)
    assert not out["argmax_unstable"].any() and not out["gate_unstable"].any()
    assert out["accept_len"][0] == 2 and out["rescued_mask"].tolist() == [[0, 1]]     # 4 - 5 = -1 >= ln 0.3 = -1.204, lambda = 0
    out = o.verify(h, w, np.array([[0, 0]]), o.OCM(64, 0), 1.0)               # tau = 1: a match sits exactly on the threshold,
    assert not out["gate_unstable"].any() and out["accept_len"][0] == 2       # but a match never reaches the gate
    w2 = w.copy(); w2[2, 0] = 5.0 - 1.5 * tol                               # runner-up within 2 tol of the top
    out = o.verify(h, w2, draft, o.OCM(64, 0), 0.3)
    assert out["argmax_unstable"].all() and o.rows_excused(out)[0]
    w3 = w.copy(); w3[2, 0] = 5.0 + GREEDY.scg_threshold(0.3) + tol         # the gate's margin is one tol
    out = o.verify(h, w3, draft, o.OCM(64, 0), 0.3)
    assert out["gate_unstable"].tolist() == [[False, True]] and not out["argmax_unstable"].any() and o.rows_excused(out)[0]
    out = o.verify(h, w3, np.array([[3, 2]]), o.OCM(64, 2), 0.3)             # the row stops at position 0 (nothing stored)
    assert out["accept_len"][0] == 0 and out["gate_unstable"].tolist() == [[False, True]] and not o.rows_excused(out)[0]


PINS = [pin_product_is_the_definition, pin_selection_matrix_reduces_to_the_greedy_oracle,
        pin_tolerance_closed_form_and_float32_accumulation, pin_unstable_flags]


@pytest.mark.parametrize("pin", PINS, ids=[p.__name__ for p in PINS])
def test_pin(pin):
    pin(ORACLE)


MUTANTS = [
    ("weight not transposed", "return h @ w.T", "return (w @ h.reshape(-1, h.shape[-1]).T).T.reshape(h.shape[:-1] + (w.shape[0],))[..., ::-1]"),
    ("product in float32", "    h = np.asarray(hidden, dtype=np.float64)\n    w = np.asarray(weight, dtype=np.float64)\n    return h @ w.T",
     "    h = np.asarray(hidden, dtype=np.float16)\n    w = np.asarray(weight, dtype=np.float16)\n    return (h @ w.T).astype(np.float64)"),
    ("tolerance from the smallest weight row", "np.sqrt((w * w).sum(axis=-1)).max()", "np.sqrt((w * w).sum(axis=-1)).min()"),
    ("tolerance without the hidden norm", "return REL_TOL * np.sqrt((h * h).sum(axis=-1)) * ", "return REL_TOL * "),
    ("arg-max flag compares with the third logit", "top2 = np.partition(z, -2, axis=-1)[..., -2:]", "top2 = np.partition(z, -3, axis=-1)[..., [-3, -1]]"),
    ("gate flag on matches too", "out[\"gate_unstable\"] = mismatch & ~np.isnan(out[\"zd\"]) & (margin <= 2 * tol[:, :K])", "out[\"gate_unstable\"] = ~np.isnan(out[\"zd\"]) & (margin <= 2 * tol[:, :K])"),
    ("gate margin against zero", "margin = np.abs((out[\"zd\"] - out[\"m\"][:, :K]) - lf)", "margin = np.abs((out[\"zd\"] - out[\"m\"][:, :K]))"),
    ("excuse looks past the stop", "exc[b] = out[\"argmax_unstable\"][b, :n + 1].any() or out[\"gate_unstable\"][b, :min(n + 1, K)].any()",
     "exc[b] = out[\"argmax_unstable\"][b].any() or out[\"gate_unstable\"][b].any()"),
    ("update skipped", "    ocm.update(zip(out[\"rej_draft\"].reshape(-1), out[\"rej_target\"].reshape(-1)))\n    return out", "    return out"),
]


def _mutant(old, new):
    path = ORACLE.__file__
    src = open(path).read().replace("from . import csd_oracle as greedy", "from oracle import csd_oracle as greedy")
    src = src.replace("from .csd_oracle import", "from oracle.csd_oracle import")
    assert src.count(old) >= 1, f"mutation anchor not found: {old[:40]!r}"
    src = src.replace(old, new)
    spec = importlib.util.spec_from_loader("csd_lmhead_oracle_mutant", loader=None)
    mod = importlib.util.module_from_spec(spec)
    exec(compile(src, path + "<mutant>", "exec"), mod.__dict__)
    return mod


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistakes(name, old, new):
    mod = _mutant(old, new)
    caught = []
    for pin in PINS:
        try:
            pin(mod)
        except Exception:
            caught.append(pin.__name__)
            break
    assert caught, f"no pin notices the planted mistake: {name}"
