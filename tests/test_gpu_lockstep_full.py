"""Long lock-step runs of the full-size workloads: the CUDA path against the CPU oracle, step by step.

Every step's accepted lengths, next tokens, rescue masks and rejection lists must equal the oracle's;
the diagnostics (t*, m, z_d, counts exact; s, lse, score, p_d, p_t within 1e-5) are compared on the first
100 steps and every 100th after; the memory's (pair, count) set, n_keys and n_dropped at every checkpoint
and at the end.  Each workload runs in both launch shapes: a step that runs alone (four blocks per SM)
and the shape the benchmark times (step overlap on: one block per SM and launch, programmatic launches).
The stochastic step (Algorithm 1 at T > 0) is checked on whole steps of the largest workload.
"""
import numpy as np
import pytest
import torch

import lockstep_run as LR
import test_gpu_sampled_parity as S
from paper_2604_13634_b200 import Ocm, SampledBuffers, csd_set_overlap, csd_step_sampled
from synth_inputs import WORKLOADS, Synth

pytestmark = pytest.mark.gpu


def _run(name, tau, steps, checkpoint, overlap, prewarm_steps=0):
    wl = WORKLOADS[name]
    try:
        csd_set_overlap(overlap)
        LR.OVERLAP = overlap
        out = LR.run(wl, tau, steps, checkpoint, prewarm_steps)
    finally:
        csd_set_overlap(False)
        LR.OVERLAP = False
    assert out["verdict"] == "identical" and out["rescued"] > 0
    print(out)
    return out


@pytest.mark.parametrize("overlap", [False, True], ids=["alone", "overlap"])
@pytest.mark.parametrize("tau", [0.2, 0.4])
def test_large_batch(tau, overlap):
    out = _run("large_batch", tau, 150, 50, overlap)             # 200 000-pair pre-warm inside; 153 600 positions
    assert out["n_keys"] > 5000


@pytest.mark.parametrize("overlap", [False, True], ids=["alone", "overlap"])
def test_batched_serving(overlap):
    _run("batched_serving", 0.3, 2000, 250, overlap)             # 320 000 positions


@pytest.mark.parametrize("overlap", [False, True], ids=["alone", "overlap"])
def test_ocm_contention(overlap):
    out = _run("ocm_contention", 0.3, 1500, 100, overlap)        # 576 000 positions, memory compared every 100 steps
    assert out["checkpoints"] == 15


@pytest.mark.parametrize("overlap", [False, True], ids=["alone", "overlap"])
@pytest.mark.parametrize("tau", [0.1, 0.3, 0.5])
def test_single_stream(tau, overlap):
    _run("single_stream", tau, 3000, 500, overlap, prewarm_steps=500)


def _oracle_sampled_by_rows(z, y, d, r, seed, T, mem, tau, rows_at_a_time=16):
    """The stochastic oracle on a whole step, a few batch rows at a time (bounds the float64 copies): batch rows
    are independent given the memory snapshot; each keeps the clock streams of its own row index; the memory
    is updated afterwards with the recorded pairs in (b, i) order, as the oracle's own `step` does."""
    B, K1, _ = z.shape
    parts = []
    orig = S.ORACLE.race_clocks
    try:
        for b0 in range(0, B, rows_at_a_time):
            S.ORACLE.race_clocks = lambda s, row, stream, first, n, b0=b0: orig(s, row + b0 * K1, stream, first, n)
            sl = slice(b0, b0 + rows_at_a_time)
            parts.append(S.ORACLE.verify(S._f64(z[sl]), S._f64(y[sl]), d[sl].cpu().numpy(), r[sl].cpu().numpy(), seed, T, mem, tau))
    finally:
        S.ORACLE.race_clocks = orig
    out = {k: np.concatenate([p[k] for p in parts], axis=0) for k in parts[0]}
    mem.update(zip(out["rej_draft"].reshape(-1), out["rej_target"].reshape(-1)))
    return out


@pytest.mark.parametrize("name,steps,T", [("large_batch", 4, 0.3), ("ocm_contention", 12, 0.3), ("batched_serving", 40, 0.3)])
def test_stochastic_whole_steps(name, steps, T):
    """Whole stochastic steps of the full-size workloads, every batch row, memory carried from step to step."""
    wl = WORKLOADS[name]
    syn = Synth(wl, 1, "cuda")
    ocm, mem = Ocm(wl.ocm_slots, 2), S.ORACLE.OCM(wl.ocm_slots, 2)
    buf = SampledBuffers(wl.B, wl.K, wl.V, wl.torch_dtype)
    excused = rescued = failed = 0
    for s in range(steps):
        z, y, d, r = syn.step_sampled(s % 3)             # revisited inputs: their pairs reach lambda, rescues follow
        csd_step_sampled(z, y, d, r, 4000 + s, T, ocm, 0.2, buf)
        ref = _oracle_sampled_by_rows(z, y, d, r, 4000 + s, T, mem, 0.2)
        e = S.compare(buf, ref)
        excused += e
        if e:
            S.resync(ocm, mem)
        S.compare_memory(ocm, mem)
        rescued += int(ref["rescued_mask"].sum())
        failed += int((~ref["accepted"]).sum())
    st = ocm.stats()
    assert st["flags"] == 0 and failed > 0 and rescued > 0
    assert excused <= max(1, steps * wl.B // 500), excused
    print(name, dict(steps=steps, positions=steps * wl.B * wl.K, failed=failed, rescued=rescued, excused=excused))
    ocm.close()
