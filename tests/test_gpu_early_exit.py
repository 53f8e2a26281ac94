"""csd_step_early_exit: the step in two phases (batch rows that stop within the first phase are not read any
further) must give exactly what csd_step gives -- accepted lengths, next tokens, masks, rejection lists, the
memory -- because Algorithm 1 never looks past a row's first un-rescued rejection."""
import dataclasses

import numpy as np
import pytest
import torch

import test_gpu_parity as T
from oracle import csd_oracle as ORACLE
from paper_2604_13634_b200 import EarlyExitBuffers, Ocm, csd_step_early_exit
from synth_inputs import WORKLOADS, Synth

pytestmark = pytest.mark.gpu


def check(buf, ref, first):
    """Outputs equal the oracle's; diagnostics are compared on the logit rows the two phases read."""
    g = lambda t: t.cpu().numpy()
    for k in ("accept_len", "next_token", "rescued_mask", "rej_draft", "rej_target"):
        assert np.array_equal(g(getattr(buf, k)), ref[k]), k
    if buf.diag is not None:
        B, K = ref["rescued_mask"].shape
        alive = ref["accept_len"] >= first
        rows_read = np.arange(K + 1)[None, :] <= np.where(alive, K, first)[:, None]
        pos_read = np.arange(K)[None, :] < np.where(alive, K, first)[:, None]
        dg = {k: g(v) for k, v in buf.diag.items()}
        assert np.array_equal(dg["t"][rows_read], ref["t"][rows_read]) and np.array_equal(dg["m"][rows_read].astype(np.float64), ref["m"][rows_read])
        np.testing.assert_allclose(dg["s"][rows_read], ref["s"][rows_read], rtol=1e-5)
        assert np.array_equal(dg["cnt"][pos_read].astype(np.int64) & 0xFFFFFFFF, ref["cnt"][pos_read])
        ok = pos_read & ~np.isnan(ref["zd"])
        assert np.array_equal(dg["zd"][ok].astype(np.float64), ref["zd"][ok])
        np.testing.assert_allclose(dg["score"][ok], ref["score"][ok], rtol=1e-5, atol=1e-37)


def lockstep(wl, steps, tau, lam, first, seed=0, diag=True, match_boost=0.0):
    syn = Synth(wl, seed, "cuda")
    ocm, mem = Ocm(wl.ocm_slots, lam), ORACLE.OCM(wl.ocm_slots, lam)
    buf = EarlyExitBuffers(wl.B, wl.K, wl.V, wl.torch_dtype, first=first, diag=diag)
    alive_rows = rows = 0
    f = first if first > 0 else max(1, (wl.K + 1) // 3)
    f = min(f, wl.K - 1)
    for s in range(steps):
        z, d = syn.step(s % 4)                    # revisits: pairs reach lambda, rescues keep rows alive
        csd_step_early_exit(z, d, ocm, tau, buf)
        ref = T.oracle_step(z, d, mem, tau)
        check(buf, ref, f)
        alive_rows += int((ref["accept_len"] >= f).sum())
        rows += wl.B
    st = T.compare_memory(ocm, mem)
    assert st["flags"] == 0 and st["steps"] == steps and st["positions"] == steps * wl.B * wl.K
    ocm.close()
    return alive_rows / rows


@pytest.mark.parametrize("B,K,V,dtype,first", [
    (3, 4, 5000, torch.float32, 0), (2, 5, 20000, torch.bfloat16, 1), (2, 5, 20000, torch.bfloat16, 4), (1, 2, 8, torch.bfloat16, 0),
    (4, 32, 3000, torch.bfloat16, 0), (4, 32, 3000, torch.bfloat16, 31), (5, 3, 70001, torch.float32, 2),
    (300, 3, 160, torch.float32, 0), (97, 8, 520, torch.bfloat16, 3), (2, 3, 4099, torch.float32, 0)])
def test_small_shapes(B, K, V, dtype, first):
    ocm, mem = Ocm(1024, 1), ORACLE.OCM(1024, 1)
    buf = EarlyExitBuffers(B, K, V, dtype, first=first, diag=True)
    f = min(first if first > 0 else max(1, (K + 1) // 3), K - 1)
    for rep in range(5):
        z, d = T._random_inputs(B, K, V, dtype, seed=200 + rep % 3, match_p=0.7)
        csd_step_early_exit(z, d, ocm, 1e-4, buf)
        check(buf, T.oracle_step(z, d, mem, 1e-4), f)
    T.compare_memory(ocm, mem)
    ocm.close()


def test_nobody_and_everybody_survives_the_first_phase():
    B, K, V = 6, 5, 9000
    z, d = T._random_inputs(B, K, V, torch.bfloat16, seed=9, match_p=1.0)          # every draft matches
    ocm, mem = Ocm(256, 1), ORACLE.OCM(256, 1)
    buf = EarlyExitBuffers(B, K, V, torch.bfloat16, first=2, diag=True)
    csd_step_early_exit(z, d, ocm, 0.3, buf)
    ref = T.oracle_step(z, d, mem, 0.3)
    check(buf, ref, 2)
    assert (ref["accept_len"] == K).all()
    d0 = ((d + 1) % V).contiguous()                                                   # nothing matches, nothing stored: all stop at 0
    csd_step_early_exit(z, d0, ocm, 0.3, buf)
    ref = T.oracle_step(z, d0, mem, 0.3)
    check(buf, ref, 2)
    assert (ref["accept_len"] == 0).all()
    csd_step_early_exit(z, d, ocm, 0.3, buf)                                          # and a full house again on the same buffers
    check(buf, T.oracle_step(z, d, mem, 0.3), 2)
    T.compare_memory(ocm, mem)
    ocm.close()


@pytest.mark.parametrize("name,steps,tau", [("tiny", 200, 0.3), ("single_stream", 60, 0.1), ("batched_serving", 40, 0.3),
                                             ("ocm_contention", 30, 0.3), ("large_batch", 6, 0.2)])
def test_workloads(name, steps, tau):
    wl = WORKLOADS[name]
    frac = lockstep(wl, steps, tau, lam=2, first=0)
    print(name, "batch rows alive after the first phase:", round(frac, 3))


def test_strided_views():
    B, K, V = 3, 6, 6000
    big, d = T._random_inputs(B, K, V + 24, torch.bfloat16, seed=7, match_p=0.8)
    d = (d % V).contiguous()
    for view in (big[:, :, :V], big[:, :, 1:V + 1], big[:, :, 8:V + 8]):
        ocm, mem = Ocm(256, 0), ORACLE.OCM(256, 0)
        buf = EarlyExitBuffers(B, K, V, torch.bfloat16, first=2, diag=True)
        csd_step_early_exit(view, d, ocm, 0.05, buf)
        check(buf, ORACLE.step(view.float().cpu().numpy(), d.cpu().numpy(), mem, 0.05), 2)
        T.compare_memory(ocm, mem)
        ocm.close()
