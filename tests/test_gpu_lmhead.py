"""GPU parity of the step taken straight from the LM head (csd_verify_lmhead / csd_step_lmhead) against its
oracle: the logits are exact float64 products there, float32 tensor-core accumulations here.

Bar: every batch row whose result does not hang on a difference below the accumulation tolerance (the oracle
flags those: arg-max or gate margins within 2 tol) has identical accepted length, next token, rescue mask and
rejection list, and the memories agree; the reported logits (m, z_d) lie within tol = 2^-16 ||hidden row|| max
||weight row|| of the oracle's, arg-max indices agree on stable rows, and s, lse, score, p_d, p_t agree to the
relative accuracy that a logit error of tol allows (4 tol + 1e-5)."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import csd_lmhead_oracle as ORACLE
from paper_2604_13634_b200 import (LmheadBuffers, Ocm, csd_lmhead_set_pairing, csd_lmhead_shape, csd_set_overlap,
                                   csd_step_lmhead, csd_verify_lmhead)
from synth_inputs import WORKLOADS, Synth

pytestmark = pytest.mark.gpu

KERNELS = {"lone": 1, "pairs": 2}        # one block per SM / clusters of two blocks (csd_lmhead_set_pairing)


@pytest.fixture(autouse=True)
def _automatic_kernel_choice_afterwards():
    yield
    csd_lmhead_set_pairing(0)


def _f64(t):
    return t.detach().to("cpu").to(torch.float64).numpy()


def compare(buf, ref, K):
    g = lambda t: t.cpu().numpy()
    exc = ORACLE.rows_excused(ref)
    ok_rows = ~exc
    for k in ("accept_len", "next_token", "rescued_mask", "rej_draft", "rej_target"):
        got = g(getattr(buf, k))
        assert np.array_equal(got[ok_rows], ref[k][ok_rows]), k
    dg = {k: g(v) for k, v in buf.diag.items()}
    tol = ref["tol"]
    stable = ~ref["argmax_unstable"]
    assert np.array_equal(dg["t"][stable], ref["t"][stable]), "t"
    worst = float(np.max(np.abs(dg["m"] - ref["m"]) / tol))
    assert worst <= 1.0, f"m off by {worst} tol"
    zd_ok = ~np.isnan(ref["zd"])
    assert np.array_equal(np.isnan(dg["zd"]), ~zd_ok)
    if zd_ok.any():
        w2 = float(np.max(np.abs(dg["zd"][zd_ok] - ref["zd"][zd_ok]) / tol[:, :K][zd_ok]))
        assert w2 <= 1.0, f"zd off by {w2} tol"
        worst = max(worst, w2)
    rt_row = 4 * tol + 1e-5
    def close(name, got, want, rt):
        bad = ~(np.isnan(got) & np.isnan(want)) & ~(np.abs(got - want) <= rt * np.abs(want) + 1e-37)
        assert not bad.any(), f"{name}: {int(bad.sum())} off: {got[bad][:3]} vs {want[bad][:3]}"
    close("s", dg["s"], ref["s"], rt_row)
    close("lse", dg["lse"], ref["lse"], rt_row)
    st_pos = stable[:, :K]
    for name in ("score", "p_d", "p_t"):
        close(name, np.where(st_pos, dg[name], 0.0), np.where(st_pos, ref[name], 0.0), rt_row[:, :K])
    cnt = dg["cnt"].astype(np.int64) & 0xFFFFFFFF
    assert np.array_equal(cnt[st_pos], ref["cnt"][st_pos]), "cnt"
    return int(exc.sum()), worst


def resync(ocm, mem):
    rd, rt, rc = mem.export()
    ocm.reset()
    if len(rd):
        dev = ocm.device
        ocm.import_(torch.tensor(rd, dtype=torch.int32, device=dev), torch.tensor(rt, dtype=torch.int32, device=dev),
                    torch.tensor(rc.astype(np.int64), dtype=torch.int64, device=dev).to(torch.int32))


def compare_memory(ocm, mem):
    d, t, c = ocm.export()
    rd, rt, rc = mem.export()
    assert np.array_equal(d.numpy(), rd) and np.array_equal(t.numpy(), rt) and np.array_equal(c.numpy(), rc)
    st = ocm.stats()
    assert st["flags"] == 0, st
    return st


def lockstep(wl, H, steps, tau, lam, seed=0):
    syn = Synth(wl, seed, "cuda")
    W = syn.lmhead_weight(H)
    Wf = _f64(W)
    ocm, mem = Ocm(wl.ocm_slots, lam), ORACLE.OCM(wl.ocm_slots, lam)
    buf = LmheadBuffers(wl.B, wl.K, H, wl.V, diag=True)
    excused = rescued = accepted = 0
    worst = 0.0
    for s in range(steps):
        h, d = syn.step_lmhead(s % 3, W)                    # revisited inputs: their pairs reach lambda
        csd_step_lmhead(h, W, d, ocm, tau, buf)
        ref = ORACLE.step(_f64(h), Wf, d.cpu().numpy(), mem, tau)
        e, w = compare(buf, ref, wl.K)
        worst = max(worst, w)
        excused += e
        if e:
            resync(ocm, mem)
        compare_memory(ocm, mem)
        rescued += int(ref["rescued_mask"].sum())
        accepted += int(ref["accept_len"].sum())
    ocm.close()
    return dict(excused=excused, rescued=rescued, accepted=accepted, worst_logit_error_in_tol=worst)


SMALL = [(2, 3, 64, 96), (1, 1, 128, 1000), (5, 4, 256, 5000), (16, 7, 512, 4099), (7, 32, 128, 777), (32, 5, 1024, 20000),
         (42, 5, 320, 33000),      # 252 rows, two row tiles
         (64, 6, 256, 9000), (50, 8, 192, 5000), (128, 8, 128, 3000),      # 448, 450 and 1152 rows: two to five row groups
         (30, 9, 128, 2000)]                                               # 300 rows: a last group of 44


@pytest.mark.parametrize("kernel", list(KERNELS))
@pytest.mark.parametrize("B,K,H,V", SMALL)
def test_small_shapes(B, K, H, V, kernel):
    csd_lmhead_set_pairing(KERNELS[kernel])
    assert csd_lmhead_shape(B, K, H, V)["kernel"] == ("lmhead_stats_pair_kernel" if kernel == "pairs" else "lmhead_stats_kernel")
    wl = dataclasses.replace(WORKLOADS["batched_serving"], B=B, K=K, V=V, n_pairs=min(5000, V // 2), ocm_slots=4096)
    out = lockstep(wl, H, 4, 0.3, 1)
    assert out["excused"] <= max(1, B // 8), out
    print((B, K, H, V), csd_lmhead_shape(B, K, H, V), out)


@pytest.mark.parametrize("kernel", ["automatic"] + list(KERNELS))
def test_batched_serving_shape_with_a_llm_sized_head(kernel):
    """The serving workload with H = 4096: 192 logit rows, 151 936 tokens, a 1.2 GB weight matrix."""
    csd_lmhead_set_pairing(KERNELS.get(kernel, 0))
    wl = WORKLOADS["batched_serving"]
    out = lockstep(wl, 4096, 4, 0.3, 2)
    assert out["rescued"] > 0 and out["excused"] <= 2, out
    print(csd_lmhead_shape(wl.B, wl.K, 4096, wl.V), out)


@pytest.mark.parametrize("kps", [2, 4])
def test_more_k_blocks_per_stage(kps):
    from paper_2604_13634_b200 import csd_lmhead_set_tuning
    try:
        csd_lmhead_set_tuning(kps, 0)
        for (B, K, H, V) in ((16, 7, 512, 4099), (42, 5, 256, 33000), (64, 6, 256, 9000)):
            wl = dataclasses.replace(WORKLOADS["batched_serving"], B=B, K=K, V=V, n_pairs=min(5000, V // 2), ocm_slots=4096)
            out = lockstep(wl, H, 3, 0.3, 1)
            assert out["excused"] <= max(1, B // 8), out
    finally:
        csd_lmhead_set_tuning(0, 0)


@pytest.mark.parametrize("kernel", list(KERNELS))
@pytest.mark.parametrize("shape", [(8, 5, 512, 40000), (42, 5, 256, 33000), (64, 6, 256, 9000), (32, 5, 4096, 151936)])
def test_back_to_back_steps_with_step_overlap(shape, kernel):
    """csd_set_overlap on: the GEMM of a step is launched programmatically and may run beside the decisions and the
    update of the step before it; all steps share one workspace and one memory and are enqueued without a
    synchronisation in between.  Every step is compared with the oracle afterwards."""
    B, K, H, V = shape
    csd_lmhead_set_pairing(KERNELS[kernel])
    wl = dataclasses.replace(WORKLOADS["batched_serving"], B=B, K=K, V=V, n_pairs=min(5000, V // 2), ocm_slots=4096)
    syn = Synth(wl, 5, "cuda")
    W = syn.lmhead_weight(H)
    Wf = _f64(W)
    n_steps = 4 if V > 100000 else 8
    ins = [syn.step_lmhead(s % 3, W) for s in range(n_steps)]
    ocm, mem = Ocm(wl.ocm_slots, 1), ORACLE.OCM(wl.ocm_slots, 1)
    bufs = [LmheadBuffers(B, K, H, V, diag=True) for _ in range(n_steps)]
    for b in bufs[1:]:
        b.workspace, b.ws_bytes = bufs[0].workspace, bufs[0].ws_bytes
    torch.cuda.synchronize()
    # the full-size shape has near-ties (excused rows), after which a memory carried along may legitimately differ:
    # it runs the read-only call, where a near-tie stays in its own step
    carry = V < 100000
    try:
        csd_set_overlap(True)
        for (h, d), buf in zip(ins, bufs):
            (csd_step_lmhead if carry else csd_verify_lmhead)(h, W, d, ocm, 0.3, buf)
        torch.cuda.synchronize()
    finally:
        csd_set_overlap(False)
    excused = 0
    for (h, d), buf in zip(ins, bufs):
        ref = (ORACLE.step if carry else ORACLE.verify)(_f64(h), Wf, d.cpu().numpy(), mem, 0.3)
        e, _ = compare(buf, ref, K)
        excused += e
    if carry:
        assert excused == 0, "a near-tie in this seed: the memories cannot be compared step by step"
        compare_memory(ocm, mem)
    else:
        assert excused <= n_steps and ocm.stats()["flags"] == 0
    ocm.close()


@pytest.mark.parametrize("kernel", list(KERNELS))
def test_steps_captured_in_a_cuda_graph(kernel):
    """The three launches of a call can be captured (after one eager call has set the device up) and replayed:
    same bits as the eager call."""
    csd_lmhead_set_pairing(KERNELS[kernel])
    wl = dataclasses.replace(WORKLOADS["batched_serving"], B=24, K=5, V=20000, n_pairs=5000, ocm_slots=4096)
    syn = Synth(wl, 9, "cuda")
    W = syn.lmhead_weight(256)
    ins = [syn.step_lmhead(s, W) for s in range(3)]
    ocm = Ocm(wl.ocm_slots, 1)
    eager = [LmheadBuffers(wl.B, wl.K, 256, wl.V, diag=True) for _ in ins]
    for (h, d), buf in zip(ins, eager):
        csd_verify_lmhead(h, W, d, ocm, 0.3, buf)
    torch.cuda.synchronize()
    replayed = [LmheadBuffers(wl.B, wl.K, 256, wl.V, diag=True) for _ in ins]
    g, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for (h, d), buf in zip(ins, replayed):
                csd_verify_lmhead(h, W, d, ocm, 0.3, buf)
    for _ in range(2):
        g.replay()
    torch.cuda.synchronize()
    for a, b in zip(eager, replayed):
        for k in ("accept_len", "next_token", "rescued_mask", "rej_draft", "rej_target"):
            assert torch.equal(getattr(a, k), getattr(b, k)), k
        for k in a.diag:
            assert torch.equal(a.diag[k].view(torch.int32), b.diag[k].view(torch.int32)), k
    assert ocm.stats()["flags"] == 0
    ocm.close()


@pytest.mark.parametrize("kernel", list(KERNELS))
def test_other_mma_widths(kernel):
    """Tile widths other than the automatic cut: narrow, odd multiples of 16, the widest; ragged last tiles."""
    from paper_2604_13634_b200 import csd_lmhead_set_tuning
    csd_lmhead_set_pairing(KERNELS[kernel])
    try:
        for cols in (16, 48, 112, 256):
            csd_lmhead_set_tuning(0, cols)
            for (B, K, H, V) in ((5, 4, 256, 5000), (42, 5, 128, 33000), (50, 8, 192, 5000)):
                wl = dataclasses.replace(WORKLOADS["batched_serving"], B=B, K=K, V=V, n_pairs=min(5000, V // 2), ocm_slots=4096)
                out = lockstep(wl, H, 2, 0.3, 1)
                assert out["excused"] <= max(1, B // 8), out
    finally:
        csd_lmhead_set_tuning(0, 0)


@pytest.mark.parametrize("kernel", list(KERNELS))
def test_verify_is_read_only_reproducible_and_checks_its_arguments(kernel):
    from paper_2604_13634_b200 import CsdError
    csd_lmhead_set_pairing(KERNELS[kernel])
    wl = dataclasses.replace(WORKLOADS["batched_serving"], B=4, V=8192, n_pairs=2000)
    syn = Synth(wl, 3, "cuda")
    W = syn.lmhead_weight(256)
    h, d = syn.step_lmhead(0, W)
    ocm = Ocm(4096, 1)
    buf = LmheadBuffers(wl.B, wl.K, 256, wl.V, diag=True)
    csd_step_lmhead(h, W, d, ocm, 0.3, buf)
    before = [x.clone() for x in ocm.export()]
    csd_verify_lmhead(h, W, d, ocm, 0.3, buf)
    first = {k: v.clone() for k, v in buf.diag.items()}
    csd_verify_lmhead(h, W, d, ocm, 0.3, buf)
    assert all(torch.equal(a, b) for a, b in zip(before, ocm.export()))
    for k, v in buf.diag.items():
        assert torch.equal(v.view(torch.int32), first[k].view(torch.int32)), k       # bit-reproducible
    with pytest.raises(CsdError):
        LmheadBuffers(4, 5, 100, 8192)                     # H not a multiple of 64
    d2 = d.clone(); d2[0, 0] = wl.V; d2[1, 1] = -4         # bad draft ids: flagged, never rescued
    csd_verify_lmhead(h, W, d2, ocm, 0.0, buf)
    torch.cuda.synchronize()
    assert ocm.stats()["flags"] == 2 and buf.accept_len[0].item() == 0 and buf.accept_len[1].item() <= 1
    ocm.close()
