"""Several streams stepping on ONE memory at the same time (csd_ocm_set_shared).

The paper runs one sequence at a time and leaves concurrent updates of the memory open (Limitations).  The
library's reading: every recorded pair is counted exactly once whatever the interleaving; a look-up sees its
pair's count at some moment between the start and the end of its own step; the table never exceeds its key
limit.  What is unique is compared with the oracle exactly, the rest is checked for validity:
  * lambda = 0 (every divergence is a candidate: the gate alone decides) and lambda beyond any count (nothing is
    ever rescued) make every decision independent of the counts a look-up happens to see, so every step of
    every stream must equal the oracle's step, and the final table must equal the union of all recorded pairs;
  * with the paper's lambda = 6 the decisions depend on the interleaving; each step's outputs must then follow
    from the counts the step itself reports to have seen, those counts must lie between 0 and the final count,
    and the counts stored at the end must add up to the number of pairs recorded;
  * with a table far too small the key limit must hold and every recorded pair is either counted or dropped.
Nothing here waits on another stream inside a kernel: streams only share the table through atomics.
"""
import dataclasses

import numpy as np
import pytest
import torch

import test_gpu_parity as T
from oracle import csd_oracle as ORACLE
from paper_2604_13634_b200 import Ocm, StepBuffers, csd_set_overlap, csd_step
from synth_inputs import WORKLOADS, Synth

pytestmark = pytest.mark.gpu


def _run_streams(wl, n_streams, n_steps, lam, tau, slots=None, diag=True):
    """n_streams x n_steps steps, stream s stepping over its own inputs, all on one shared memory; the launches
    of different streams are issued round-robin without any synchronisation between them."""
    slots = slots or wl.ocm_slots
    ocm = Ocm(slots, lam)
    ocm.set_shared(True)
    streams = [torch.cuda.Stream() for _ in range(n_streams)]
    inputs = [[Synth(wl, 100 + s, "cuda").step(j) for j in range(n_steps)] for s in range(n_streams)]
    bufs = [[StepBuffers(wl.B, wl.K, wl.V, wl.torch_dtype, diag=diag) for _ in range(n_steps)] for _ in range(n_streams)]
    for s in range(n_streams):                       # one workspace per stream, its own output buffers per step
        for b in bufs[s][1:]:
            b.workspace, b.ws_bytes = bufs[s][0].workspace, bufs[s][0].ws_bytes
    torch.cuda.synchronize()
    try:
        csd_set_overlap(True)                        # one block per SM and launch: launches of several streams are resident together
        for j in range(n_steps):
            for s in range(n_streams):
                z, d = inputs[s][j]
                csd_step(z, d, ocm, tau, bufs[s][j], stream=streams[s])
        torch.cuda.synchronize()
    finally:
        csd_set_overlap(False)
    return ocm, inputs, bufs


def _export_dict(ocm):
    d, t, c = ocm.export()
    return {(int(a), int(b)): int(n) for a, b, n in zip(d, t, c)}


@pytest.mark.parametrize("n_streams", [2, 4])
@pytest.mark.parametrize("lam", [0, 2 ** 31])
def test_decisions_that_cannot_depend_on_the_interleaving(n_streams, lam):
    wl = WORKLOADS["ocm_contention"]
    n_steps = 6
    ocm, inputs, bufs = _run_streams(wl, n_streams, n_steps, lam, 0.3)
    union = ORACLE.OCM(wl.ocm_slots, lam)
    for s in range(n_streams):
        for j in range(n_steps):
            z, d = inputs[s][j]
            ref = T.oracle_step(z, d, union, 0.3)            # its look-ups cannot matter at these lambdas; its update builds the union
            got = bufs[s][j]
            for k in ("accept_len", "next_token", "rescued_mask", "rej_draft", "rej_target"):
                assert np.array_equal(getattr(got, k).cpu().numpy(), ref[k]), (s, j, k)
            assert np.array_equal(got.diag["t"].cpu().numpy(), ref["t"])
    st = T.compare_memory(ocm, union)                         # the multiset union, pair by pair
    assert st["flags"] == 0 and st["steps"] == n_streams * n_steps and st["n_dropped"] == 0
    final = _export_dict(ocm)
    for s in range(n_streams):                                # what a look-up saw lies between nothing and everything
        for j in range(n_steps):
            got = bufs[s][j]
            cnt = got.diag["cnt"].cpu().numpy().astype(np.int64) & 0xFFFFFFFF
            dd, tt = inputs[s][j][1].cpu().numpy(), got.diag["t"].cpu().numpy()[:, :wl.K]
            for b, i in zip(*np.nonzero(cnt)):
                assert cnt[b, i] <= final[(int(dd[b, i]), int(tt[b, i]))]
    if lam == 0:
        assert st["rescues"] > 0
    ocm.close()


@pytest.mark.parametrize("n_streams", [2, 4])
def test_interleaving_dependent_decisions_are_valid(n_streams):
    wl = WORKLOADS["ocm_contention"]
    n_steps = 10
    lam, tau = 6, 0.3
    ocm, inputs, bufs = _run_streams(wl, n_streams, n_steps, lam, tau)
    final = _export_dict(ocm)
    st = ocm.stats()
    assert st["flags"] == 0 and st["n_dropped"] == 0 and st["n_keys"] == len(final)
    assert sum(final.values()) == st["rejections"]            # every recorded pair counted exactly once
    lf = ORACLE.scg_threshold(tau)
    K = wl.K
    recorded = rescued = 0
    for s in range(n_streams):
        for j in range(n_steps):
            got = bufs[s][j]
            g = {k: v.cpu().numpy() for k, v in got.diag.items()}
            d = inputs[s][j][1].cpu().numpy()
            cnt = g["cnt"].astype(np.int64) & 0xFFFFFFFF
            ref = T.oracle_step(*inputs[s][j], ORACLE.OCM(64, lam), tau, update=False)      # t, m, zd do not depend on the memory
            assert np.array_equal(g["t"], ref["t"]) and np.array_equal(g["m"].astype(np.float64), ref["m"])
            assert np.array_equal(g["zd"].astype(np.float64), ref["zd"])
            for b in range(wl.B):
                n = K
                for i in range(K):
                    t = int(g["t"][b, i])
                    if d[b, i] == t:
                        assert got.rescued_mask[b, i].item() == 0 and got.rej_draft[b, i].item() == -1
                        continue
                    assert cnt[b, i] <= final.get((int(d[b, i]), t), 0)
                    assert got.rej_draft[b, i].item() == d[b, i] and got.rej_target[b, i].item() == t
                    recorded += 1
                    ok = cnt[b, i] >= lam and (float(g["zd"][b, i]) - float(g["m"][b, i])) >= lf
                    assert got.rescued_mask[b, i].item() == int(ok), (s, j, b, i)
                    if not ok:
                        n = i
                        break
                    rescued += 1
                assert got.accept_len[b].item() == n and got.next_token[b].item() == int(g["t"][b, n])
                assert (got.rej_draft[b, n + 1:] == -1).all() and (got.rescued_mask[b, n + 1:] == 0).all()
    assert recorded == st["rejections"] and rescued == st["rescues"] and rescued > 0
    ocm.close()


def test_key_limit_holds_under_concurrent_admission():
    wl = dataclasses.replace(WORKLOADS["ocm_contention"], V=32768)
    ocm, inputs, bufs = _run_streams(wl, 4, 12, 6, 0.3, slots=512, diag=False)
    final = _export_dict(ocm)
    st = ocm.stats()
    assert st["flags"] == 0 and st["n_keys"] == len(final) and 200 <= len(final) <= 256     # full (within the margin of claims in flight), never beyond the limit
    assert st["n_dropped"] > 0 and sum(final.values()) + st["n_dropped"] == st["rejections"]
    # back to a single writer: the ordered path carries on from the right key count
    ocm.set_shared(False)
    mem = ORACLE.OCM(512, 6)
    mem.table = dict(final)
    mem.n_dropped = st["n_dropped"]
    buf = StepBuffers(wl.B, wl.K, wl.V, wl.torch_dtype, diag=True)
    for j in range(3):
        z, d = inputs[0][j]
        csd_step(z, d, ocm, 0.3, buf)
        T.compare(buf, T.oracle_step(z, d, mem, 0.3))
    T.compare_memory(ocm, mem)
    ocm.close()


def test_concurrent_bulk_updates():
    """csd_ocm_update from four streams at once: every occurrence counted once."""
    g = torch.Generator(device="cuda").manual_seed(31)
    ocm = Ocm(1 << 16, 6)
    ocm.set_shared(True)
    mem = ORACLE.OCM(1 << 16, 6)
    streams = [torch.cuda.Stream() for _ in range(4)]
    batches = [(torch.randint(0, 120, (60000,), generator=g, device="cuda", dtype=torch.int32),
                torch.randint(0, 120, (60000,), generator=g, device="cuda", dtype=torch.int32)) for _ in range(12)]
    torch.cuda.synchronize()
    for k, (d, t) in enumerate(batches):
        ocm.update(d, t, stream=streams[k % 4])
    torch.cuda.synchronize()
    for d, t in batches:
        mem.update(zip(d.cpu().tolist(), t.cpu().tolist()))
    st = T.compare_memory(ocm, mem)
    assert st["n_dropped"] == 0 and st["flags"] == 0
    ocm.close()
